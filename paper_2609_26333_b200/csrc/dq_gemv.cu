// LUT3 weight-only decode mat-vec / skinny GEMM (App. C.2 "Kernel specification"):
//   Y[b][n] = bf16( s * sum_blk d_blk * sum_{k in blk} G[idx(n,k)] * X[b][k] )
// Weights stream from HBM as 3 bit-planes + one signed E4M3 scale per 16
// (3.5 bit per weight); dequantisation happens in registers, accumulation in fp32.
#include "dq_common.cuh"

namespace dq {

__device__ __forceinline__ float e4m3_to_f32_gemv(uint32_t b)
{
    unsigned short in = (unsigned short)(b & 0xFFu);
    unsigned int h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(in));
    return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

// One warp per weight row; lane l walks the 128-weight chunks l, l+32, ...
// Each chunk is 3 x 16 B of bit-planes (plane-major) and 8 scale bytes.
template <int BT>
__global__ void __launch_bounds__(256) gemv_lut3_kernel(const uint32_t *__restrict__ planes,
                                                        const uint8_t *__restrict__ sf,
                                                        const PackedHeader *__restrict__ hdr,
                                                        const __nv_bfloat16 *__restrict__ X, int64_t ldx, int B,
                                                        __nv_bfloat16 *__restrict__ Y, int64_t ldy, int64_t N,
                                                        int64_t K)
{
    __shared__ float lut[8];
    if (threadIdx.x < 8) lut[threadIdx.x] = hdr->lut_levels[threadIdx.x];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int warps_per_block = blockDim.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    const int b0 = blockIdx.y * BT;
    if (row >= N) return;
    const int64_t nchunks = K / kLutChunk;
    float acc[BT];
#pragma unroll
    for (int t = 0; t < BT; ++t) acc[t] = 0.0f;

    for (int64_t c = lane; c < nchunks; c += 32) {
        const uint4 *pp = reinterpret_cast<const uint4 *>(planes + (row * nchunks + c) * 12);
        const uint4 q0 = __ldg(pp), q1 = __ldg(pp + 1), q2 = __ldg(pp + 2);
        const uint2 sc = __ldg(reinterpret_cast<const uint2 *>(sf + row * (K / 16) + c * 8));
        const uint32_t P0[4] = {q0.x, q0.y, q0.z, q0.w};
        const uint32_t P1[4] = {q1.x, q1.y, q1.z, q1.w};
        const uint32_t P2[4] = {q2.x, q2.y, q2.z, q2.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int blk = w * 2 + h;
                const uint32_t d8 = ((blk < 4 ? sc.x : sc.y) >> (8 * (blk & 3))) & 0xFFu;
                const float d = e4m3_to_f32_gemv(d8);
                float g[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int bit = h * 16 + i;
                    const uint32_t idx = ((P0[w] >> bit) & 1u) | (((P1[w] >> bit) & 1u) << 1) |
                                         (((P2[w] >> bit) & 1u) << 2);
                    g[i] = lut[idx];
                }
#pragma unroll
                for (int t = 0; t < BT; ++t) {
                    if (b0 + t < B) {
                        const uint4 *xp = reinterpret_cast<const uint4 *>(X + (int64_t)(b0 + t) * ldx + c * kLutChunk +
                                                                          w * 32 + h * 16);
                        const uint4 xa = __ldg(xp), xb = __ldg(xp + 1);
                        const uint32_t xw[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
                        float part = 0.0f;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            part = fmaf(g[2 * i], __uint_as_float(xw[i] << 16), part);
                            part = fmaf(g[2 * i + 1], __uint_as_float(xw[i] & 0xFFFF0000u), part);
                        }
                        acc[t] = fmaf(d, part, acc[t]);
                    }
                }
            }
        }
    }
    const float s = hdr->s;
#pragma unroll
    for (int t = 0; t < BT; ++t) {
        float v = acc[t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0 && b0 + t < B) Y[(int64_t)(b0 + t) * ldy + row] = __float2bfloat16_rn(v * s);
    }
}

cudaError_t launch_gemv_lut3(const GemvArgs &a, cudaStream_t stream)
{
    const int warps = 8;
    const __nv_bfloat16 *X = reinterpret_cast<const __nv_bfloat16 *>(a.X);
    __nv_bfloat16 *Y = reinterpret_cast<__nv_bfloat16 *>(a.Y);
    dim3 block(warps * 32);
    const unsigned gx = (unsigned)((a.N + warps - 1) / warps);
    const int B = (int)a.B;
    if (B == 1) {
        gemv_lut3_kernel<1><<<dim3(gx, 1), block, 0, stream>>>(a.planes, a.sf, a.hdr, X, a.ldx, B, Y, a.ldy, a.N, a.K);
    } else if (B == 2) {
        gemv_lut3_kernel<2><<<dim3(gx, 1), block, 0, stream>>>(a.planes, a.sf, a.hdr, X, a.ldx, B, Y, a.ldy, a.N, a.K);
    } else {
        gemv_lut3_kernel<4><<<dim3(gx, (B + 3) / 4), block, 0, stream>>>(a.planes, a.sf, a.hdr, X, a.ldx, B, Y, a.ldy,
                                                                        a.N, a.K);
    }
    return cudaGetLastError();
}

}  // namespace dq
