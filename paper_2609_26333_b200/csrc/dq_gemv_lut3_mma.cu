// LUT3 decode with the products on tensor cores (App. C.2 kernel specification; the
// skinny-batch case the paper leaves open, Sec. 5):
//   Y[b][n] = bf16( s * sum_k d_blk(n,k) * G[idx(n,k)] * X[b][k] ),   up to eight batch columns per pass.
// Same skeleton as the NVFP4 tensor-core decode kernel: a warp owns 16 consecutive rows and a 1024-weight
// slice of K; lane (g, t) of the mma fragment layout holds rows g / g+8 and, per 512-weight half slice, four
// consecutive plane words (128 weights) of each row; mma i contracts every lane's weights 4 i .. 4 i + 3.
// Dequantisation without shared memory: the device bit order stores indices as nibbles, which are the
// selectors of byte-permute; the eight fp16 levels live in four registers (low bytes, high bytes), two
// permutes look up the bytes of four weights and two more interleave them into two fp16 pairs.  The block
// scale is applied in fp16: hi = rn(level * d) goes through mma.sync.m16n8k16 with fp32 accumulation.  For
// K < 2048 the exact remainder lo = level * d - hi (one fused multiply-add) goes through a second mma, so that
// nothing is lost.  For K >= 2048 it is left out: the per-weight rounding errors (relative 2^-11 at most,
// independent) add a standard deviation of about 2e-4 * rms|a w| * sqrt(K) to a sum whose tolerance is
// 1e-4 * K * mean|a w|, i.e. 3.3 / sqrt(K) of it; measured, the largest error-to-tolerance ratio over whole
// layers is the same with and without the remainder from K = 1024 on (0.46: the bf16 rounding of the output).
// Activations: power-of-two scaling, fp16 in shared memory, one 8-byte load per mma (pair).
// Used from batch 2 on (the batch rides along in the B operand) and at batch 1 for 2048 <= K <= 16384, where it
// is faster than the CUDA-core kernel (28672x8192: 39.6 against 45.3 us).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_common.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

constexpr int kSlots = 4;                         // cross-warp reduction slots per row group
constexpr uint32_t kRedAddr = 0x1000;             // shared-window address of [G][kSlots][W][32 lanes][4] floats
constexpr uint32_t kSmemLimit = 227 * 1024;       // the x columns follow the reduction buffers, up to this window address

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t hmul2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
// a * b - h on both halves (h = rn(a * b): the result is the exact rounding error of the product)
__device__ __forceinline__ uint32_t hres2(uint32_t a, uint32_t b, uint32_t h)
{
    uint32_t r;
    asm("{\n\t.reg .b32 n;\n\tneg.f16x2 n, %3;\n\tfma.rn.f16x2 %0, %1, %2, n;\n\t}" : "=r"(r) : "r"(a), "r"(b), "r"(h));
    return r;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

// one 512-weight half slice of rows g / g+8: four plane words per plane and eight scale bytes per row
struct HalfRegs { uint4 p[2][3]; uint2 sc[2]; };

template <int MAXT>
__global__ void __launch_bounds__(MAXT, 1)
gemv_lut3_mma_kernel(const uint8_t *__restrict__ lut, const PackedHeader *__restrict__ hdr,
                     const __nv_bfloat16 *__restrict__ X, int64_t ldx, int b0, int cols,
                     __nv_bfloat16 *__restrict__ Y, int64_t ldy, int N, int K, int W, int G, uint32_t col_stride,
                     uint32_t x_addr, StatusWord *status, int hi_only)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const uint32_t win0 = (uint32_t)__cvta_generic_to_shared(smem_raw);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw);
    volatile int *sync_words = reinterpret_cast<volatile int *>(smem_raw + 64);          // [G][kSlots] x (generation, count)
    float *xmax_s = reinterpret_cast<float *>(smem_raw + 768);                          // 32 per-warp maxima
    if (win0 + 1024 > kRedAddr) {
        if (threadIdx.x == 0) { atomicExch(&status->status, (int)DQ_ERR_INTERNAL); atomicExch(&status->detail, 0x35000); }
        return;
    }
    float *red = reinterpret_cast<float *>(smem_raw + (kRedAddr - win0));
    uint8_t *xh = smem_raw + (x_addr - win0);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int grp = warp / W;
    const int w = warp - grp * W;
    const int g = lane >> 2, t = lane & 3;
    const int slices = W;                                   // ceil(K / 1024)
    const int kpad = slices * 1024;

    if (threadIdx.x < 16 * kSlots * 2) sync_words[threadIdx.x] = 0;
    if (threadIdx.x == 0) *abort_flag = 0;
    // the eight fp16 levels as byte-permute tables: low bytes of levels 0-3 / 4-7, high bytes of levels 0-3 / 4-7
    uint32_t tl0 = 0, tl1 = 0, th0 = 0, th1 = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        tl0 |= (hdr->lut_f16[j] & 0xFFu) << (8 * j);
        th0 |= ((hdr->lut_f16[j] >> 8) & 0xFFu) << (8 * j);
        tl1 |= (hdr->lut_f16[4 + j] & 0xFFu) << (8 * j);
        th1 |= ((hdr->lut_f16[4 + j] >> 8) & 0xFFu) << (8 * j);
    }

    const int ntiles = N / 16;                              // N % 16 == 0
    const int stride = gridDim.x * G;
    const int first = blockIdx.x * G + grp;

    auto load_half = [&](HalfRegs &R, int tile, int h) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int row = tile * 16 + g + 8 * half;
            const uint8_t *blk = lut + ((size_t)row * slices + w) * kLutBlockBytes;
#pragma unroll
            for (int p = 0; p < 3; ++p)
                R.p[half][p] = __ldg(reinterpret_cast<const uint4 *>(blk + p * 128 + h * 64 + t * 16));
            R.sc[half] = __ldg(reinterpret_cast<const uint2 *>(blk + kLutScaleOff + h * 32 + t * 8));
        }
    };
    // Register ring of two half slices: position p of the warp's stream is half p % 2 of tile first + (p / 2) * stride.
    // The weights are constant data: start streaming before waiting for the kernel ahead of this one.
    HalfRegs ring[2];
#pragma unroll
    for (int p = 0; p < 2; ++p) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            ring[p].sc[half] = make_uint2(0, 0);
#pragma unroll
            for (int q = 0; q < 3; ++q) ring[p].p[half][q] = make_uint4(0, 0, 0, 0);
        }
        if (first < ntiles) load_half(ring[p], first, p);
    }

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- activations of this pass: largest magnitude -> power-of-two scale -> fp16 in shared memory
    float m = 0.0f;
    for (int c = 0; c < cols; ++c) {
        const uint4 *xp = reinterpret_cast<const uint4 *>(X + (int64_t)(b0 + c) * ldx);
        for (int i = threadIdx.x; i < K / 8; i += blockDim.x) {
            const uint4 v = __ldg(xp + i);
            // |bf16| pairs compare like unsigned integers once the sign bits are cleared
            const uint32_t a0 = v.x & 0x7FFF7FFFu, a1 = v.y & 0x7FFF7FFFu, a2 = v.z & 0x7FFF7FFFu, a3 = v.w & 0x7FFF7FFFu;
            const uint32_t hi = max(max(a0 >> 16, a1 >> 16), max(a2 >> 16, a3 >> 16));
            const uint32_t lo = max(max(a0 & 0xFFFFu, a1 & 0xFFFFu), max(a2 & 0xFFFFu, a3 & 0xFFFFu));
            m = fmaxf(m, __uint_as_float(max(hi, lo) << 16));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) xmax_s[warp] = m;
    __syncthreads();
    m = 0.0f;
    for (int i = 0; i < nwarps; ++i) m = fmaxf(m, xmax_s[i]);
    int ex = (int)((__float_as_uint(m) >> 23) & 0xFFu) - 127;           // floor(log2(max)); -127 for zero / subnormal
    ex = max(-100, min(100, ex));
    const float xscale = __uint_as_float((uint32_t)(127 + 14 - ex) << 23);   // 2^(14 - ex)
    const float xinv = __uint_as_float((uint32_t)(127 - 14 + ex) << 23);
    for (int c = 0; c < cols; ++c) {
        const uint4 *xp = reinterpret_cast<const uint4 *>(X + (int64_t)(b0 + c) * ldx);
        for (int i = threadIdx.x; i < kpad / 8; i += blockDim.x) {
            uint32_t r[4] = {0u, 0u, 0u, 0u};                       // the padding of a short last slice reads as zero
            if (i < K / 8) {
                const uint4 v = __ldg(xp + i);
                const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int z = 0; z < 4; ++z) {
                    const __half2 h = __floats2half2_rn(__uint_as_float(ww[z] << 16) * xscale,
                                                        __uint_as_float(ww[z] & 0xFFFF0000u) * xscale);
                    r[z] = *reinterpret_cast<const uint32_t *>(&h);
                }
            }
            // Inside a 512-weight half slice lane t owns weights 128 t .. 128 t + 127; the four weights
            // 128 t + 32 wi + 4 i .. + 3 (word wi, mma i of that word) sit at byte 256 wi + 32 i + 8 t, so that the
            // B-fragment reads of one mma (lanes t, columns g 32 bytes apart mod 128) hit distinct banks.
            const int k0 = i * 8;
            const int hs = k0 >> 9, tt = (k0 >> 7) & 3, wi = (k0 >> 5) & 3, ii = (k0 & 31) >> 2;
            uint8_t *dst = xh + (size_t)c * col_stride + (size_t)hs * 1024 + wi * 256 + ii * 32 + tt * 8;
            *reinterpret_cast<uint2 *>(dst) = make_uint2(r[0], r[1]);
            *reinterpret_cast<uint2 *>(dst + 32) = make_uint2(r[2], r[3]);
        }
    }
    __syncthreads();
    const float out_scale = hdr->s * xinv;
    const uint32_t xlane = x_addr + (uint32_t)((g < cols) ? g : 0) * col_stride + (uint32_t)t * 8 + (uint32_t)w * 2048;

    bool ok = true;
    int it = 0;
    for (int tile = first; tile < ntiles; tile += stride, ++it) {
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            HalfRegs &cur = ring[h];
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                uint32_t pw[2][3], dA[2], dB[2];
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const uint4 q0 = cur.p[half][0], q1 = cur.p[half][1], q2 = cur.p[half][2];
                    pw[half][0] = wi == 0 ? q0.x : wi == 1 ? q0.y : wi == 2 ? q0.z : q0.w;
                    pw[half][1] = wi == 0 ? q1.x : wi == 1 ? q1.y : wi == 2 ? q1.z : q1.w;
                    pw[half][2] = wi == 0 ? q2.x : wi == 1 ? q2.y : wi == 2 ? q2.z : q2.w;
                    const uint32_t scw = (wi < 2) ? (cur.sc[half].x >> (16 * wi)) : (cur.sc[half].y >> (16 * (wi - 2)));
                    uint32_t d2;
                    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(d2) : "h"((unsigned short)scw));
                    dA[half] = __byte_perm(d2, d2, 0x1010);          // first block of the word on both halves
                    dB[half] = __byte_perm(d2, d2, 0x3232);          // second block
                }
                const uint32_t xa = xlane + (uint32_t)h * 1024 + (uint32_t)wi * 256;
                uint32_t sel[2][4];
                lut3_selectors(pw[0][0], pw[0][1], pw[0][2], sel[0]);
                lut3_selectors(pw[1][0], pw[1][1], pw[1][2], sel[1]);
#pragma unroll
                for (int gg = 0; gg < 4; ++gg) {                     // weights 8 gg .. 8 gg + 7: mmas 2 gg and 2 gg + 1
                    const uint32_t d0 = (gg < 2) ? dA[0] : dB[0], d1 = (gg < 2) ? dA[1] : dB[1];
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {                 // four weights (two pairs) of each row per mma
                        const uint32_t s0 = jj ? (sel[0][gg] >> 16) : sel[0][gg];
                        const uint32_t s1 = jj ? (sel[1][gg] >> 16) : sel[1][gg];
                        const uint32_t lo0 = __byte_perm(tl0, tl1, s0), hi0 = __byte_perm(th0, th1, s0);   // row g
                        const uint32_t lo1 = __byte_perm(tl0, tl1, s1), hi1 = __byte_perm(th0, th1, s1);   // row g + 8
                        const uint32_t v0 = __byte_perm(lo0, hi0, 0x5140), v2 = __byte_perm(lo0, hi0, 0x7362);
                        const uint32_t v1 = __byte_perm(lo1, hi1, 0x5140), v3 = __byte_perm(lo1, hi1, 0x7362);
                        const uint32_t h0 = hmul2(v0, d0), h1 = hmul2(v1, d1), h2 = hmul2(v2, d0), h3 = hmul2(v3, d1);
                        const uint2 xv = lds_v2(xa + (uint32_t)(2 * gg + jj) * 32);
                        mma16816(acc, h0, h1, h2, h3, xv.x, xv.y);
                        if (!hi_only) mma16816(acc, hres2(v0, d0, h0), hres2(v1, d1, h1), hres2(v2, d0, h2), hres2(v3, d1, h3), xv.x, xv.y);
                    }
                }
            }
            // the slot is consumed: refill it with the same half of the warp's next tile (the other half
            // slice, loaded one step earlier, is what the warp works on meanwhile)
            if (tile + stride < ntiles) load_half(cur, tile + stride, h);
        }
        // ---- cross-warp sum: last-arriving warp of the group adds the W partial fragments in order and stores
        const int slot = it & (kSlots - 1);
        volatile int *gen = sync_words + (grp * kSlots + slot) * 2;
        int *cnt = const_cast<int *>(gen) + 1;
        if (ok) {
            uint32_t good = 1;
            if (lane == 0) {
                const int want = it / kSlots;
                long long t0 = 0;
                uint32_t spins = 0;
                while (*gen != want) {
                    if ((++spins & 255u) == 0u) {
                        if (t0 == 0) t0 = clock64();
                        if (*abort_flag || clock64() - t0 > tc::kWaitBudgetCycles) { *abort_flag = 1; good = 0; break; }
                    }
                }
            }
            ok = __shfl_sync(0xffffffffu, good, 0) != 0;
        }
        float4 *rbuf = reinterpret_cast<float4 *>(red) + (size_t)((grp * kSlots + slot) * W) * 32;
        rbuf[w * 32 + lane] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        __syncwarp();
        int prev = 0;
        if (lane == 0) { __threadfence_block(); prev = atomicAdd(cnt, 1); }
        prev = __shfl_sync(0xffffffffu, prev, 0);
        if (prev == W - 1) {
            __threadfence_block();
            float tot[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            for (int ww = 0; ww < W; ++ww) {
                const volatile float *p = reinterpret_cast<const volatile float *>(rbuf + ww * 32 + lane);
                tot[0] += p[0]; tot[1] += p[1]; tot[2] += p[2]; tot[3] += p[3];
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {                    // c0, c1: row g, columns 2t, 2t+1; c2, c3: row g + 8
                const int col = 2 * t + (j & 1);
                const int row = tile * 16 + g + 8 * (j >> 1);
                if (ok && col < cols) Y[(int64_t)(b0 + col) * ldy + row] = __float2bfloat16_rn(tot[j] * out_scale);
            }
            __syncwarp();
            if (lane == 0) { *cnt = 0; __threadfence_block(); *gen = it / kSlots + 1; }
        }
    }
    if (*abort_flag && lane == 0) {
        atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
        atomicExch(&status->detail, 0x36000 | (int)blockIdx.x);
    }
}

template <int MAXT>
cudaError_t launch_one(const GemvArgs &a, int b0, int cols, int grid, int threads, int W, int G, uint32_t col_stride,
                       uint32_t x_addr, uint32_t smem, cudaStream_t stream)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(gemv_lut3_mma_kernel<MAXT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_lut3_mma_kernel<MAXT>, a.lut, a.hdr, reinterpret_cast<const __nv_bfloat16 *>(a.X),
                              (int64_t)a.ldx, b0, cols, reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.N,
                              (int)a.K, W, G, col_stride, x_addr, a.status, 0);
}

}  // namespace

// Whether dq_decode_linear should take this kernel rather than the CUDA-core one.  Two and more columns: always
// (the batch rides along in the B operand).  Batch 1: where it was measured faster, i.e. K from 2048 (one mma per
// step) to 16384 (at most 16 slice warps per row group) and a tile count that fills the last round of the grid:
// with 16-row tiles a 5120-row layer leaves half of the SMs idle in its second round, where the CUDA-core kernel
// works in 4-row units.
bool gemv_lut3_mma_preferred(int64_t N, int64_t K, int64_t B)
{
    if (B >= 2) return true;
    if (K < 2048 || K > 16384) return false;
    const int W = (int)((K + 1023) / 1024);
    int G = 20 / W;
    if (G < 1) G = 1;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t ntiles = N / 16;
    int64_t grid = (ntiles + G - 1) / G;
    if (grid > sms) grid = sms;
    const int64_t groups = grid * G;
    const int64_t rounds = (ntiles + groups - 1) / groups;
    return (double)ntiles / (double)(rounds * groups) >= 0.85;
}

// up to eight columns per pass on tensor cores
cudaError_t launch_gemv_lut3_mma(const GemvArgs &a, cudaStream_t stream)
{
    const int K = (int)a.K, N = (int)a.N, B = (int)a.B;
    const int W = (K + 1023) / 1024;                  // warps per row group (one 1024-weight slice each)
    if (W > 32) return cudaErrorInvalidValue;
    const int max_warps = (W > 20) ? 32 : 20;
    int G = max_warps / W;
    if (G < 1) G = 1;
    if (G > 15) G = 15;
    const int threads = G * W * 32;
    const uint32_t red_bytes = (uint32_t)G * kSlots * W * 32 * 16;
    const uint32_t x_addr = kRedAddr + ((red_bytes + 1023u) & ~1023u);
    const uint32_t col_stride = (uint32_t)W * 2048u + 32u;       // padded K in fp16, 32 mod 128 (see the layout note)
    int cols_max = (int)((kSmemLimit - 2048u - x_addr) / col_stride);
    if (cols_max > 8) cols_max = 8;
    if (cols_max < 1) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int ntiles = N / 16;
    int grid = (ntiles + G - 1) / G;
    if (grid > sms) grid = sms;
    for (int b0 = 0; b0 < B; b0 += cols_max) {
        const int cols = (B - b0 < cols_max) ? (B - b0) : cols_max;
        const uint32_t smem = x_addr + (uint32_t)cols * col_stride;
        cudaError_t e = (threads <= 512)   ? launch_one<512>(a, b0, cols, grid, threads, W, G, col_stride, x_addr, smem, stream)
                        : (threads <= 640) ? launch_one<640>(a, b0, cols, grid, threads, W, G, col_stride, x_addr, smem, stream)
                                           : launch_one<1024>(a, b0, cols, grid, threads, W, G, col_stride, x_addr, smem, stream);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace dq
