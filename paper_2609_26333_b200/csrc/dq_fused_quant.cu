// Activation processing fused with the NVFP4 activation quantiser (App. C.1: the prefill stack fuses activation
// processing with the quantiser; the per-component latency table counts the quantiser inside "norms"):
//   RMSNorm          h = bf16( (x * r) * gamma ),  r = 1 / sqrt(mean(x^2) + eps)
//   SiLU(gate) * up  h = bf16( silu(g) * u )
// followed by the quantiser of App. A.3 "NVFP4" on h with the static input scale.  The normalised / gated
// activation never goes to HBM: one read of the bf16 input, 0.5625 byte per element written.
//
// The paper gives no arithmetic for the fused operators; the fp32 sequence below is fixed so that codes and scales
// can be compared bit for bit with a CPU evaluation of the same sequence:
//   sum of squares: x^2 summed in order inside each 16-element block, the block sums combined 32 blocks at a time by
//   a balanced binary tree (neighbours first: the warp butterfly), the group sums added in increasing order;
//   r by IEEE divide, add, square root, reciprocal;
//   exp(-g) = 2^t, t = -g log2(e): n = rint(t clamped to +-126), f = fma(g, -L_hi, -n), f = fma(g, -L_lo, f),
//   p = degree-7 Taylor polynomial of 2^f by fused multiply-adds, e = p * 2^n;  silu = g / (1 + e).
#include "dq_common.cuh"
#include "dq_quant.cuh"

namespace dq {

namespace {

constexpr int kNormMaxThreads = 256;        // one thread per 16-block where the row has that few
constexpr int kNormMaxGroups = 256;          // groups of 32 blocks per row: K <= 131072

// scale bytes of the four blocks of one 64-wide k atom (lanes 4q .. 4q+3) -> one 32-bit store
template <bool SWIZZLED>
__device__ __forceinline__ void store_scales(uint32_t d8, bool live, int r, int b, int nb, uint8_t *sf)
{
    uint32_t w = d8 << (8 * (threadIdx.x & 3));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    if (live && (threadIdx.x & 3) == 0) {
        if (SWIZZLED) {
            const int rr = r & 127;
            const size_t off = ((size_t)(r >> 7) * (size_t)(nb >> 2) + (size_t)(b >> 2)) * 512 + (size_t)((rr & 31) * 16 + (rr >> 5) * 4);
            *reinterpret_cast<uint32_t *>(sf + off) = w;
        } else {
            *reinterpret_cast<uint32_t *>(sf + (int64_t)r * nb + b) = w;
        }
    }
}

// One CTA per row.  Pass 1: sum of squares in the fixed order; pass 2: the row again (from L1 / L2), normalise,
// round to bf16, quantise.  Thread t owns blocks t, t + blockDim, ..: a warp's 32 blocks are consecutive, i.e. one group
// of the summation order, whatever the CTA size.
template <bool SWIZZLED>
__global__ void __launch_bounds__(kNormMaxThreads) rmsnorm_quant_kernel(const __nv_bfloat16 *__restrict__ X, int64_t ldx,
                                                                     const __nv_bfloat16 *__restrict__ gamma, float eps,
                                                                     int M, int K, float s, uint8_t *codes, uint8_t *sf)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ float gs[kNormMaxGroups];
    const int r = blockIdx.x;
    const int nb = K / 16;
    const int ngroups = (nb + 31) / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const __nv_bfloat16 *xr = X + (int64_t)r * ldx;
    for (int b0 = 0; b0 < nb; b0 += (int)blockDim.x) {           // all lanes of a warp walk together
        const int b = b0 + threadIdx.x;
        float bs = 0.0f;
        if (b < nb) {
            const uint4 *p = reinterpret_cast<const uint4 *>(xr + b * 16);
            const uint4 v0 = __ldg(p), v1 = __ldg(p + 1);
            const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float a = __uint_as_float(w[i] << 16), c = __uint_as_float(w[i] & 0xFFFF0000u);
                bs = __fadd_rn(bs, __fmul_rn(a, a));
                bs = __fadd_rn(bs, __fmul_rn(c, c));
            }
        }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) bs = __fadd_rn(bs, __shfl_xor_sync(0xffffffffu, bs, o));   // neighbours first
        if (lane == 0 && (b0 >> 5) + warp < ngroups) gs[(b0 >> 5) + warp] = bs;
    }
    __syncthreads();
    float total = 0.0f;
    for (int g = 0; g < ngroups; ++g) total = __fadd_rn(total, gs[g]);
    const float rr = __frcp_rn(__fsqrt_rn(__fadd_rn(__fdiv_rn(total, (float)K), eps)));
    const float rc6 = __frcp_rn(__fmul_rn(6.0f, s));
    for (int b0 = 0; b0 < nb; b0 += (int)blockDim.x) {
        const int b = b0 + threadIdx.x;
        const bool live = b < nb;
        uint32_t d8 = 0;
        if (live) {
            const uint4 *p = reinterpret_cast<const uint4 *>(xr + b * 16);
            const uint4 *q = reinterpret_cast<const uint4 *>(gamma + b * 16);
            const uint4 v0 = __ldg(p), v1 = __ldg(p + 1), g0 = __ldg(q), g1 = __ldg(q + 1);
            const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
            const uint32_t gw[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            uint32_t h[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float lo = __fmul_rn(__fmul_rn(__uint_as_float(w[i] << 16), rr), __uint_as_float(gw[i] << 16));
                const float hi = __fmul_rn(__fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), rr), __uint_as_float(gw[i] & 0xFFFF0000u));
                h[i] = pack_bf16_rn(lo, hi);
            }
            uint2 c;
            d8 = quant_block_nvfp4_bf16(h, s, rc6, c);
            *reinterpret_cast<uint2 *>(codes + ((int64_t)r * nb + b) * 8) = c;
        }
        store_scales<SWIZZLED>(d8, live, r, b, nb, sf);
    }
}

// The same operator with the row held in registers between the two phases (one read of X instead of two): thread t
// owns blocks t, t + blockDim, .. (BPT of them, 16 bytes of packed bf16 pairs each twice), a warp's 32 blocks are again one
// group of the summation order.  One CTA per row, as many threads as the row has blocks / BPT: several CTAs share an SM
// and cover each other's wait at the barrier.
template <bool SWIZZLED, int BPT>
__global__ void __launch_bounds__(1024) rmsnorm_quant_regs_kernel(const __nv_bfloat16 *__restrict__ X, int64_t ldx,
                                                                  const __nv_bfloat16 *__restrict__ gamma, float eps,
                                                                  int M, int K, float s, uint8_t *codes, uint8_t *sf)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ float gs[kNormMaxGroups];
    const int r = blockIdx.x;
    const int nb = K / 16;
    const int ngroups = (nb + 31) / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const __nv_bfloat16 *xr = X + (int64_t)r * ldx;
    uint32_t w[BPT][8];
#pragma unroll
    for (int j = 0; j < BPT; ++j) {
        const int b = j * (int)blockDim.x + threadIdx.x;
        float bs = 0.0f;
        if (b < nb) {
            const uint4 *p = reinterpret_cast<const uint4 *>(xr + b * 16);
            const uint4 v0 = __ldg(p), v1 = __ldg(p + 1);
            w[j][0] = v0.x; w[j][1] = v0.y; w[j][2] = v0.z; w[j][3] = v0.w;
            w[j][4] = v1.x; w[j][5] = v1.y; w[j][6] = v1.z; w[j][7] = v1.w;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float a = __uint_as_float(w[j][i] << 16), c = __uint_as_float(w[j][i] & 0xFFFF0000u);
                bs = __fadd_rn(bs, __fmul_rn(a, a));
                bs = __fadd_rn(bs, __fmul_rn(c, c));
            }
        }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) bs = __fadd_rn(bs, __shfl_xor_sync(0xffffffffu, bs, o));   // neighbours first
        const int grp = ((j * (int)blockDim.x) >> 5) + warp;
        if (lane == 0 && grp < ngroups) gs[grp] = bs;
    }
    __syncthreads();
    float total = 0.0f;
    for (int g = 0; g < ngroups; ++g) total = __fadd_rn(total, gs[g]);
    const float rr = __frcp_rn(__fsqrt_rn(__fadd_rn(__fdiv_rn(total, (float)K), eps)));
    const float rc6 = __frcp_rn(__fmul_rn(6.0f, s));
#pragma unroll
    for (int j = 0; j < BPT; ++j) {
        const int b = j * (int)blockDim.x + threadIdx.x;
        const bool live = b < nb;
        uint32_t d8 = 0;
        if (live) {
            const uint4 *q = reinterpret_cast<const uint4 *>(gamma + b * 16);
            const uint4 g0 = __ldg(q), g1 = __ldg(q + 1);
            const uint32_t gw[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            uint32_t h[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float lo = __fmul_rn(__fmul_rn(__uint_as_float(w[j][i] << 16), rr), __uint_as_float(gw[i] << 16));
                const float hi = __fmul_rn(__fmul_rn(__uint_as_float(w[j][i] & 0xFFFF0000u), rr), __uint_as_float(gw[i] & 0xFFFF0000u));
                h[i] = pack_bf16_rn(lo, hi);
            }
            uint2 c;
            d8 = quant_block_nvfp4_bf16(h, s, rc6, c);
            *reinterpret_cast<uint2 *>(codes + ((int64_t)r * nb + b) * 8) = c;
        }
        store_scales<SWIZZLED>(d8, live, r, b, nb, sf);
    }
}

// One thread per 16-block of the output; gate and up are the two halves of a row of the fused gate/up output.
template <bool SWIZZLED>
__global__ void __launch_bounds__(256) silu_mul_quant_kernel(const __nv_bfloat16 *__restrict__ GU, int64_t ldgu, int M, int nb,
                                                             float s, uint8_t *codes, uint8_t *sf)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int b = blockIdx.y * 64 + threadIdx.x;
    const int r = blockIdx.x * 4 + threadIdx.y;
    const bool live = (b < nb) && (r < M);
    const float rc6 = __frcp_rn(__fmul_rn(6.0f, s));
    uint32_t d8 = 0;
    if (live) {
        const uint4 *pg = reinterpret_cast<const uint4 *>(GU + (int64_t)r * ldgu + b * 16);
        const uint4 *pu = reinterpret_cast<const uint4 *>(GU + (int64_t)r * ldgu + (int64_t)nb * 16 + b * 16);
        const uint4 g0 = __ldg(pg), g1 = __ldg(pg + 1), u0 = __ldg(pu), u1 = __ldg(pu + 1);
        const uint32_t gw[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        const uint32_t uw[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
        uint32_t h[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) h[i] = silu_mul_bf16x2(gw[i], uw[i]);
        uint2 c;
        d8 = quant_block_nvfp4_bf16(h, s, rc6, c);
        *reinterpret_cast<uint2 *>(codes + ((int64_t)r * nb + b) * 8) = c;
    }
    store_scales<SWIZZLED>(d8, live, r, b, nb, sf);
}

// test hook: the SiLU the kernels above and the gated GEMM epilogue evaluate, value by value
__global__ void silu_probe_kernel(const __nv_bfloat16 *__restrict__ g, int64_t n, float *__restrict__ out)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float x = __bfloat162float(g[i]);
    out[i] = silu_f32(x);
}

template <typename Kern, typename... Args>
cudaError_t launch_pdl(Kern kern, dim3 grid, dim3 block, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace

cudaError_t launch_rmsnorm_quant(const void *X_bf16, int64_t M, int64_t K, int64_t ldx, const void *gamma_bf16, float eps,
                                 float act_scale, uint8_t *codes, uint8_t *sf, int swizzled, cudaStream_t stream)
{
    if (K / 16 > (int64_t)kNormMaxGroups * 32) return cudaErrorInvalidValue;
    const __nv_bfloat16 *X = reinterpret_cast<const __nv_bfloat16 *>(X_bf16);
    const __nv_bfloat16 *G = reinterpret_cast<const __nv_bfloat16 *>(gamma_bf16);
    const int64_t nb = K / 16;
    const dim3 grid((unsigned)M);
    if (nb <= 2048) {                                   // the row fits the registers of one CTA
        const int bpt = nb <= 1024 ? 1 : 2;
        const dim3 block((unsigned)(((nb + bpt - 1) / bpt + 31) / 32 * 32));
        if (bpt == 1) {
            if (swizzled) return launch_pdl(rmsnorm_quant_regs_kernel<true, 1>, grid, block, stream, X, ldx, G, eps, (int)M, (int)K, act_scale, codes, sf);
            return launch_pdl(rmsnorm_quant_regs_kernel<false, 1>, grid, block, stream, X, ldx, G, eps, (int)M, (int)K, act_scale, codes, sf);
        }
        if (swizzled) return launch_pdl(rmsnorm_quant_regs_kernel<true, 2>, grid, block, stream, X, ldx, G, eps, (int)M, (int)K, act_scale, codes, sf);
        return launch_pdl(rmsnorm_quant_regs_kernel<false, 2>, grid, block, stream, X, ldx, G, eps, (int)M, (int)K, act_scale, codes, sf);
    }
    const int threads = (int)(nb >= kNormMaxThreads ? kNormMaxThreads : (nb + 31) / 32 * 32);
    const dim3 block((unsigned)threads);
    if (swizzled) return launch_pdl(rmsnorm_quant_kernel<true>, grid, block, stream, X, ldx, G, eps, (int)M, (int)K, act_scale, codes, sf);
    return launch_pdl(rmsnorm_quant_kernel<false>, grid, block, stream, X, ldx, G, eps, (int)M, (int)K, act_scale, codes, sf);
}

cudaError_t launch_silu_probe(const void *g_bf16, int64_t n, float *out, cudaStream_t stream)
{
    silu_probe_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16 *>(g_bf16), n, out);
    return cudaGetLastError();
}

cudaError_t launch_silu_mul_quant(const void *GU_bf16, int64_t M, int64_t F, int64_t ldgu, float act_scale, uint8_t *codes,
                                  uint8_t *sf, int swizzled, cudaStream_t stream)
{
    const int nb = (int)(F / 16);
    const __nv_bfloat16 *GU = reinterpret_cast<const __nv_bfloat16 *>(GU_bf16);
    const dim3 grid((unsigned)((M + 3) / 4), (unsigned)((nb + 63) / 64)), block(64, 4);
    if (swizzled) return launch_pdl(silu_mul_quant_kernel<true>, grid, block, stream, GU, ldgu, (int)M, nb, act_scale, codes, sf);
    return launch_pdl(silu_mul_quant_kernel<false>, grid, block, stream, GU, ldgu, (int)M, nb, act_scale, codes, sf);
}

}  // namespace dq
