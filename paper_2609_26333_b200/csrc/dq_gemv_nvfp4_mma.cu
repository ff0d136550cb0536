// Weight-only decode on the NVFP4 view with the products on tensor cores (NVFP4A16, Sec. 2.3 / Table 1):
//   Y[b][n] = bf16( s * sum_k d_blk(n,k) * e2m1(code[n][k]) * X[b][k] )
// No lookups: a code byte (two weights) becomes an fp16 pair with one convert, is multiplied by its block
// scale in fp16 -- exact, a 3-bit significand times a 4-bit one -- and goes into mma.sync.m16n8k16 as an A
// fragment; activations are the B operand (up to eight batch columns per pass at no extra cost), products
// are exact and accumulate in fp32.  The tensor-core instruction also does the reduction along K that the
// CUDA-core kernels need shuffles for.
//
// Mapping.  A warp owns a 16-row tile and a 1024-weight slice of K, 128 weights (one 16-byte piece per lane
// and row) at a time.  Rows of a tile: four consecutive rows in each of the four 32-row quarters of a 128-row
// band, because the scale layout of the prefill GEMM keeps the scales of rows r, r+32, r+64, r+96 in one
// 16-byte group (so every fetched scale byte is used).  Lane (g, t) of the mma fragment layout holds rows
// g / g+8 of the tile and the 32 weights 32 t .. 32 t + 31 of the chunk; mma i of a chunk contracts, for every
// lane, its weights 4 i .. 4 i + 3 -- any assignment of weights to the sixteen k slots is fine as long as the
// B fragment uses the same one, and block scales are already folded into A.
// Activations: scaled by a power of two (exact) so that the largest magnitude of the pass lands in
// [2^14, 2^15), converted to fp16 and kept in shared memory; every element within 2^29 of the largest is
// exact.  One 8-byte shared-memory load per mma gives the B fragment.
// Partial sums of the K slices meet in shared memory; the warp that arrives last adds them in a fixed order.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_common.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

constexpr int kSlots = 4;                         // cross-warp reduction slots per row group
constexpr int kChunksPerSlice = 8;                // 128-weight chunks per 1024-weight slice
constexpr uint32_t kCtrlBytes = 1024;             // abort flag, reduction counters
constexpr uint32_t kRedBytes = 65536;             // [G][kSlots][W][32 lanes][4] floats
constexpr uint32_t kMaxXBytes = 128 * 1024;       // activation columns in fp16

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// four code bytes -> four fp16 pairs (low nibble first)
__device__ __forceinline__ void e2m1x8_to_f16(uint32_t w, uint32_t &p0, uint32_t &p1, uint32_t &p2, uint32_t &p3)
{
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\tmov.b32 {b0, b1, b2, b3}, %4;\n\t"
        "cvt.rn.f16x2.e2m1x2 %0, b0;\n\tcvt.rn.f16x2.e2m1x2 %1, b1;\n\t"
        "cvt.rn.f16x2.e2m1x2 %2, b2;\n\tcvt.rn.f16x2.e2m1x2 %3, b3;\n\t}"
        : "=r"(p0), "=r"(p1), "=r"(p2), "=r"(p3) : "r"(w));
}
__device__ __forceinline__ uint32_t hmul2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

struct ChunkRegs { uint4 c[2]; uint32_t sc[2]; };          // code pieces and scale byte pairs of rows g / g+8

template <int MAXT, int NPF>
__global__ void __launch_bounds__(MAXT, 1)
gemv_nvfp4_mma_kernel(const uint8_t *__restrict__ codes, const uint8_t *__restrict__ sf,
                      const PackedHeader *__restrict__ hdr, const __nv_bfloat16 *__restrict__ X, int64_t ldx, int b0,
                      int cols, __nv_bfloat16 *__restrict__ Y, int64_t ldy, int N, int K, int W, int G,
                      uint32_t col_stride, StatusWord *status)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const uint32_t win0 = (uint32_t)__cvta_generic_to_shared(smem_raw);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw);
    volatile int *sync_words = reinterpret_cast<volatile int *>(smem_raw + 64);          // [G][kSlots] x (generation, count)
    float *xmax_s = reinterpret_cast<float *>(smem_raw + 768);                          // 32 per-warp maxima
    float *red = reinterpret_cast<float *>(smem_raw + kCtrlBytes);                       // partial accumulators
    uint8_t *xh = smem_raw + kCtrlBytes + kRedBytes;                                     // fp16 activations [cols][col_stride]
    const uint32_t xh0 = win0 + kCtrlBytes + kRedBytes;

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int grp = warp / W;
    const int w = warp - grp * W;
    const int g = lane >> 2, t = lane & 3;
    const int katoms = K / 64;
    const int nchunks = K / 128;
    const size_t row_bytes = (size_t)K / 2;

    if (threadIdx.x < 16 * kSlots * 2) sync_words[threadIdx.x] = 0;
    if (threadIdx.x == 0) *abort_flag = 0;

    const int bands = (N + 127) / 128;
    const int ntiles = bands * 8;                           // 16-row tiles
    const int stride = gridDim.x * G;
    const int first = blockIdx.x * G + grp;

    // rows g and g+8 of tile (band, j): quarter (g >> 2) + 2 * half of the band, row 4 j + (g & 3) of the quarter
    auto tile_row = [&](int tile, int half) {
        const int band = tile >> 3, j = tile & 7;
        return band * 128 + ((g >> 2) + 2 * half) * 32 + 4 * j + (g & 3);
    };
    auto load_chunk = [&](ChunkRegs &R, int tile, int c) {
        const int band = tile >> 3, j = tile & 7;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int row = tile_row(tile, half);
            R.c[half] = (row < N) ? __ldg(reinterpret_cast<const uint4 *>(codes + (size_t)row * row_bytes + (size_t)c * 64 + t * 16))
                                  : make_uint4(0, 0, 0, 0);
            const uint8_t *sp = sf + ((size_t)band * katoms + (size_t)(2 * c + (t >> 1))) * 512 + (4 * j + (g & 3)) * 16 +
                                ((g >> 2) + 2 * half) * 4 + (t & 1) * 2;
            R.sc[half] = __ldg(reinterpret_cast<const unsigned short *>(sp));
        }
    };
    const int c_begin = w * kChunksPerSlice;
    const int c_end = min(c_begin + kChunksPerSlice, nchunks);

    // Register ring of NPF chunks in flight per lane.  Every tile takes eight ring positions (a short last
    // slice leaves some unused), so position p of the warp's stream is chunk c_begin + p % 8 of tile
    // first + (p / 8) * stride and lives in ring[p % NPF].
    // The weights are constant data: start streaming before waiting for the kernel ahead of this one.
    ChunkRegs ring[NPF];
#pragma unroll
    for (int p = 0; p < NPF; ++p) {
        ring[p].c[0] = ring[p].c[1] = make_uint4(0, 0, 0, 0);
        ring[p].sc[0] = ring[p].sc[1] = 0;
        const int tile2 = first + (p >> 3) * stride, c2 = c_begin + (p & 7);
        if (tile2 < ntiles && c2 < c_end) load_chunk(ring[p], tile2, c2);
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
        for (int i = threadIdx.x; i < K / 8; i += blockDim.x) {
            const uint4 v = __ldg(xp + i);
            const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
            uint32_t r[4];
#pragma unroll
            for (int z = 0; z < 4; ++z) {
                const __half2 h = __floats2half2_rn(__uint_as_float(ww[z] << 16) * xscale,
                                                    __uint_as_float(ww[z] & 0xFFFF0000u) * xscale);
                r[z] = *reinterpret_cast<const uint32_t *>(&h);
            }
            // inside a 128-weight chunk the four weights 32 t + 4 i .. + 3 sit at byte 32 i + 8 t, so that the
            // B-fragment reads of one mma (fixed i; lanes t, columns g 32 bytes apart mod 128) hit distinct banks
            const int k0 = i * 8;                                   // first of the 8 weights in v
            const int ch = k0 >> 7, tt = (k0 >> 5) & 3, ii = (k0 & 31) >> 2;
            uint8_t *dst = xh + (size_t)c * col_stride + (size_t)ch * 256 + ii * 32 + tt * 8;
            *reinterpret_cast<uint2 *>(dst) = make_uint2(r[0], r[1]);
            *reinterpret_cast<uint2 *>(dst + 32) = make_uint2(r[2], r[3]);
        }
    }
    __syncthreads();
    const float out_scale = hdr->s * xinv;
    // this lane's B fragments come from column g (any valid column for g >= cols: those outputs are not stored)
    const uint32_t xlane = xh0 + (uint32_t)((g < cols) ? g : 0) * col_stride + (uint32_t)t * 8;

    bool ok = true;
    int it = 0;
    for (int tile = first; tile < ntiles; tile += stride, ++it) {
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int k8 = 0; k8 < 8; ++k8) {
            const int c = c_begin + k8;
            const ChunkRegs cur = ring[k8 % NPF];
            {   // issue the loads of the chunk NPF positions ahead into this slot before working on the current one
                const int k2 = k8 + NPF;
                const int tile2 = tile + (k2 >> 3) * stride, c2 = c_begin + (k2 & 7);
                if (tile2 < ntiles && c2 < c_end) load_chunk(ring[k8 % NPF], tile2, c2);
            }
            if (c < c_end) {
            uint32_t dA[2], dB[2];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t d2;
                asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(d2) : "h"((unsigned short)cur.sc[half]));
                dA[half] = __byte_perm(d2, d2, 0x1010);      // scale of the lane's first block on both halves
                dB[half] = __byte_perm(d2, d2, 0x3232);      // second block
            }
            const uint32_t xa = xlane + (uint32_t)c * 256;
#pragma unroll
            for (int q = 0; q < 4; ++q) {                    // word q of the 16-byte pieces: mmas 2q and 2q + 1
                const uint32_t w0 = q == 0 ? cur.c[0].x : q == 1 ? cur.c[0].y : q == 2 ? cur.c[0].z : cur.c[0].w;
                const uint32_t w1 = q == 0 ? cur.c[1].x : q == 1 ? cur.c[1].y : q == 2 ? cur.c[1].z : cur.c[1].w;
                uint32_t p[4], r[4];
                e2m1x8_to_f16(w0, p[0], p[1], p[2], p[3]);
                e2m1x8_to_f16(w1, r[0], r[1], r[2], r[3]);
                const uint32_t s0 = (q < 2) ? dA[0] : dB[0], s1 = (q < 2) ? dA[1] : dB[1];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint2 xv = lds_v2(xa + (uint32_t)(2 * q + h) * 32);
                    mma16816(acc, hmul2(p[2 * h], s0), hmul2(r[2 * h], s1), hmul2(p[2 * h + 1], s0), hmul2(r[2 * h + 1], s1),
                             xv.x, xv.y);
                }
            }
            }
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
                const int row = tile_row(tile, j >> 1);
                if (ok && col < cols && row < N) Y[(int64_t)(b0 + col) * ldy + row] = __float2bfloat16_rn(tot[j] * out_scale);
            }
            __syncwarp();
            if (lane == 0) { *cnt = 0; __threadfence_block(); *gen = it / kSlots + 1; }
        }
    }
    if (*abort_flag && lane == 0) {
        atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
        atomicExch(&status->detail, 0x34000 | (int)blockIdx.x);
    }
}

template <int MAXT, int NPF>
cudaError_t launch_one(const GemvNvArgs &a, int b0, int cols, int grid, int threads, int W, int G, uint32_t col_stride,
                       uint32_t smem, cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemv_nvfp4_mma_kernel<MAXT, NPF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(kCtrlBytes + kRedBytes + kMaxXBytes));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
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
    return cudaLaunchKernelEx(&cfg, gemv_nvfp4_mma_kernel<MAXT, NPF>, a.codes, a.sf, a.hdr,
                              reinterpret_cast<const __nv_bfloat16 *>(a.X), (int64_t)a.ldx, b0, cols,
                              reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.N, (int)a.K, W, G, col_stride,
                              a.status);
}

}  // namespace

cudaError_t launch_gemv_nvfp4_mma(const GemvNvArgs &a, cudaStream_t stream)
{
    const int K = (int)a.K, N = (int)a.N, B = (int)a.B;
    const int W = (K + 1023) / 1024;                  // warps per row group (one 1024-weight slice each)
    if (W > 32) return cudaErrorInvalidValue;
    // measured: 20 warps with three chunks in flight per lane beat 16 warps with four (17408x5120: 15.0 vs 17.4 us);
    // 24 warps with two and any configuration that spills are slower
    const int max_warps = (W > 20) ? 32 : 20;
    int G = max_warps / W;
    if (G < 1) G = 1;
    if (G > 15) G = 15;
    const int threads = G * W * 32;
    if ((size_t)G * kSlots * W * 32 * 16 > kRedBytes) return cudaErrorInvalidValue;
    const uint32_t col_stride = (uint32_t)K * 2u + 32u;          // 32 mod 128: see the layout note in the kernel
    int cols_max = (int)(kMaxXBytes / col_stride);
    if (cols_max > 8) cols_max = 8;
    if (cols_max < 1) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int ntiles = ((N + 127) / 128) * 8;
    int grid = (ntiles + G - 1) / G;
    if (grid > sms) grid = sms;
    for (int b0 = 0; b0 < B; b0 += cols_max) {
        const int cols = (B - b0 < cols_max) ? (B - b0) : cols_max;
        const uint32_t smem = kCtrlBytes + kRedBytes + (uint32_t)cols * col_stride;
        cudaError_t e;
        if (threads <= 512) {
            e = launch_one<512, 4>(a, b0, cols, grid, threads, W, G, col_stride, smem, stream);
        } else if (threads <= 640) {
            e = launch_one<640, 3>(a, b0, cols, grid, threads, W, G, col_stride, smem, stream);
        } else {
            e = launch_one<1024, 2>(a, b0, cols, grid, threads, W, G, col_stride, smem, stream);
        }
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace dq
