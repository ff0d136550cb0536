// Weight-only decode on the NVFP4 view (NVFP4A16, Sec. 2.3 / Table 1 "format-disaggregated NVFP4"):
//   Y[b][n] = bf16( s * sum_blk d_blk(n) * sum_{k in blk} e2m1(code[n][k]) * X[b][k] ),  fp32 accumulation,
// on the same 4.5-bit codes and scale atoms the prefill GEMM reads, so that one stored NVFP4 matrix
// serves both phases.  Memory-bound by intent (0.5625 byte per weight).
//
// Mapping.  K is cut into 1024-weight slices; warp w of a row group owns slice w and lane l the 32
// weights (16 code bytes, one 128-bit load) starting at 1024 w + 32 l, whose activations stay in
// registers as fp32 pairs.  A work unit is four rows r, r+32, r+64, r+96 of a 128-row band: the scale
// layout of the tensor-core GEMM stores the scales of exactly these four rows for one 64-weight atom in
// one 16-byte group, so one 128-bit load per lane brings the eight scale bytes it needs (and the four
// rows' code rows are whole 128-byte lines).  A code byte holds two weights; it is turned into the
// address of a 256-entry table of fp32 value pairs in shared memory (one byte-permute), looked up
// (ld.shared.u64, one 8-byte slot per lane: conflict free) and multiplied with the activation pair by one
// packed FMA.  No bit merging is needed, unlike LUT3.  Loads of the next unit are issued before the
// arithmetic of the current one.  Warp butterfly, then shared memory across the warps of the group.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_common.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

constexpr int kRows = 4;                                  // rows per work unit
constexpr int kSlots = 4;                                 // cross-warp reduction slots per row group
constexpr uint32_t kTableWindowAddr = 65536;              // table base in the CTA's shared window (64 KiB aligned)
constexpr uint32_t kTableBytes = 65536;                   // 256 entries x 32 lane slots x (fp32, fp32)
constexpr uint32_t kDynSmemBytes = 2 * 65536;             // [control + reduction | table]

// value pairs of all 256 code bytes, replicated per lane; filled whenever a handle with an NVFP4 view is made
__device__ __align__(256) unsigned char g_e2m1_pair_table[kTableBytes];

__global__ void fill_e2m1_table_kernel(unsigned char *table)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 256 * 32) return;
    const int e = i >> 5, l = i & 31;
    auto val = [](int c) {
        const float mag[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};      // App. A.3 "NVFP4"
        const float m = mag[c & 7];
        return (c & 8) ? -m : m;
    };
    *reinterpret_cast<float2 *>(table + e * 256 + l * 8) = make_float2(val(e & 15), val(e >> 4));
}

__device__ __forceinline__ unsigned long long lds_u64(uint32_t addr)
{
    unsigned long long v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void ffma2(unsigned long long &acc, unsigned long long a, unsigned long long b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b)
{
    unsigned long long r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// two E4M3 bytes (low 16 bits) -> two floats
__device__ __forceinline__ void e4m3x2_to_f32(uint32_t two, float &d0, float &d1)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)two));
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}"
        : "=f"(d0), "=f"(d1) : "r"(h2));
}

struct UnitRegs { uint4 c[kRows]; uint4 sc; };

template <int BT, int MAXT>
__global__ void __launch_bounds__(MAXT, 1)
gemv_nvfp4_kernel(const uint8_t *__restrict__ codes, const uint8_t *__restrict__ sf,
                  const uint8_t *__restrict__ table_img, const PackedHeader *__restrict__ hdr,
                  const __nv_bfloat16 *__restrict__ X, int64_t ldx, int b0, int B, __nv_bfloat16 *__restrict__ Y,
                  int64_t ldy, int N, int K, int W, int G, StatusWord *status)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const uint32_t win0 = (uint32_t)__cvta_generic_to_shared(smem_raw);
    float *red = reinterpret_cast<float *>(smem_raw);                         // [G][kSlots][rows][BT][W] partial sums
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + 32768);
    const uint32_t table_bar = win0 + 32768 + 64;
    volatile int *sync_words = reinterpret_cast<volatile int *>(smem_raw + 32768 + 128);   // [G][kSlots] x (generation, count)

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int grp = warp / W;
    const int w = warp - grp * W;
    const int pieces = K / 32;                               // 16-byte code pieces per row
    const int widx = w * 32 + lane;
    const bool active = widx < pieces;
    const int katoms = K / 64;

    if (win0 + 32768 + 128 + 16 * kSlots * 8 > kTableWindowAddr || (size_t)G * kSlots * kRows * BT * W * sizeof(float) > 32768) {
        if (threadIdx.x == 0) { atomicExch(&status->status, (int)DQ_ERR_INTERNAL); atomicExch(&status->detail, 0x32000); }
        return;
    }
    if (threadIdx.x < 16 * kSlots * 2) sync_words[threadIdx.x] = 0;
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        tc::mbar_init(table_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        tc::mbar_expect_tx(table_bar, kTableBytes);
        tc::bulk_load(kTableWindowAddr, table_img, kTableBytes, table_bar);
    }

    const int bands = (N + 127) / 128;
    const int nunits = bands * 32;
    const int stride = gridDim.x * G;
    const int first = blockIdx.x * G + grp;
    const size_t row_bytes = (size_t)K / 2;

    // loads of one unit: four code pieces (rows r32 + 32 i of the band) and the 16-byte scale group
    auto load_unit = [&](UnitRegs &R, int u) {
        const int band = u >> 5, r32 = u & 31;
#pragma unroll
        for (int i = 0; i < kRows; ++i) {
            const int row = band * 128 + r32 + 32 * i;
            R.c[i] = (active && row < N)
                         ? __ldg(reinterpret_cast<const uint4 *>(codes + (size_t)row * row_bytes + (size_t)widx * 16))
                         : make_uint4(0, 0, 0, 0);
        }
        R.sc = active ? __ldg(reinterpret_cast<const uint4 *>(sf + ((size_t)band * katoms + (widx >> 1)) * 512 + r32 * 16))
                      : make_uint4(0, 0, 0, 0);
    };
    // the weights are constant data: start streaming before waiting for the kernel ahead of this one
    UnitRegs cur;
    if (first < nunits) load_unit(cur, first);

    // Programmatic dependent launch: activations and output may belong to the previous kernel in the stream
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    unsigned long long xs[BT][16];
#pragma unroll
    for (int t = 0; t < BT; ++t) {
        const bool col_ok = active && (b0 + t < B);
        const uint4 *xp = reinterpret_cast<const uint4 *>(X + (int64_t)(col_ok ? b0 + t : 0) * ldx + (int64_t)(active ? widx : 0) * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint4 v = col_ok ? __ldg(xp + q) : make_uint4(0, 0, 0, 0);
            const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int z = 0; z < 4; ++z)
                xs[t][4 * q + z] = pack_f32x2(__uint_as_float(ww[z] << 16), __uint_as_float(ww[z] & 0xFFFF0000u));
        }
    }
    const float s_w = hdr->s;
    const uint32_t lane_base = kTableWindowAddr | (uint32_t)(lane * 8);
    bool ok = true;
    {
        uint32_t good = 1;
        if (lane == 0) good = tc::mbar_wait(table_bar, 0u, abort_flag) ? 1u : 0u;
        ok = __shfl_sync(0xffffffffu, good, 0) != 0;
    }

    int it = 0;
    for (int u = first; u < nunits; u += stride, ++it) {
        UnitRegs nxt;
        const int un = u + stride;
        if (un < nunits) load_unit(nxt, un);
        else { nxt = cur; }

        float v[kRows][BT];
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const uint32_t cw[4] = {cur.c[r].x, cur.c[r].y, cur.c[r].z, cur.c[r].w};
            const uint32_t scw = r == 0 ? cur.sc.x : r == 1 ? cur.sc.y : r == 2 ? cur.sc.z : cur.sc.w;
            float d0, d1;
            e4m3x2_to_f32((widx & 1) ? (scw >> 16) : (scw & 0xFFFFu), d0, d1);
            unsigned long long rowacc[BT];
#pragma unroll
            for (int t = 0; t < BT; ++t) rowacc[t] = 0ull;
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                unsigned long long g[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const uint32_t word = cw[2 * blk + (q >> 2)];
                    g[q] = lds_u64(__byte_perm(word, lane_base, 0x7604 | ((q & 3) << 4)));
                }
                const float d = blk ? d1 : d0;
                const unsigned long long dd = pack_f32x2(d, d);
#pragma unroll
                for (int t = 0; t < BT; ++t) {
                    unsigned long long acc = mul2(g[0], xs[t][8 * blk]);
#pragma unroll
                    for (int q = 1; q < 8; ++q) ffma2(acc, g[q], xs[t][8 * blk + q]);
                    ffma2(rowacc[t], acc, dd);                    // block scale on both halves
                }
            }
#pragma unroll
            for (int t = 0; t < BT; ++t) {
                float lo, hi;
                unpack_f32x2(rowacc[t], lo, hi);
                v[r][t] = lo + hi;
            }
        }
        // butterfly: afterwards lane l holds the warp total of row ((l>>4)&1)*2 + ((l>>3)&1)
#pragma unroll
        for (int t = 0; t < BT; ++t) {
#pragma unroll
            for (int st = 0; st < 2; ++st) {
                const int off = 16 >> st, cnt = 2 >> st;
                const bool upper = (lane & off) != 0;
#pragma unroll
                for (int i = 0; i < cnt; ++i) {
                    const float send = upper ? v[i][t] : v[i + cnt][t];
                    const float keep = upper ? v[i + cnt][t] : v[i][t];
                    v[i][t] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                }
            }
            v[0][t] += __shfl_xor_sync(0xffffffffu, v[0][t], 4);
            v[0][t] += __shfl_xor_sync(0xffffffffu, v[0][t], 2);
            v[0][t] += __shfl_xor_sync(0xffffffffu, v[0][t], 1);
        }
        // Cross-warp sum without a barrier: every warp of the group drops its partial sums into slot it % kSlots
        // and bumps the slot's counter; the warp that arrives last adds the W partials in a fixed order (so the
        // result does not depend on arrival order), stores the outputs and frees the slot for iteration it + kSlots.
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
        float *rbuf = red + ((grp * kSlots + slot) * kRows * BT) * W;
        if ((lane & 7) == 0) {
            const int row_l = ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
#pragma unroll
            for (int t = 0; t < BT; ++t) rbuf[(row_l * BT + t) * W + w] = v[0][t];
        }
        __syncwarp();
        int prev = 0;
        if (lane == 0) { __threadfence_block(); prev = atomicAdd(cnt, 1); }
        prev = __shfl_sync(0xffffffffu, prev, 0);
        if (prev == W - 1) {
            __threadfence_block();
            if (lane < kRows * BT) {
                const int row_l = lane / BT, t = lane % BT;
                float tot = 0.0f;
                for (int ww = 0; ww < W; ++ww) tot += reinterpret_cast<volatile float *>(rbuf)[(row_l * BT + t) * W + ww];
                const int row = (u >> 5) * 128 + (u & 31) + 32 * row_l;
                if (ok && b0 + t < B && row < N) Y[(int64_t)(b0 + t) * ldy + row] = __float2bfloat16_rn(tot * s_w);
            }
            __syncwarp();
            if (lane == 0) { *cnt = 0; __threadfence_block(); *gen = it / kSlots + 1; }
        }
        cur = nxt;
    }
    if (*abort_flag) {
        if (lane == 0) atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
        if (lane == 0) atomicExch(&status->detail, 0x33000 | (int)blockIdx.x);
    }
}

template <int BT, int MAXT>
cudaError_t launch_one(const GemvNvArgs &a, const uint8_t *table, int b0, int grid, int threads, int W, int G,
                       cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    int attr_dev = 0;
    if (cudaGetDevice(&attr_dev) != cudaSuccess || attr_dev < 0 || attr_dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[attr_dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemv_nvfp4_kernel<BT, MAXT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kDynSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[attr_dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = kDynSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_nvfp4_kernel<BT, MAXT>, a.codes, a.sf, table, a.hdr,
                              reinterpret_cast<const __nv_bfloat16 *>(a.X), (int64_t)a.ldx, b0, (int)a.B,
                              reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.N, (int)a.K, W, G, a.status);
}

}  // namespace

cudaError_t launch_fill_e2m1_table(cudaStream_t stream)
{
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_e2m1_pair_table);
    if (e != cudaSuccess) return e;
    fill_e2m1_table_kernel<<<32, 256, 0, stream>>>(reinterpret_cast<unsigned char *>(p));
    return cudaGetLastError();
}

cudaError_t launch_gemv_nvfp4(const GemvNvArgs &a, cudaStream_t stream)
{
    const int K = (int)a.K, N = (int)a.N, B = (int)a.B;
    const int W = (K + 1023) / 1024;
    if (W > 32) return cudaErrorInvalidValue;
    int G = 16 / W;                                   // row groups per CTA: up to 512 threads when K allows
    if (G < 1) G = 1;
    if (G > 15) G = 15;                               // one named barrier per group
    const int threads = G * W * 32;
    void *table = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&table, g_e2m1_pair_table);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int nunits = ((N + 127) / 128) * 32;
    int grid = (nunits + G - 1) / G;
    if (grid > sms) grid = sms;
    for (int b0 = 0; b0 < B; b0 += 2) {
        const uint8_t *tb = reinterpret_cast<const uint8_t *>(table);
        const bool two = B - b0 >= 2;
        if (threads <= 512) e = two ? launch_one<2, 512>(a, tb, b0, grid, threads, W, G, stream) : launch_one<1, 512>(a, tb, b0, grid, threads, W, G, stream);
        else if (threads <= 576) e = two ? launch_one<2, 576>(a, tb, b0, grid, threads, W, G, stream) : launch_one<1, 576>(a, tb, b0, grid, threads, W, G, stream);
        else e = two ? launch_one<2, 1024>(a, tb, b0, grid, threads, W, G, stream) : launch_one<1, 1024>(a, tb, b0, grid, threads, W, G, stream);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace dq
