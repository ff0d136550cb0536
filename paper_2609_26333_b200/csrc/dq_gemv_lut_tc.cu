// LUT3 / LUT2 weight-only mat-vec (batch 1) on the 5th-generation tensor cores (App. C.2 "Kernel specification"):
//   y[n] = bf16( s * sum_blk d_blk(n) * sum_{k in blk} G[idx(n,k)] * x[k] ).
//
// Same arithmetic as the mma.sync kernel (dq_gemv_lut.cu): fp16 codebook levels unscaled, activations scaled by one
// power of two into fp16, every product exact, one 16-weight block per contraction, the signed E4M3 block scale applied
// to the block's fp32 sum in fp32.  What changes is who does the contraction.  There a lane pays, per 8 weights, one
// HMMA, four FFMA and its share of the B-fragment loads on top of the lookups; here the dequantising warps only look
// levels up and store them to tensor memory, tcgen05.mma contracts them from there, and a thread meets its row again
// as eight block sums per 128 weights.
//
// Roles.  A CTA (one per SM) works on a tile of 128 rows: 2 or 3 warpgroups of 4 dequantising warps split K between
// them, one more warp per warpgroup issues its MMAs.  Warp q of a warpgroup owns rows 32q .. 32q+31 of the tile, which are the
// tensor-memory lanes it may access, i.e. four atoms (8 rows x 512 weights) of the device layout per 512-weight stage;
// it streams them through its own ring of bulk copies, as in the mma.sync kernel.
//
// A operand.  Lane (g, t) of the device layout holds weights 4t .. 4t+3 of every block of row g: exactly the
// registers tcgen05.st.16x256b wants from it for lane g (and g + 8 from the atom of the other row half), so one
// store of 32 registers puts eight blocks (K = 128) of 16 rows into 64 columns of tensor memory, two stores a warp's
// 32 rows.
//
// B operand.  tcgen05.mma needs N >= 16 and one MMA contracts K = 16, one block.  Eight MMAs (the eight blocks of a
// step) accumulate into one 128 x 16 accumulator, block j into column j (j < 4) or 8 + (j - 4): the B tile of block j
// is zero except for its row j, which holds the block's 16 activations.  Shared memory keeps every 8-activation half
// row in a 64-byte slot (16 bytes of data, 48 of zeros); a descriptor that starts 16 j bytes before the block's
// first half then sees the data in row j and zeros in the other rows below 4, whatever follows in rows 4-7 only
// reaches accumulator columns nobody reads, and the second 8-row group is pointed at a zero region (blocks 0-3) or
// the first at one (blocks 4-7).  That is 8 bytes of shared memory per activation, which is what limits K here;
// longer rows and batches above 1 take the mma.sync kernel.
//
// Pipeline per warpgroup and step (K = 128): dequantise -> tcgen05.st -> arrive on a_full[buf]; the warpgroup's MMA
// warp waits for the four warps, issues 8 MMAs, commits to d_full[buf]; the dequantising warps read the accumulator of
// the step two back (tcgen05.ld, 8 FFMA with the row's block scales) around the stores of the current one.  Two A
// buffers and two accumulators per warpgroup (160 of the 512 tensor-memory columns).  Every wait is bounded.
//
// Status: exact (outputs equal the mma.sync kernel's up to the order of the fp32 sums) but slower, and therefore only
// reachable through the test hook.  Measured on 17408 x 5120 (LUT3, launches back to back): 23.7 us against 16.3 us.
// One MMA of 128 x 16 x 16 from tensor memory takes 45 cycles whatever N is (the A operand is what it reads), so the
// 24 MMAs of a round of three warpgroups keep the tensor pipe busy for 1080 cycles, as long as the three dequantising
// warps of a scheduler need to issue their permutes; with two buffers per warpgroup a step cannot start before the
// MMAs two steps back have finished, the two costs add up instead of overlapping (1850 cycles per step measured, 840
// with the dequantisation left out), more buffers do not fit tensor memory beside three warpgroups, and set-up
// (tensor-memory allocation, 8 bytes of shared memory per activation to fill) costs about 3 us more than the
// mma.sync kernel's.  Kept as the measured answer to whether tcgen05 helps this contraction on this GPU.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_common.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

constexpr int kMaxWgs = 3;
constexpr int kTcMaxThreads = (4 * kMaxWgs + kMaxWgs) * 32;
constexpr uint32_t kTcSmemLimit = 227 * 1024;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kWgCols = 160;          // per warpgroup: A0 at +0, A1 at +64, D0 at +128, D1 at +144
constexpr int kRing = 2;                   // ring stages per warp; a stage = this warp's 32 rows x 512 weights = 4 atoms
constexpr uint32_t kZeroPad = 256;         // zero regions below and above the activations

struct TcPlan {
    int wgs;                     // dequantising warpgroups per CTA
    uint32_t bar_off;            // a_full[wg][2] | d_full[wg][2] | ring[warp][kRing] | fin
    uint32_t red_off;            // [2][wgs][128] floats
    uint32_t ring_off;           // [warp][kRing][4 atoms]
    uint32_t x_off;              // zero | activations (128 bytes per 16-block) | zero
    uint32_t x_bytes;
    long long wait_cycles;
    int drop_first_copy;
};

// mbarrier wait that lets the hardware park the thread (up to the hint, in ns) instead of spinning on issue slots
__device__ __forceinline__ bool mbar_try_park(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, long long budget)
{
    if (mbar_try_park(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_park(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > budget) { *abort_flag = 1; return false; }
    }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
template <int OFF>
__device__ __forceinline__ uint4 lds_v4_at(uint32_t base)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+%5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(base), "n"(OFF) : "memory");
    return v;
}
// four signed E4M3 bytes -> four floats (exact)
__device__ __forceinline__ float4 e4m3x4_to_f32(uint32_t four)
{
    uint32_t h01, h23;
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, lo;\n\tcvt.rn.f16x2.e4m3x2 %1, hi;\n\t}"
        : "=r"(h01), "=r"(h23) : "r"(four));
    float4 r;
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}" : "=f"(r.x), "=f"(r.y) : "r"(h01));
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}" : "=f"(r.z), "=f"(r.w) : "r"(h23));
    return r;
}

struct Codebook { uint32_t tl0, tl1, th0, th1; };    // low bytes of levels 0-3 / 4-7, high bytes of levels 0-3 / 4-7

// The eight blocks of one word group of two atoms (rows g and g + 8 of a 16-row tile) as the 32 registers of one
// tcgen05.st.16x256b.x8: block i takes registers 4i .. 4i+3 = (row g: weights 4t, 4t+1 | 4t+2, 4t+3), (row g + 8: same).
template <int BITS>
__device__ __forceinline__ void dequant_group(const uint32_t (&w0)[BITS], const uint32_t (&w1)[BITS], const Codebook &cb,
                                              uint32_t (&r)[32])
{
    uint32_t s0[4], s1[4];
    lut_selectors<BITS>(w0, s0);
    lut_selectors<BITS>(w1, s1);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = 2 * a + h;
            const uint32_t u0 = h ? (s0[a] >> 16) : s0[a], u1 = h ? (s1[a] >> 16) : s1[a];
            const uint32_t lo0 = prmt(cb.tl0, cb.tl1, u0), hi0 = prmt(cb.th0, cb.th1, u0);
            r[4 * i + 0] = prmt(lo0, hi0, 0x5140u);
            r[4 * i + 1] = prmt(lo0, hi0, 0x7362u);
            const uint32_t lo1 = prmt(cb.tl0, cb.tl1, u1), hi1 = prmt(cb.th0, cb.th1, u1);
            r[4 * i + 2] = prmt(lo1, hi1, 0x5140u);
            r[4 * i + 3] = prmt(lo1, hi1, 0x7362u);
        }
    }
}

__device__ __forceinline__ void tmem_st_16x256b_x8(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.16x256b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
          "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
          "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32b_x4(uint32_t taddr, float (&v)[4])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]) : "r"(taddr) : "memory");
}
// K-major, unswizzled operand: 8-row groups of 16-byte rows; `kstep` bytes between the two 8-element halves of K,
// `nstep` bytes between the two 8-row groups of N
__device__ __forceinline__ uint64_t make_desc_plain(uint32_t saddr, uint32_t kstep, uint32_t nstep)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)((kstep >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((nstep >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// D (tensor memory, fp32) (+)= A (tensor memory, fp16, 128 x 16) * B (shared memory, fp16, 16 x 16)
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// instruction descriptor, kind::f16: fp32 accumulator, fp16 A and B, both K-major, N = 16, M = 128
constexpr uint32_t kIdesc = (1u << 4) | ((16u >> 3) << 17) | ((128u >> 4) << 24);

template <int BITS>
__global__ void __launch_bounds__(kTcMaxThreads, 1)
gemv_lut_tc_kernel(const uint8_t *__restrict__ lut, const PackedHeader *__restrict__ hdr, const __nv_bfloat16 *__restrict__ X,
                   __nv_bfloat16 *__restrict__ Y, int N, int K, TcPlan L, StatusWord *status)
{
    constexpr uint32_t kAtom = (uint32_t)lut_atom_bytes(BITS);
    constexpr uint32_t kPlanes = (uint32_t)lut_plane_bytes(BITS);
    constexpr uint32_t kStage = 4u * kAtom;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t win0 = (uint32_t)__cvta_generic_to_shared(smem_raw);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw);
    volatile uint32_t *tmem_base_s = reinterpret_cast<volatile uint32_t *>(smem_raw + 8);
    float *xmax_s = reinterpret_cast<float *>(smem_raw + 64);                      // one per warp

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wgs = L.wgs, ndq = 4 * wgs;                // dequantising warps; warp ndq + g issues the MMAs of warpgroup g
    const int nwarps = ndq + wgs;
    const bool is_dq = warp < ndq;
    const int wg = warp >> 2, q = warp & 3;
    const int nslices = (int)lut_slices(K);
    const int kpad = nslices * kLutSlice;
    const int nst = 2 * nslices;                         // 512-weight stages along K
    const int ntiles = (N + 127) >> 7;
    const int ntile16 = N >> 4;
    const long long budget = L.wait_cycles;

    auto a_full = [&](int g_, int b) { return win0 + L.bar_off + (uint32_t)(g_ * 2 + b) * 8u; };
    auto d_full = [&](int g_, int b) { return win0 + L.bar_off + 64u + (uint32_t)(g_ * 2 + b) * 8u; };
    const uint32_t ring_bars = win0 + L.bar_off + 128u + (uint32_t)warp * (kRing * 8u);
    const uint32_t fin_bar = win0 + L.bar_off + 128u + (uint32_t)(4 * kMaxWgs) * (kRing * 8u);
    const uint32_t ring0 = win0 + L.ring_off + (uint32_t)warp * (kRing * kStage);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int g_ = 0; g_ < wgs; ++g_)
            for (int b = 0; b < 2; ++b) { tc::mbar_init(a_full(g_, b), 4); tc::mbar_init(d_full(g_, b), 1); }
        for (int g_ = 0; g_ < wgs; ++g_) tc::mbar_init(fin_bar + 8u * g_, 1);
    }
    if (is_dq && lane == 0)
        for (int i = 0; i < kRing; ++i) tc::mbar_init(ring_bars + 8u * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == ndq) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(win0 + 8u), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    // this warpgroup's share of K, in stages
    const int st0 = is_dq ? (wg * nst) / wgs : 0, st1 = is_dq ? ((wg + 1) * nst) / wgs : 0;
    // producer state (lane 0 of a dequantising warp): next (tile, stage) to request
    int ptile = blockIdx.x, pst = st0, pslot = 0;
    auto issue_next = [&](bool drop) {
        const uint32_t bar = ring_bars + 8u * pslot;
        const int t16 = 8 * ptile + 2 * q;
        const int natoms = (t16 + 1 < ntile16) ? 4 : ((t16 < ntile16) ? 2 : 0);
        if (!drop) {
            if (natoms == 0) tc::mbar_arrive(bar);
            else tc::mbar_expect_tx(bar, (uint32_t)natoms * kAtom);
            for (int j = 0; j < natoms; ++j) {
                const size_t atom = (((size_t)(t16 + (j >> 1)) * nslices + (pst >> 1)) * 2 + (j & 1)) * 2 + (pst & 1);
                tc::bulk_load(ring0 + (uint32_t)pslot * kStage + (uint32_t)j * kAtom, lut + atom * kAtom, kAtom, bar);
            }
        }
        if (++pst == st1) { pst = st0; ptile += gridDim.x; }
        pslot ^= 1;
    };
    // The weights are constant data: start streaming before waiting for the kernel ahead of this one.
    if (is_dq && lane == 0 && st1 > st0) {
        const bool drop = L.drop_first_copy && blockIdx.x == 0 && warp == 0;
        for (int i = 0; i < kRing && ptile < ntiles; ++i) issue_next(drop && i == 0);
    }
    const uint4 cbv = *reinterpret_cast<const uint4 *>(BITS == 3 ? hdr->lut_prmt : hdr->lut2_prmt);
    const Codebook cb = {cbv.x, cbv.y, cbv.z, cbv.w};
    const float s_w = hdr->s;

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- activations: raw bf16 parked at their slots (with the zeros around them) while the largest magnitude is
    //      found, then power-of-two scale -> fp16 in place
    uint8_t *xz = smem_raw + L.x_off;                       // zero region below
    uint8_t *xb = xz + kZeroPad;
    const int nthreads = nwarps * 32;
    if (threadIdx.x < (int)(kZeroPad / 16)) {
        *reinterpret_cast<uint4 *>(xz + threadIdx.x * 16) = make_uint4(0u, 0u, 0u, 0u);
        *reinterpret_cast<uint4 *>(xb + L.x_bytes + threadIdx.x * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    float m = 0.0f;
    {
        const uint4 *xp = reinterpret_cast<const uint4 *>(X);
        for (int i = threadIdx.x; i < kpad / 8; i += nthreads) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);             // the padding of a short last slice reads as zero
            if (i < K / 8) v = __ldg(xp + i);
            const uint32_t a0 = v.x & 0x7FFF7FFFu, a1 = v.y & 0x7FFF7FFFu, a2 = v.z & 0x7FFF7FFFu, a3 = v.w & 0x7FFF7FFFu;
            const uint32_t hi = max(max(a0 >> 16, a1 >> 16), max(a2 >> 16, a3 >> 16));
            const uint32_t lo = max(max(a0 & 0xFFFFu, a1 & 0xFFFFu), max(a2 & 0xFFFFu, a3 & 0xFFFFu));
            m = fmaxf(m, __uint_as_float(max(hi, lo) << 16));
            uint4 *dst = reinterpret_cast<uint4 *>(xb + (size_t)i * 64);
            dst[0] = v;
            dst[1] = make_uint4(0u, 0u, 0u, 0u);
            dst[2] = make_uint4(0u, 0u, 0u, 0u);
            dst[3] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) xmax_s[warp] = m;
    __syncthreads();
    m = (lane < nwarps) ? xmax_s[lane] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    int ex = (int)((__float_as_uint(m) >> 23) & 0xFFu) - 127;           // floor(log2(max)); -127 for zero / subnormal
    ex = max(-100, min(100, ex));
    const float xscale = __uint_as_float((uint32_t)(127 + 14 - ex) << 23);   // 2^(14 - ex)
    const float out_scale = s_w * __uint_as_float((uint32_t)(127 - 14 + ex) << 23);
    for (int i = threadIdx.x; i < kpad / 8; i += nthreads) {              // every thread converts what it parked itself
        uint4 *px = reinterpret_cast<uint4 *>(xb + (size_t)i * 64);
        const uint4 v = *px;
        const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
        uint32_t r[4];
#pragma unroll
        for (int z = 0; z < 4; ++z) {
            const __half2 h = __floats2half2_rn(__uint_as_float(ww[z] << 16) * xscale, __uint_as_float(ww[z] & 0xFFFF0000u) * xscale);
            r[z] = *reinterpret_cast<const uint32_t *>(&h);
        }
        *px = make_uint4(r[0], r[1], r[2], r[3]);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");        // the tensor cores read the activations
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_base_s;

    if (is_dq) {
        // ================= dequantising warps =================
        const uint32_t wg_cols = tmem + (uint32_t)wg * kWgCols;
        const uint32_t lane_lo = ((uint32_t)(32 * q) << 16), lane_hi = ((uint32_t)(32 * q + 16) << 16);
        const uint32_t lane_plane = (uint32_t)lane * 16u;
        const uint32_t scale_at = (uint32_t)(lane >> 3) * kAtom + kPlanes + (uint32_t)(lane & 7) * 32u;   // this thread's row
        float *red = reinterpret_cast<float *>(smem_raw + L.red_off);
        bool ok = true;
        int slot = 0;
        uint32_t ring_phase = 0;
        uint32_t step = 0;                                   // MMA steps of this warpgroup so far
        int tpar = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, tpar ^= 1) {
            float acc = 0.0f;
            // Steps whose accumulator has not been read yet: at most two.  The accumulator of step s - 2 is fetched at
            // the start of step s (its MMAs finished long ago; the wait also says that A buffer s % 2 is free again) and
            // folded in after the stores of step s are issued, so that neither tcgen05.ld nor tcgen05.st is waited for
            // with nothing else to do; MMAs of step s - 1 have all of step s to finish.
            uint32_t qa0 = 0u, qa1 = 0u, qb0 = 0u, qb1 = 0u;      // scale bytes of the queued steps, by step parity
            int npend = 0;
            float d0[4], d1[4];
            auto fetch = [&](uint32_t ps) {                   // start reading the accumulator of step ps
                if (ok) ok = wait_bar(d_full(wg, (int)(ps & 1u)), (ps >> 1) & 1u, abort_flag, budget);
                if (ok) {
                    tc::tc_fence_after();
                    const uint32_t dcol = wg_cols + 128u + (ps & 1u) * 16u + lane_lo;
                    tmem_ld_32x32b_x4(dcol, d0);
                    tmem_ld_32x32b_x4(dcol + 8u, d1);
                }
            };
            auto fold = [&](uint32_t ps) {                    // eight block sums of this thread's row times their block scales
                if (ok) {
                    tc::tmem_ld_wait();
                    const float4 fa = e4m3x4_to_f32((ps & 1u) ? qa1 : qa0), fb = e4m3x4_to_f32((ps & 1u) ? qb1 : qb0);
                    acc = fmaf(d0[0], fa.x, acc);
                    acc = fmaf(d0[1], fa.y, acc);
                    acc = fmaf(d0[2], fa.z, acc);
                    acc = fmaf(d0[3], fa.w, acc);
                    acc = fmaf(d1[0], fb.x, acc);
                    acc = fmaf(d1[1], fb.y, acc);
                    acc = fmaf(d1[2], fb.z, acc);
                    acc = fmaf(d1[3], fb.w, acc);
                }
            };
            for (int st = st0; st < st1; ++st) {
                if (ok) ok = wait_bar(ring_bars + 8u * slot, ring_phase, abort_flag, budget);
                uint4 pw[4][BITS];
                uint4 sc0 = make_uint4(0u, 0u, 0u, 0u), sc1 = sc0;
                if (ok) {
                    const uint32_t base = ring0 + (uint32_t)slot * kStage;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        pw[j][0] = lds_v4_at<0>(base + (uint32_t)j * kAtom + lane_plane);
                        pw[j][1] = lds_v4_at<512>(base + (uint32_t)j * kAtom + lane_plane);
                        if (BITS == 3) pw[j][BITS - 1] = lds_v4_at<1024>(base + (uint32_t)j * kAtom + lane_plane);
                    }
                    sc0 = lds_v4_at<0>(base + scale_at);
                    sc1 = lds_v4_at<16>(base + scale_at);
                }
                // the stage is in registers: refill it with the stage kRing steps ahead
                __syncwarp();
                if (lane == 0 && ptile < ntiles) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    issue_next(false);
                }
                const uint32_t scw[8] = {sc0.x, sc0.y, sc0.z, sc0.w, sc1.x, sc1.y, sc1.z, sc1.w};
#pragma unroll
                for (int wi = 0; wi < 4; ++wi) {
                    const uint32_t buf = step & 1u;
                    const bool two = npend == 2;
                    if (two) fetch(step - 2u);
                    if (ok) {
                        uint32_t w0[BITS], w1[BITS], r[32];
                        const uint32_t acol = wg_cols + buf * 64u;
#pragma unroll
                        for (int p = 0; p < BITS; ++p) {
                            w0[p] = wi == 0 ? pw[0][p].x : wi == 1 ? pw[0][p].y : wi == 2 ? pw[0][p].z : pw[0][p].w;
                            w1[p] = wi == 0 ? pw[1][p].x : wi == 1 ? pw[1][p].y : wi == 2 ? pw[1][p].z : pw[1][p].w;
                        }
                        dequant_group<BITS>(w0, w1, cb, r);
                        tmem_st_16x256b_x8(acol + lane_lo, r);
#pragma unroll
                        for (int p = 0; p < BITS; ++p) {
                            w0[p] = wi == 0 ? pw[2][p].x : wi == 1 ? pw[2][p].y : wi == 2 ? pw[2][p].z : pw[2][p].w;
                            w1[p] = wi == 0 ? pw[3][p].x : wi == 1 ? pw[3][p].y : wi == 2 ? pw[3][p].z : pw[3][p].w;
                        }
                        dequant_group<BITS>(w0, w1, cb, r);
                        tmem_st_16x256b_x8(acol + lane_hi, r);
                    }
                    if (two) { fold(step - 2u); --npend; }
                    if (buf) { qa1 = scw[2 * wi]; qb1 = scw[2 * wi + 1]; } else { qa0 = scw[2 * wi]; qb0 = scw[2 * wi + 1]; }
                    ++npend;
                    if (ok) {
                        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                        tc::tc_fence_before();
                    }
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(a_full(wg, (int)buf));   // also after a wait ran out: the MMA warp gives up by itself
                    ++step;
                    }
                if (++slot == kRing) { slot = 0; ring_phase ^= 1u; }
            }
            for (; npend > 0; --npend) { fetch(step - (uint32_t)npend); fold(step - (uint32_t)npend); }
            // ---- the warpgroups' partial sums of the tile, added in order by the first one
            red[(tpar * wgs + wg) * 128 + 32 * q + lane] = acc;
            asm volatile("bar.sync 1, %0;" ::"r"(ndq * 32) : "memory");
            if (wg == 0) {
                float tot = 0.0f;
                for (int g_ = 0; g_ < wgs; ++g_) tot += red[(tpar * wgs + g_) * 128 + 32 * q + lane];
                const int row = tile * 128 + 32 * q + lane;
                if (ok && !*abort_flag && row < N) Y[row] = __float2bfloat16_rn(tot * out_scale);
            }
        }
    } else if (lane == 0) {
        // ================= MMA issue: one warp per warpgroup =================
        const int g_ = warp - ndq;
        const uint32_t xaddr = win0 + L.x_off + kZeroPad, zlo = win0 + L.x_off, zhi = xaddr + L.x_bytes;
        const int s0 = (g_ * nst) / wgs, s1 = ((g_ + 1) * nst) / wgs;
        const int nsteps = 4 * (s1 - s0);
        // descriptors of the eight blocks of the K range's first step; a step further on every one moves by eight blocks
        // (1024 bytes): the start address for blocks 0-3, the offset of the second 8-row group for blocks 4-7
        uint64_t desc0[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t row0 = xaddr + ((uint32_t)(s0 * 32) + (uint32_t)j) * 128u - 16u * (uint32_t)(j & 3);   // data in row j % 4
            desc0[j] = j < 4 ? make_desc_plain(row0, 64u, zhi - row0) : make_desc_plain(zlo, 64u, row0 - zlo);
        }
        const uint64_t step_lo = 64ull - (64ull << 32), step_hi = 64ull << 32;     // in 16-byte units: 1024 bytes
        uint32_t sdone = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
            for (int i = 0; i < nsteps; ++i) {
                const uint32_t buf = sdone & 1u;
                ok = wait_bar(a_full(g_, (int)buf), (sdone >> 1) & 1u, abort_flag, budget);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t acol = tmem + (uint32_t)g_ * kWgCols + buf * 64u;
                const uint32_t dcol = tmem + (uint32_t)g_ * kWgCols + 128u + buf * 16u;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    mma_f16_ts(dcol, acol + 8u * (uint32_t)j, desc0[j] + (uint64_t)i * (j < 4 ? step_lo : step_hi), kIdesc, j == 0 ? 0u : 1u);
                tc::mma_commit(d_full(g_, (int)buf));
                ++sdone;
            }
        }
        // nothing this thread issued may still be in flight when tensor memory is handed back
        tc::mma_commit(fin_bar + 8u * g_);
        wait_bar(fin_bar + 8u * g_, 0u, abort_flag, budget);
    }
    // ---- common exit: nothing of this CTA may still be in flight when tensor memory is handed back
    tc::tc_fence_before();
    __syncthreads();
    if (warp == ndq) {
        tc::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (*abort_flag) {
        // a wait ran out: let copies in flight land before the CTA's shared memory is handed on, then report
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        if (threadIdx.x == 0) {
            atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
            atomicExch(&status->detail, 0x37000 | (int)blockIdx.x);
        }
    }
}

// shared-memory map; returns the bytes needed
uint32_t tc_plan(int bits, int K, int wgs, TcPlan &L)
{
    const uint32_t stage = 4u * (uint32_t)lut_atom_bytes(bits);
    L.wgs = wgs;
    L.bar_off = 128;
    L.red_off = 1024;
    L.ring_off = 1024 + 2u * (uint32_t)kMaxWgs * 128u * 4u;
    L.x_off = L.ring_off + (uint32_t)(4 * wgs) * kRing * stage;
    L.x_bytes = (uint32_t)lut_slices(K) * (kLutSlice / 16) * 128u;
    return L.x_off + kZeroPad + L.x_bytes + kZeroPad;
}

template <int BITS>
cudaError_t launch_tc(const GemvArgs &a, const TcPlan &L, uint32_t smem, int grid, cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemv_lut_tc_kernel<BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(gemv_lut_tc_kernel<BITS>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)(5 * L.wgs * 32));
    // all of the SM's shared memory: the kernel allocates all of tensor memory, so a second CTA (of this or the next
    // launch) on the same SM would only wait for it
    cfg.dynamicSmemBytes = smem < kTcSmemLimit ? kTcSmemLimit : smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_lut_tc_kernel<BITS>, a.lut, a.hdr, reinterpret_cast<const __nv_bfloat16 *>(a.X),
                              reinterpret_cast<__nv_bfloat16 *>(a.Y), (int)a.N, (int)a.K, L, a.status);
}

}  // namespace

// Whether the tcgen05 kernel can take this call (batch 1; the activations' 8 bytes per element and the rings fit shared
// memory; unless `any_size`, enough 128-row tiles to occupy the GPU), and with how many warpgroups.
int gemv_lut_tc_warpgroups(int bits, int64_t N, int64_t K, int64_t B, int sms, bool any_size)
{
    if (B != 1 || K > kLutMaxK) return 0;
    const int64_t ntiles = (N + 127) / 128;
    if (!any_size && ntiles * 10 < (int64_t)sms * 6) return 0;
    TcPlan L;
    for (int wgs = kMaxWgs; wgs >= 2; --wgs)
        if (tc_plan(bits, (int)K, wgs, L) <= kTcSmemLimit && 2 * lut_slices(K) >= wgs) return wgs;
    return 0;
}

cudaError_t launch_gemv_lut_tc(const GemvArgs &a, int wgs, cudaStream_t stream)
{
    if (a.bits != 2 && a.bits != 3) return cudaErrorInvalidValue;
    if (a.B != 1 || wgs < 1 || wgs > kMaxWgs) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    TcPlan L;
    const uint32_t smem = tc_plan(a.bits, (int)a.K, wgs, L);
    if (smem > kTcSmemLimit) return cudaErrorInvalidValue;
    L.wait_cycles = a.wait_cycles > 0 ? a.wait_cycles : tc::kWaitBudgetCycles;
    L.drop_first_copy = a.drop_first_copy;
    const int64_t ntiles = (a.N + 127) / 128;
    const int grid = (int)(ntiles < sms ? ntiles : sms);
    return a.bits == 3 ? launch_tc<3>(a, L, smem, grid, stream) : launch_tc<2>(a, L, smem, grid, stream);
}

}  // namespace dq
