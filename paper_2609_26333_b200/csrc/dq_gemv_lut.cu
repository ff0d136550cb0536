// LUT3 / LUT2 weight-only decode (App. C.2 "Kernel specification"; the skinny-batch case the paper leaves open, Sec. 5):
//   Y[b][n] = bf16( s * sum_blk d_blk(n) * sum_{k in blk} G[idx(n,k)] * X[b][k] ),   up to eight batch columns per pass.
//
// Arithmetic.  Every product G[idx] * x is exact: the fp16 codebook levels go to the tensor cores unscaled
// (mma.sync.m16n8k16, fp32 accumulation), the bf16 activations are scaled by one power of two into fp16 (no
// rounding for any element within 2^28 of the largest of the pass), and one mma contracts exactly one 16-weight
// block per row, so that the signed E4M3 block scale multiplies the block's fp32 sum afterwards, in fp32:
//   acc += d_blk * (sum of 16 exact products).
// Nothing is rounded before the fp32 accumulation, whatever the activations look like (dense, sparse, cancelling).
//
// Work split.  A row tile is 8 rows.  The 16 rows of the mma's A operand are the 8 rows of the tile against two
// neighbouring blocks b, b+1; the B operand holds block b of the activations in columns 0-3 (one per batch column)
// and block b+1 in columns 4-7, so accumulator entries (row g, column c) and (row g+8, column 4+c) are the two
// halves of one output and the cross terms are dropped.  With five to eight batch columns the levels of a lane, once
// looked up, go through a second mma against the activations of columns 4-7 (template parameter CG, column groups).
// Lane (g, t) supplies weights 4t .. 4t+3 of both blocks of row g, which is how the device layout stores them
// (dq_common.cuh).  A group of P warps shares a tile, warp w
// taking 1024-weight slices w, w+P, .. (P = 1: a warp owns whole tiles and stores its outputs itself; otherwise
// the last warp of the group to arrive adds the partial tiles in a fixed order); G groups per CTA, one or two
// CTAs per SM, tiles dealt round robin.
//
// Memory.  Every warp streams its own chunks (8 rows x 1024 weights = two atoms, 3584 B for LUT3) through a ring of
// S bulk copies (cp.async.bulk + mbarrier) in shared memory, refilling a stage as soon as its words sit in registers.
// Dequantisation is register-only: the stored words are byte-permute selectors after one AND, two permutes fetch the
// low and high bytes of four levels from the codebook held in four registers and two more interleave them into two
// fp16 pairs.  The 256 block scales of an atom are converted to fp32 once per warp (eight per lane) and parked in a
// small per-warp buffer; a lane reads its row's scales and its B fragments with 16-byte loads, two mmas per load.
//
// What bounds it.  On this GPU a warp instruction of the integer / logic / permute class occupies the issue port of
// its SM sub-partition for two cycles (measured: 8 PRMT + 8 FFMA take 24 cycles, not 16), so the kernel is bound by
// instruction issue: about 8 permutes, 2 logic ops, 2 shifts, 1 mma, 4 FFMA and 2 shared loads per 8 weights of a lane.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_common.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

constexpr int kSlots = 4;                         // cross-warp reduction slots per row group
constexpr uint32_t kSmemLimit = 227 * 1024;
constexpr uint32_t kSmemLimitHalf = 113 * 1024;   // two CTAs per SM
constexpr int kMaxWarps = 24;
constexpr int kMaxGroups = 16;
constexpr uint32_t kScaleBufBytes = 1152;         // per warp: 8 rows x 36 floats (32 block scales + 4 of padding)

// shared-memory map (byte offsets from the start of dynamic shared memory) and work split, filled in by the launcher
struct LutPlan {
    int P, G, S;                      // warps per row group, row groups per CTA, ring stages per warp
    uint32_t bar_off;                 // ring barriers: [warp][S] x 8 B
    uint32_t red_off;                 // reduction slots: [G][kSlots][P][32] floats
    uint32_t sbuf_off;                // per warp: 8 rows x 32 fp32 block scales of the atom being worked on
    uint32_t ring_off;                // [warp][S][atom]
    uint32_t x_off;                   // [cols][col_stride] fp16 activations
    uint32_t col_stride;
    long long wait_cycles;
    int drop_first_copy;              // test hook: CTA 0 / warp 0 never requests its first atom, so that its wait runs out
};

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1)
{
    // C = 0 as an operand of its own: tied to D it would have to be cleared in registers before every mma
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%10, %10, %10, %10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}
// 8-byte shared-memory load at base + OFF (the offset is an immediate of the instruction)
template <int OFF>
__device__ __forceinline__ uint2 lds_v2_at(uint32_t base)
{
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2+%3];" : "=r"(v.x), "=r"(v.y) : "r"(base), "n"(OFF));
    return v;
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
__device__ __forceinline__ void sts_v4f(uint32_t addr, float4 v)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
template <int OFF>
__device__ __forceinline__ float4 lds_v4f_at(uint32_t base)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+%5];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(base), "n"(OFF));
    return v;
}

// byte permute, selector taken as it is (nibbles with the top bit clear select bytes 0-7 of {a, b})
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

struct Codebook { uint32_t tl0, tl1, th0, th1; };    // low bytes of levels 0-3 / 4-7, high bytes of levels 0-3 / 4-7

// Two neighbouring blocks of the atom (selector word `sel`: low half the first block, high half the second) against
// their activations: the levels are looked up once, then one mma per group of four batch columns (x0[c], x1[c] its B
// fragments) and the two block scales d0, d1 (fp32) on the two block sums.
// (ONE: a single batch column; the odd accumulator columns are never read and are not kept up.)
template <int CG, bool ONE>
__device__ __forceinline__ void block_pair(uint32_t sel, const uint32_t (&x0)[CG], const uint32_t (&x1)[CG], float d0, float d1,
                                           const Codebook &cb, float (&acc)[CG][4])
{
    const uint32_t u1 = sel >> 16;
    const uint32_t lo0 = prmt(cb.tl0, cb.tl1, sel), hi0 = prmt(cb.th0, cb.th1, sel);
    const uint32_t a0 = prmt(lo0, hi0, 0x5140u), a2 = prmt(lo0, hi0, 0x7362u);     // row g, first block
    const uint32_t lo1 = prmt(cb.tl0, cb.tl1, u1), hi1 = prmt(cb.th0, cb.th1, u1);
    const uint32_t a1 = prmt(lo1, hi1, 0x5140u), a3 = prmt(lo1, hi1, 0x7362u);     // "row g+8": second block
#pragma unroll
    for (int c = 0; c < CG; ++c) {
        float d[4];
        mma16816(d, a0, a1, a2, a3, x0[c], x1[c]);
        acc[c][0] = fmaf(d[0], d0, acc[c][0]);
        if (!ONE) acc[c][1] = fmaf(d[1], d0, acc[c][1]);
        acc[c][2] = fmaf(d[2], d1, acc[c][2]);
        if (!ONE) acc[c][3] = fmaf(d[3], d1, acc[c][3]);
    }
}

// One word group (32 weights of this lane: four of each of the blocks 8 WI .. 8 WI + 7 of the atom).  The group's
// activations (this lane's column of column group c, block parity and quarter of a block) are 32 contiguous bytes at
// xa[c] + 256 WI, its eight block scales eight contiguous floats at sa + 32 WI: 16-byte loads serve two mmas each.
template <int BITS, int WI, int CG, bool ONE>
__device__ __forceinline__ void group_dot(const uint32_t (&w)[BITS], const uint32_t (&xa)[CG], uint32_t sa, const Codebook &cb,
                                          float (&acc)[CG][4])
{
    uint32_t sel[4];
    lut_selectors<BITS>(w, sel);
    uint4 xA[CG], xB[CG];
#pragma unroll
    for (int c = 0; c < CG; ++c) {
        xA[c] = lds_v4_at<WI * 256>(xa[c]);
        xB[c] = lds_v4_at<WI * 256 + 16>(xa[c]);
    }
    const float4 dA = lds_v4f_at<WI * 32>(sa), dB = lds_v4f_at<WI * 32 + 16>(sa);
    uint32_t p0[CG], p1[CG];
#pragma unroll
    for (int c = 0; c < CG; ++c) { p0[c] = xA[c].x; p1[c] = xA[c].y; }
    block_pair<CG, ONE>(sel[0], p0, p1, dA.x, dA.y, cb, acc);
#pragma unroll
    for (int c = 0; c < CG; ++c) { p0[c] = xA[c].z; p1[c] = xA[c].w; }
    block_pair<CG, ONE>(sel[1], p0, p1, dA.z, dA.w, cb, acc);
#pragma unroll
    for (int c = 0; c < CG; ++c) { p0[c] = xB[c].x; p1[c] = xB[c].y; }
    block_pair<CG, ONE>(sel[2], p0, p1, dB.x, dB.y, cb, acc);
#pragma unroll
    for (int c = 0; c < CG; ++c) { p0[c] = xB[c].z; p1[c] = xB[c].w; }
    block_pair<CG, ONE>(sel[3], p0, p1, dB.z, dB.w, cb, acc);
}

// One atom of this lane's row: BITS index words x 4 word groups, against the fp16 activations at shared addresses xa[c]
// + xoff (this lane's column of every column group and block parity; layout in the kernel) and the row's 32 block
// scales as fp32 at shared address sa.
template <int BITS, int CG, bool ONE>
__device__ __forceinline__ void atom_dot(const uint4 (&pw)[BITS], const uint32_t (&xlane)[CG], uint32_t xoff, uint32_t sa,
                                         const Codebook &cb, float (&acc)[CG][4])
{
    uint32_t xa[CG];
#pragma unroll
    for (int c = 0; c < CG; ++c) xa[c] = xlane[c] + xoff;      // xoff is 0 or one atom: folded where it is 0
    uint32_t w[BITS];
#pragma unroll
    for (int p = 0; p < BITS; ++p) w[p] = pw[p].x;
    group_dot<BITS, 0, CG, ONE>(w, xa, sa, cb, acc);
#pragma unroll
    for (int p = 0; p < BITS; ++p) w[p] = pw[p].y;
    group_dot<BITS, 1, CG, ONE>(w, xa, sa, cb, acc);
#pragma unroll
    for (int p = 0; p < BITS; ++p) w[p] = pw[p].z;
    group_dot<BITS, 2, CG, ONE>(w, xa, sa, cb, acc);
#pragma unroll
    for (int p = 0; p < BITS; ++p) w[p] = pw[p].w;
    group_dot<BITS, 3, CG, ONE>(w, xa, sa, cb, acc);
}

// Activations of one column in shared memory, fp16.  An atom (512 weights, 32 blocks) takes 1024 bytes ordered
// [word group 4][block parity 2][quarter t 4][block pair 4][4 weights], so that the four B fragments lane (., t) needs for
// the four mmas of a word group (blocks 8 wi + 2a + parity, weights 4t .. 4t+3, a = 0..3) are 32 contiguous bytes.
// Byte offset of the eight weights 8 i .. 8 i + 7 (a quarter pair t = 2h, 2h+1 of one block; the second quarter 32 bytes on):
__device__ __forceinline__ uint32_t x_offset(int i)
{
    const uint32_t atom = (uint32_t)i >> 6, bb = ((uint32_t)i >> 1) & 31u, h = (uint32_t)i & 1u;
    return atom * 1024u + (bb >> 3) * 256u + (bb & 1u) * 128u + h * 64u + ((bb >> 1) & 3u) * 8u;
}

__device__ __forceinline__ uint32_t lds_u32_volatile(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void fence_cta() { asm volatile("fence.acq_rel.cta;" ::: "memory"); }

template <int BITS, int MAXT, int MINB, int CG, bool ONE>
__global__ void __launch_bounds__(MAXT, MINB)
gemv_lut_kernel(const uint8_t *__restrict__ lut, const PackedHeader *__restrict__ hdr,
                const __nv_bfloat16 *__restrict__ X, int64_t ldx, int b0, int cols,
                __nv_bfloat16 *__restrict__ Y, int64_t ldy, int N, int K, LutPlan L, StatusWord *status)
{
    constexpr uint32_t kAtom = (uint32_t)lut_atom_bytes(BITS);
    constexpr uint32_t kChunk = 2u * kAtom;                 // one ring stage: 8 rows x 1024 weights
    constexpr uint32_t kPlanes = (uint32_t)lut_plane_bytes(BITS);
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t win0 = (uint32_t)__cvta_generic_to_shared(smem_raw);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw);
    int *sync_words = reinterpret_cast<int *>(smem_raw + 64);                           // [G][kSlots] x (generation, count)
    float *xmax_s = reinterpret_cast<float *>(smem_raw + 640);                          // 32 per-warp maxima
    float *red = reinterpret_cast<float *>(smem_raw + L.red_off);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int P = L.P, G = L.G, S = L.S;
    const int grp = warp / P;
    const int w = warp - grp * P;
    const int g = lane >> 2, t = lane & 3;
    const int nslices = (int)lut_slices(K);
    const int kpad = nslices * kLutSlice;

    // ---- this warp's ring: S stages of one chunk each, one barrier per stage; nobody else touches them
    const uint32_t ring0 = win0 + L.ring_off + (uint32_t)warp * (uint32_t)S * kChunk;
    const uint32_t bars0 = win0 + L.bar_off + (uint32_t)warp * (uint32_t)S * 8u;
    if (lane == 0) {
        for (int i = 0; i < S; ++i) tc::mbar_init(bars0 + 8u * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x < kMaxGroups * kSlots * 2) sync_words[threadIdx.x] = 0;
    if (threadIdx.x == 0) *abort_flag = 0;
    __syncwarp();

    // slices w, w + P, .. of every tile this warp's group owns
    const int ns = (w < nslices) ? (nslices - w + P - 1) / P : 0;
    const int ntiles = N / kLutAtomRows;
    const int stride = gridDim.x * G;
    const int first = blockIdx.x * G + grp;
    const size_t slice_step = (size_t)P * 4u * kAtom;         // bytes between slices s and s + P of one tile
    auto tile_base = [&](int tile) {                           // chunk (tile, slice w)
        return lut + (((size_t)(tile >> 1) * nslices + w) * 4u + (size_t)(tile & 1) * 2u) * kAtom;
    };
    // Producer state: next chunk to request, its ring stage and barrier.  Every lane keeps it (the arithmetic is uniform),
    // lane 0 issues: fence, expected bytes and copy are predicated instructions, not a divergent branch.
    const uint8_t *psrc = tile_base(first);
    int pslice = 0, ptile = (ns > 0) ? first : ntiles;                   // ptile >= ntiles: nothing left to request
    uint32_t pdst = ring0, pbar = bars0;
    const uint32_t ring_end = ring0 + (uint32_t)S * kChunk;
    auto advance = [&]() {
        if (++pslice == ns) { pslice = 0; ptile += stride; psrc = tile_base(ptile); }
        else psrc += slice_step;
        pdst += kChunk;
        pbar += 8u;
        if (pdst == ring_end) { pdst = ring0; pbar = bars0; }
    };
    auto issue_next = [&](bool skip_copy) {
        const uint32_t doit = (lane == 0 && ptile < ntiles && !skip_copy) ? 1u : 0u;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %0, 0;\n\t"
            "@p fence.proxy.async.shared::cta;\n\t"
            "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%1], %2;\n\t"
            "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%3], [%4], %2, [%1];\n\t}"
            ::"r"(doit), "r"(pbar), "r"(kChunk), "r"(pdst), "l"(psrc) : "memory");
        advance();
    };
    // The weights are constant data: start streaming before waiting for the kernel ahead of this one.
    {
        const bool drop = L.drop_first_copy && blockIdx.x == 0 && warp == 0;
        for (int i = 0; i < S && ptile < ntiles; ++i) issue_next(drop && i == 0);    // test hook: the dropped chunk is never requested
    }
    const uint4 cbv = *reinterpret_cast<const uint4 *>(BITS == 3 ? hdr->lut_prmt : hdr->lut2_prmt);
    const Codebook cb = {cbv.x, cbv.y, cbv.z, cbv.w};
    const float s_w = hdr->s;

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- activations of this pass: one read from global memory (raw bf16 parked in shared memory, largest
    //      magnitude on the way), then power-of-two scale -> fp16 in place
    uint8_t *xh = smem_raw + L.x_off;
    float m = 0.0f;
    for (int c = 0; c < cols; ++c) {
        const uint4 *xp = reinterpret_cast<const uint4 *>(X + (int64_t)(b0 + c) * ldx);
        for (int i = threadIdx.x; i < kpad / 8; i += blockDim.x) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);                 // the padding of a short last slice reads as zero
            if (i < K / 8) v = __ldg(xp + i);
            // |bf16| pairs compare like unsigned integers once the sign bits are cleared
            const uint32_t a0 = v.x & 0x7FFF7FFFu, a1 = v.y & 0x7FFF7FFFu, a2 = v.z & 0x7FFF7FFFu, a3 = v.w & 0x7FFF7FFFu;
            const uint32_t hi = max(max(a0 >> 16, a1 >> 16), max(a2 >> 16, a3 >> 16));
            const uint32_t lo = max(max(a0 & 0xFFFFu, a1 & 0xFFFFu), max(a2 & 0xFFFFu, a3 & 0xFFFFu));
            m = fmaxf(m, __uint_as_float(max(hi, lo) << 16));
            uint8_t *dst = xh + (size_t)c * L.col_stride + x_offset(i);
            *reinterpret_cast<uint2 *>(dst) = make_uint2(v.x, v.y);
            *reinterpret_cast<uint2 *>(dst + 32) = make_uint2(v.z, v.w);
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
    const float xinv = __uint_as_float((uint32_t)(127 - 14 + ex) << 23);
    for (int c = 0; c < cols; ++c) {
        for (int i = threadIdx.x; i < kpad / 8; i += blockDim.x) {        // every thread converts what it parked itself
            uint8_t *px = xh + (size_t)c * L.col_stride + x_offset(i);
            const uint2 va = *reinterpret_cast<const uint2 *>(px), vb = *reinterpret_cast<const uint2 *>(px + 32);
            const uint32_t ww[4] = {va.x, va.y, vb.x, vb.y};
            uint32_t r[4];
#pragma unroll
            for (int z = 0; z < 4; ++z) {
                const __half2 h = __floats2half2_rn(__uint_as_float(ww[z] << 16) * xscale,
                                                    __uint_as_float(ww[z] & 0xFFFF0000u) * xscale);
                r[z] = *reinterpret_cast<const uint32_t *>(&h);
            }
            *reinterpret_cast<uint2 *>(px) = make_uint2(r[0], r[1]);
            *reinterpret_cast<uint2 *>(px + 32) = make_uint2(r[2], r[3]);
        }
    }
    __syncthreads();
    const float out_scale = s_w * xinv;
    // B operand of this lane in column group c: column 4c + g % 4 (column 0 where the pass has fewer), block parity g / 4,
    // weights 4t .. 4t+3
    uint32_t xlane[CG];
#pragma unroll
    for (int c = 0; c < CG; ++c) {
        const int colsel = (4 * c + (g & 3) < cols) ? 4 * c + (g & 3) : 0;
        xlane[c] = win0 + L.x_off + (uint32_t)colsel * L.col_stride + (uint32_t)(g >> 2) * 128u + (uint32_t)t * 32u +
                   (uint32_t)w * (kLutSlice * 2u);
    }
    const uint32_t lane_plane = (uint32_t)lane * 16u;
    // this warp's fp32 scale buffer: 8 rows x 32 blocks; lane l converts bytes 8 l .. 8 l + 7 of the atom's scale bytes
    // (row l / 4, blocks 8 (l % 4) ..), which land at float 8 l of the buffer: row-major like the bytes
    const uint32_t sbuf = win0 + L.sbuf_off + (uint32_t)warp * kScaleBufBytes;
    const uint32_t srow = sbuf + (uint32_t)g * 144u;                        // rows 36 floats apart: conflict-free reads
    const uint32_t swr = sbuf + (uint32_t)(lane >> 2) * 144u + (uint32_t)(lane & 3) * 32u;
    const uint32_t sync0 = win0 + 64u + (uint32_t)grp * kSlots * 8u;

    uint32_t cbase = ring0, cbar = bars0;                     // consumer's ring stage and its barrier
    uint32_t phase = 0;
    int tile = first;
    for (int it = 0; tile < ntiles; ++it, tile += stride) {
        float acc[CG][4];
#pragma unroll
        for (int c = 0; c < CG; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.0f;
        for (int sl = 0; sl < ns; ++sl) {
            // The chunk is normally there already.  Otherwise poll with back-off; a wait that runs out ends the kernel
            // for this warp (the others find the flag in their own waits).
            if (!__any_sync(0xffffffffu, tc::mbar_try(cbar, phase))) {
                const long long t0 = clock64();
                bool got = false;
                while (true) {
                    __nanosleep(32);
                    got = __any_sync(0xffffffffu, tc::mbar_try(cbar, phase));
                    if (got) break;
                    if (__any_sync(0xffffffffu, *abort_flag != 0 || clock64() - t0 > L.wait_cycles)) break;
                }
                if (!got) { *abort_flag = 1; goto give_up; }
            }
            {
                uint4 pw[BITS];
                uint2 s8;
                // atom 0: index words to registers; the warp converts the atom's 256 block scales to fp32 once (8 per
                // lane) and parks them in its scale buffer, from which every lane reads its row's
                pw[0] = lds_v4_at<0>(cbase + lane_plane);
                pw[1] = lds_v4_at<512>(cbase + lane_plane);
                if (BITS == 3) pw[BITS - 1] = lds_v4_at<1024>(cbase + lane_plane);
                s8 = lds_v2_at<(int)kPlanes>(cbase + (uint32_t)lane * 8u);
                __syncwarp();                                          // everybody is done with the buffer's last contents
                sts_v4f(swr, e4m3x4_to_f32(s8.x));
                sts_v4f(swr + 16u, e4m3x4_to_f32(s8.y));
                __syncwarp();
                atom_dot<BITS, CG, ONE>(pw, xlane, 0u, srow, cb, acc);
                pw[0] = lds_v4_at<(int)kAtom>(cbase + lane_plane);
                pw[1] = lds_v4_at<(int)kAtom + 512>(cbase + lane_plane);
                if (BITS == 3) pw[BITS - 1] = lds_v4_at<(int)kAtom + 1024>(cbase + lane_plane);
                s8 = lds_v2_at<(int)(kAtom + kPlanes)>(cbase + (uint32_t)lane * 8u);
                // the stage is in registers: refill it with the chunk S steps ahead
                __syncwarp();
                issue_next(false);
                sts_v4f(swr, e4m3x4_to_f32(s8.x));
                sts_v4f(swr + 16u, e4m3x4_to_f32(s8.y));
                __syncwarp();
                atom_dot<BITS, CG, ONE>(pw, xlane, kLutAtomK * 2u, srow, cb, acc);
            }
            cbase += kChunk;
            cbar += 8u;
            if (cbase == ring_end) { cbase = ring0; cbar = bars0; phase ^= 1u; }
#pragma unroll
            for (int c = 0; c < CG; ++c) xlane[c] += (uint32_t)P * (kLutSlice * 2u);      // this warp's next slice
        }
#pragma unroll
        for (int c = 0; c < CG; ++c) xlane[c] -= (uint32_t)(ns * P) * (kLutSlice * 2u);   // back to its first slice
        // halves of an output: (row g, column c) in lanes t < 2 and (row g + 8, column 4 + c) in lanes t >= 2
        float v0[CG], v1[CG];
#pragma unroll
        for (int c = 0; c < CG; ++c) {
            v0[c] = acc[c][0] + __shfl_xor_sync(0xffffffffu, acc[c][2], 2);
            v1[c] = acc[c][1] + __shfl_xor_sync(0xffffffffu, acc[c][3], 2);
        }
        if (P == 1) {
            // the warp owns the whole tile: lanes t < 2 hold (row g, columns 4c + 2t, 4c + 2t + 1) of column group c
            if (t < 2) {
                const int row = tile * kLutAtomRows + g;
#pragma unroll
                for (int c = 0; c < CG; ++c) {
                    const int col = 4 * c + 2 * t;
                    if (col < cols) Y[(int64_t)(b0 + col) * ldy + row] = __float2bfloat16_rn(v0[c] * out_scale);
                    if (col + 1 < cols) Y[(int64_t)(b0 + col + 1) * ldy + row] = __float2bfloat16_rn(v1[c] * out_scale);
                }
            }
            continue;
        }
        // ---- cross-warp sum: last-arriving warp of the group adds the P partial tiles in order and stores
        const int slot = it & (kSlots - 1);
        const uint32_t gen_addr = sync0 + (uint32_t)slot * 8u;
        int *cnt = sync_words + (grp * kSlots + slot) * 2 + 1;
        {
            uint32_t good = 1;
            if (lane == 0) {
                const uint32_t want = (uint32_t)(it / kSlots);
                long long t0 = 0;
                uint32_t spins = 0;
                while (lds_u32_volatile(gen_addr) != want) {
                    if ((++spins & 255u) == 0u) {
                        if (t0 == 0) t0 = clock64();
                        if (*abort_flag || clock64() - t0 > L.wait_cycles) { *abort_flag = 1; good = 0; break; }
                    }
                }
            }
            if (__shfl_sync(0xffffffffu, good, 0) == 0) goto give_up;
        }
        float *rbuf = red + (size_t)((grp * kSlots + slot) * P) * (32 * CG);        // [warp][column group][row 8][column 4]
        if (t < 2) {
#pragma unroll
            for (int c = 0; c < CG; ++c)
                *reinterpret_cast<float2 *>(rbuf + w * (32 * CG) + c * 32 + g * 4 + 2 * t) = make_float2(v0[c], v1[c]);
        }
        __syncwarp();
        int prev = 0;
        if (lane == 0) { fence_cta(); prev = atomicAdd(cnt, 1); }
        prev = __shfl_sync(0xffffffffu, prev, 0);
        if (prev == P - 1) {
            fence_cta();
#pragma unroll
            for (int c = 0; c < CG; ++c) {
                float tot = 0.0f;
                for (int ww = 0; ww < P; ++ww) tot += *reinterpret_cast<const volatile float *>(rbuf + ww * (32 * CG) + c * 32 + lane);
                const int col = 4 * c + (lane & 3), row = tile * kLutAtomRows + (lane >> 2);
                if (col < cols) Y[(int64_t)(b0 + col) * ldy + row] = __float2bfloat16_rn(tot * out_scale);
            }
            __syncwarp();
            if (lane == 0) {
                *cnt = 0;
                fence_cta();
                asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(gen_addr), "r"((uint32_t)(it / kSlots + 1)) : "memory");
            }
        }
    }
give_up:
    if (*abort_flag) {
        // a wait ran out: let copies in flight land before the CTA's shared memory is handed on, then report
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        if (lane == 0) {
            atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
            atomicExch(&status->detail, 0x36000 | (int)blockIdx.x);
        }
    }
}

template <int BITS, int MAXT, int MINB, int CG, bool ONE>
cudaError_t launch_one(const GemvArgs &a, int b0, int cols, int grid, int threads, const LutPlan &L, uint32_t smem,
                       cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemv_lut_kernel<BITS, MAXT, MINB, CG, ONE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        // every instantiation asks for the same split of the SM's memory between L1 and shared memory: a change of
        // the split between two launches has to wait until the SM is empty, which would undo the overlap of one
        // launch's set-up with the tail of the launch before it
        e = cudaFuncSetAttribute(gemv_lut_kernel<BITS, MAXT, MINB, CG, ONE>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 (int)cudaSharedmemCarveoutMaxShared);
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
    return cudaLaunchKernelEx(&cfg, gemv_lut_kernel<BITS, MAXT, MINB, CG, ONE>, a.lut, a.hdr, reinterpret_cast<const __nv_bfloat16 *>(a.X),
                              (int64_t)a.ldx, b0, cols, reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.N,
                              (int)a.K, L, a.status);
}


// ---------------------------------------------------------------------------------------------------------------
// Batches above 8: up to 32 columns in one pass over the weights.  Their activations do not fit shared memory for a
// whole row, so the CTA walks K slice by slice (1024 weights): all warps stage the slice's activations together
// (largest magnitude of the slice -> power-of-two scale -> fp16; the scale's inverse goes into the block scales of the
// slice, which keeps every product exact whatever the other slices hold), then every warp contracts the chunk of its
// own tile against them.  Here a tile is 16 rows (the two row halves of the device layout side by side): the 16 rows
// of the mma's A operand are 16 rows of one block, its 8 columns 8 batch columns, so every accumulator entry is an
// output and a column costs half the mmas and FFMA of the layout above; the levels of a word group are looked up once
// and go through one mma per block and group of eight columns.  A warp owns whole tiles (one per round over the rows);
// a ring stage is the four atoms of a tile and slice, one bulk copy.
struct WidePlan {
    uint32_t bar_off, sbuf_off, ring_off, x_off, col_stride;
    long long wait_cycles;
};

// Activations of one column and slice, fp16: an atom (32 blocks) takes 1024 bytes ordered [word group 4][block pair 4]
// [quarter t 4][block parity 2][4 weights], so that the B fragments lane (., t) needs for a pair of blocks are 16
// contiguous bytes.  Byte offset of weights 4t .. 4t+3 of block blk (0..63) of the slice:
__device__ __forceinline__ uint32_t x16_offset(uint32_t blk, uint32_t t)
{
    return (blk >> 5) * 1024u + ((blk & 31u) >> 3) * 256u + ((blk & 7u) >> 1) * 64u + t * 16u + (blk & 1u) * 8u;
}

// One word group of two atoms (rows g and g + 8 of the tile): eight blocks, one mma each per group of eight columns.
template <int BITS, int WI, int CG8>
__device__ __forceinline__ void group_dot16(const uint32_t (&w0)[BITS], const uint32_t (&w1)[BITS], uint32_t xa, uint32_t group_stride,
                                            uint32_t sa0, uint32_t sa1, const Codebook &cb, float (&acc)[CG8][4])
{
    uint32_t s0[4], s1[4];
    lut_selectors<BITS>(w0, s0);
    lut_selectors<BITS>(w1, s1);
    uint32_t a[8][4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t u0 = h ? (s0[q] >> 16) : s0[q], u1 = h ? (s1[q] >> 16) : s1[q];
            const uint32_t lo0 = prmt(cb.tl0, cb.tl1, u0), hi0 = prmt(cb.th0, cb.th1, u0);
            const uint32_t lo1 = prmt(cb.tl0, cb.tl1, u1), hi1 = prmt(cb.th0, cb.th1, u1);
            a[2 * q + h][0] = prmt(lo0, hi0, 0x5140u);       // row g,     weights 4t, 4t+1
            a[2 * q + h][1] = prmt(lo1, hi1, 0x5140u);       // row g + 8
            a[2 * q + h][2] = prmt(lo0, hi0, 0x7362u);       // row g,     weights 4t+2, 4t+3
            a[2 * q + h][3] = prmt(lo1, hi1, 0x7362u);
        }
    }
    const float4 e0 = lds_v4f_at<WI * 32>(sa0), e1 = lds_v4f_at<WI * 32 + 16>(sa0);
    const float4 f0 = lds_v4f_at<WI * 32>(sa1), f1 = lds_v4f_at<WI * 32 + 16>(sa1);
    const float dlo[8] = {e0.x, e0.y, e0.z, e0.w, e1.x, e1.y, e1.z, e1.w};     // row g
    const float dhi[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};     // row g + 8
#pragma unroll
    for (int c = 0; c < CG8; ++c) {
        const uint4 x0 = lds_v4_at<WI * 256>(xa), x1 = lds_v4_at<WI * 256 + 64>(xa);
        const uint4 x2 = lds_v4_at<WI * 256 + 128>(xa), x3 = lds_v4_at<WI * 256 + 192>(xa);
        xa += group_stride;
        const uint32_t xs[16] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w, x2.x, x2.y, x2.z, x2.w, x3.x, x3.y, x3.z, x3.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float r[4];
            mma16816(r, a[i][0], a[i][1], a[i][2], a[i][3], xs[2 * i], xs[2 * i + 1]);
            acc[c][0] = fmaf(r[0], dlo[i], acc[c][0]);
            acc[c][1] = fmaf(r[1], dlo[i], acc[c][1]);
            acc[c][2] = fmaf(r[2], dhi[i], acc[c][2]);
            acc[c][3] = fmaf(r[3], dhi[i], acc[c][3]);
        }
    }
}

template <int BITS, int CG8>
__device__ __forceinline__ void atom_dot16(const uint4 (&pw0)[BITS], const uint4 (&pw1)[BITS], uint32_t xa, uint32_t group_stride,
                                           uint32_t sa0, uint32_t sa1, const Codebook &cb, float (&acc)[CG8][4])
{
    uint32_t w0[BITS], w1[BITS];
#pragma unroll
    for (int p = 0; p < BITS; ++p) { w0[p] = pw0[p].x; w1[p] = pw1[p].x; }
    group_dot16<BITS, 0, CG8>(w0, w1, xa, group_stride, sa0, sa1, cb, acc);
#pragma unroll
    for (int p = 0; p < BITS; ++p) { w0[p] = pw0[p].y; w1[p] = pw1[p].y; }
    group_dot16<BITS, 1, CG8>(w0, w1, xa, group_stride, sa0, sa1, cb, acc);
#pragma unroll
    for (int p = 0; p < BITS; ++p) { w0[p] = pw0[p].z; w1[p] = pw1[p].z; }
    group_dot16<BITS, 2, CG8>(w0, w1, xa, group_stride, sa0, sa1, cb, acc);
#pragma unroll
    for (int p = 0; p < BITS; ++p) { w0[p] = pw0[p].w; w1[p] = pw1[p].w; }
    group_dot16<BITS, 3, CG8>(w0, w1, xa, group_stride, sa0, sa1, cb, acc);
}

template <int BITS, int CG8>
__global__ void __launch_bounds__(384, 1)
gemv_lut_wide_kernel(const uint8_t *__restrict__ lut, const PackedHeader *__restrict__ hdr,
                     const __nv_bfloat16 *__restrict__ X, int64_t ldx, int b0, int cols,
                     __nv_bfloat16 *__restrict__ Y, int64_t ldy, int N, int K, WidePlan L, StatusWord *status)
{
    constexpr uint32_t kAtom = (uint32_t)lut_atom_bytes(BITS);
    constexpr uint32_t kStage = 4u * kAtom;                  // the four atoms of one 16-row tile and slice
    constexpr uint32_t kPlanes = (uint32_t)lut_plane_bytes(BITS);
    constexpr int kCols = 8 * CG8;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t win0 = (uint32_t)__cvta_generic_to_shared(smem_raw);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw);
    float *xmax_s = reinterpret_cast<float *>(smem_raw + 64);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = blockDim.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int nslices = (int)lut_slices(K);
    const int ntiles = N / 16;
    const int per_round = gridDim.x * G;
    const int rounds = (ntiles + per_round - 1) / per_round;
    const int first = blockIdx.x * G + warp;

    const uint32_t ring0 = win0 + L.ring_off + (uint32_t)warp * 2u * kStage;
    const uint32_t bars0 = win0 + L.bar_off + (uint32_t)warp * 16u;
    const uint32_t ring_end = ring0 + 2u * kStage;
    if (lane == 0) {
        tc::mbar_init(bars0, 1);
        tc::mbar_init(bars0 + 8u, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x == 0) *abort_flag = 0;
    __syncwarp();

    // producer: the stages of this warp's tiles, slice after slice, round after round
    const uint8_t *psrc = lut + (size_t)first * nslices * kStage;
    int pslice = 0, ptile = first;
    uint32_t pdst = ring0, pbar = bars0;
    auto issue_next = [&]() {
        const uint32_t doit = (lane == 0 && ptile < ntiles) ? 1u : 0u;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %0, 0;\n\t"
            "@p fence.proxy.async.shared::cta;\n\t"
            "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%1], %2;\n\t"
            "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%3], [%4], %2, [%1];\n\t}"
            ::"r"(doit), "r"(pbar), "r"(kStage), "r"(pdst), "l"(psrc) : "memory");
        if (++pslice == nslices) { pslice = 0; ptile += per_round; psrc = lut + (size_t)ptile * nslices * kStage; }
        else psrc += kStage;
        pdst += kStage;
        pbar += 8u;
        if (pdst == ring_end) { pdst = ring0; pbar = bars0; }
    };
    issue_next();
    issue_next();
    const uint4 cbv = *reinterpret_cast<const uint4 *>(BITS == 3 ? hdr->lut_prmt : hdr->lut2_prmt);
    const Codebook cb = {cbv.x, cbv.y, cbv.z, cbv.w};
    const float s_w = hdr->s;

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    uint8_t *xh = smem_raw + L.x_off;
    // columns the pass does not have read as zero
    for (int i = threadIdx.x; i < (kCols - cols) * (int)(L.col_stride / 16); i += blockDim.x)
        *reinterpret_cast<uint4 *>(xh + (size_t)cols * L.col_stride + (size_t)i * 16) = make_uint4(0u, 0u, 0u, 0u);
    // B operand of this lane: column g of every group of eight, weights 4t .. 4t+3 of a pair of blocks per 16-byte load
    const uint32_t xlane = win0 + L.x_off + (uint32_t)g * L.col_stride + (uint32_t)t * 16u;
    const uint32_t group_stride = 8u * L.col_stride;
    const uint32_t lane_plane = (uint32_t)lane * 16u;
    // fp32 scale buffers of the two atoms (row halves) being worked on
    const uint32_t sbuf = win0 + L.sbuf_off + (uint32_t)warp * (2u * kScaleBufBytes);
    const uint32_t srow = sbuf + (uint32_t)g * 144u;
    const uint32_t swr = sbuf + (uint32_t)(lane >> 2) * 144u + (uint32_t)(lane & 3) * 32u;

    uint32_t cbase = ring0, cbar = bars0, phase = 0;
    bool dead = false;                                   // a wait of this warp ran out: it keeps walking, without data
    const int items = cols * 128;                        // 16-byte pieces of a slice's activations
    for (int r = 0, tile = first; r < rounds; ++r, tile += per_round) {
        const bool active = tile < ntiles;
        float acc[CG8][4];
#pragma unroll
        for (int c = 0; c < CG8; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.0f;
        for (int sl = 0; sl < nslices; ++sl) {
            // ---- the slice's activations: largest magnitude, power-of-two scale, fp16.  A thread's pieces are loaded in
            //      batches of eight (one trip to L2 per batch, not per piece); what does not fit one batch is read a
            //      second time after the reduction.
            constexpr int kBatch = 8;
            const int nbatch = (items + (int)blockDim.x * kBatch - 1) / ((int)blockDim.x * kBatch);
            uint4 v[kBatch];
            float m = 0.0f;
            auto piece_max = [&](const uint4 &q) {
                const uint32_t a0 = q.x & 0x7FFF7FFFu, a1 = q.y & 0x7FFF7FFFu, a2 = q.z & 0x7FFF7FFFu, a3 = q.w & 0x7FFF7FFFu;
                const uint32_t hi = max(max(a0 >> 16, a1 >> 16), max(a2 >> 16, a3 >> 16));
                const uint32_t lo = max(max(a0 & 0xFFFFu, a1 & 0xFFFFu), max(a2 & 0xFFFFu, a3 & 0xFFFFu));
                return __uint_as_float(max(hi, lo) << 16);
            };
            auto load_batch = [&](int bi) {                                   // eight loads in flight per thread
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int i = (bi * kBatch + u) * (int)blockDim.x + (int)threadIdx.x;
                    const int c = i >> 7, k8 = sl * 128 + (i & 127);
                    v[u] = make_uint4(0u, 0u, 0u, 0u);                       // beyond K (a short last slice): zero
                    if (i < items && k8 < K / 8) v[u] = __ldg(reinterpret_cast<const uint4 *>(X + (int64_t)(b0 + c) * ldx) + k8);
                }
            };
            for (int bi = 0; bi < nbatch; ++bi) {
                load_batch(bi);
#pragma unroll
                for (int u = 0; u < kBatch; ++u) m = fmaxf(m, piece_max(v[u]));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            if (lane == 0) xmax_s[(sl & 1) * 16 + warp] = m;
            __syncthreads();                             // maxima there; nobody reads the slice before this one any more
            m = (lane < G) ? xmax_s[(sl & 1) * 16 + lane] : 0.0f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            int ex = (int)((__float_as_uint(m) >> 23) & 0xFFu) - 127;
            ex = max(-100, min(100, ex));
            const float xscale = __uint_as_float((uint32_t)(127 + 14 - ex) << 23);      // 2^(14 - ex)
            const float sscale = __uint_as_float((uint32_t)(127 - 14 + ex) << 23);      // its inverse, into the block scales
            for (int bi = nbatch - 1; bi >= 0; --bi) {               // the last batch is still in registers
                if (bi != nbatch - 1) load_batch(bi);
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int i = (bi * kBatch + u) * (int)blockDim.x + (int)threadIdx.x;
                    if (i >= items) continue;
                    const uint32_t c = (uint32_t)i >> 7, j = (uint32_t)i & 127u;          // piece j: half h of block j / 2
                    const uint32_t ww[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    uint32_t h4[4];
#pragma unroll
                    for (int z = 0; z < 4; ++z) {
                        const __half2 h = __floats2half2_rn(__uint_as_float(ww[z] << 16) * xscale, __uint_as_float(ww[z] & 0xFFFF0000u) * xscale);
                        h4[z] = *reinterpret_cast<const uint32_t *>(&h);
                    }
                    uint8_t *px = xh + (size_t)c * L.col_stride + x16_offset(j >> 1, (j & 1u) * 2u);
                    *reinterpret_cast<uint2 *>(px) = make_uint2(h4[0], h4[1]);           // weights 4t .. 4t+3, t = 2h
                    *reinterpret_cast<uint2 *>(px + 16) = make_uint2(h4[2], h4[3]);      // t = 2h + 1
                }
            }
            __syncthreads();
            if (!active) continue;
            // ---- this warp's stage of the slice
            if (!dead && !__any_sync(0xffffffffu, tc::mbar_try(cbar, phase))) {
                const long long t0 = clock64();
                bool got = false;
                while (true) {
                    __nanosleep(32);
                    got = __any_sync(0xffffffffu, tc::mbar_try(cbar, phase));
                    if (got) break;
                    if (__any_sync(0xffffffffu, *abort_flag != 0 || clock64() - t0 > L.wait_cycles)) break;
                }
                if (!got) { *abort_flag = 1; dead = true; }
            }
            if (!dead) {
                // atoms of the stage: (row half 0, k half 0), (0, 1), (1, 0), (1, 1)
#pragma unroll
                for (int kh = 0; kh < 2; ++kh) {
                    uint4 pw0[BITS], pw1[BITS];
                    const uint32_t at0 = cbase + (uint32_t)kh * kAtom, at1 = cbase + (uint32_t)(2 + kh) * kAtom;
                    pw0[0] = lds_v4_at<0>(at0 + lane_plane);
                    pw0[1] = lds_v4_at<512>(at0 + lane_plane);
                    if (BITS == 3) pw0[BITS - 1] = lds_v4_at<1024>(at0 + lane_plane);
                    pw1[0] = lds_v4_at<0>(at1 + lane_plane);
                    pw1[1] = lds_v4_at<512>(at1 + lane_plane);
                    if (BITS == 3) pw1[BITS - 1] = lds_v4_at<1024>(at1 + lane_plane);
                    const uint2 sa = lds_v2_at<(int)kPlanes>(at0 + (uint32_t)lane * 8u);
                    const uint2 sb = lds_v2_at<(int)kPlanes>(at1 + (uint32_t)lane * 8u);
                    __syncwarp();                                  // everybody is done with the buffers' last contents
                    if (kh == 1) issue_next();                     // the stage is in registers: refill it
                    float4 f = e4m3x4_to_f32(sa.x);
                    sts_v4f(swr, make_float4(f.x * sscale, f.y * sscale, f.z * sscale, f.w * sscale));
                    f = e4m3x4_to_f32(sa.y);
                    sts_v4f(swr + 16u, make_float4(f.x * sscale, f.y * sscale, f.z * sscale, f.w * sscale));
                    f = e4m3x4_to_f32(sb.x);
                    sts_v4f(swr + kScaleBufBytes, make_float4(f.x * sscale, f.y * sscale, f.z * sscale, f.w * sscale));
                    f = e4m3x4_to_f32(sb.y);
                    sts_v4f(swr + kScaleBufBytes + 16u, make_float4(f.x * sscale, f.y * sscale, f.z * sscale, f.w * sscale));
                    __syncwarp();
                    atom_dot16<BITS, CG8>(pw0, pw1, xlane + (uint32_t)kh * 1024u, group_stride, srow, srow + kScaleBufBytes, cb, acc);
                }
                cbase += kStage;
                cbar += 8u;
                if (cbase == ring_end) { cbase = ring0; cbar = bars0; phase ^= 1u; }
            }
        }
        if (active && !dead) {
            // lane (g, t) holds rows g and g + 8 of the tile in columns 2t, 2t + 1 of every group of eight
#pragma unroll
            for (int c = 0; c < CG8; ++c) {
                const int row = tile * 16 + g, col = 8 * c + 2 * t;
                if (col < cols) {
                    Y[(int64_t)(b0 + col) * ldy + row] = __float2bfloat16_rn(acc[c][0] * s_w);
                    Y[(int64_t)(b0 + col) * ldy + row + 8] = __float2bfloat16_rn(acc[c][2] * s_w);
                }
                if (col + 1 < cols) {
                    Y[(int64_t)(b0 + col + 1) * ldy + row] = __float2bfloat16_rn(acc[c][1] * s_w);
                    Y[(int64_t)(b0 + col + 1) * ldy + row + 8] = __float2bfloat16_rn(acc[c][3] * s_w);
                }
            }
        }
    }
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        if (lane == 0) {
            atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
            atomicExch(&status->detail, 0x38000 | (int)blockIdx.x);
        }
    }
}

template <int BITS, int CG8>
cudaError_t launch_wide_one(const GemvArgs &a, int b0, int cols, int grid, int threads, const WidePlan &L, uint32_t smem,
                            cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemv_lut_wide_kernel<BITS, CG8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(gemv_lut_wide_kernel<BITS, CG8>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem < 114u * 1024u ? 114u * 1024u : smem;       // one CTA per SM
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_lut_wide_kernel<BITS, CG8>, a.lut, a.hdr, reinterpret_cast<const __nv_bfloat16 *>(a.X),
                              (int64_t)a.ldx, b0, cols, reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.N, (int)a.K, L,
                              a.status);
}

// all of B in passes of up to 32 columns
cudaError_t launch_wide(const GemvArgs &a, int sms, cudaStream_t stream)
{
    const int64_t ntiles = a.N / 16;
    const uint32_t stage = 4u * (uint32_t)lut_atom_bytes(a.bits);
    // Warps per CTA (each owns one 16-row tile per round): eight, two per scheduler.  A round takes about as long with
    // four warps as with eight (each warp is bound by the latency of its own instruction chain, and every CTA pays for
    // staging the slice whatever its size), nine put a third warp on one scheduler and that one sets the pace; so the
    // rounds are what counts, and fewer, fuller CTAs beat more, emptier ones even when SMs stay idle (measured on
    // ten shapes from 1024 to 34816 rows: 34816 x 5120 at batch 32, 85 us with 8 warps, 171 us with 5 warps and one
    // tile less on the busiest SM).
    int G = ntiles < 8 ? (int)ntiles : 8;
    if (a.force_G >= 1 && a.force_G <= 9) G = a.force_G;       // test hook
    WidePlan L;
    L.bar_off = 1024;
    L.sbuf_off = 2048;
    L.ring_off = L.sbuf_off + (uint32_t)G * 2u * kScaleBufBytes;
    L.x_off = (L.ring_off + (uint32_t)G * 2u * stage + 127u) & ~127u;
    L.col_stride = kLutSlice * 2u + 64u;                 // 64 mod 128: the 16-byte loads of two columns hit different banks
    L.wait_cycles = a.wait_cycles > 0 ? a.wait_cycles : tc::kWaitBudgetCycles;
    const int64_t need = (ntiles + G - 1) / G;
    const int grid = (int)(need < sms ? need : sms);
    for (int b0 = 0; b0 < (int)a.B;) {
        const int left = (int)a.B - b0;
        const int cg = left > 24 ? 4 : left > 16 ? 3 : left > 8 ? 2 : 1;
        const int cols = left < 8 * cg ? left : 8 * cg;
        const uint32_t smem = L.x_off + (uint32_t)(8 * cg) * L.col_stride;
        if (smem > kSmemLimit) return cudaErrorInvalidValue;
        cudaError_t e = cudaErrorInvalidValue;
        if (a.bits == 3) {
            if (cg == 4) e = launch_wide_one<3, 4>(a, b0, cols, grid, G * 32, L, smem, stream);
            else if (cg == 3) e = launch_wide_one<3, 3>(a, b0, cols, grid, G * 32, L, smem, stream);
            else if (cg == 2) e = launch_wide_one<3, 2>(a, b0, cols, grid, G * 32, L, smem, stream);
            else e = launch_wide_one<3, 1>(a, b0, cols, grid, G * 32, L, smem, stream);
        } else {
            if (cg == 4) e = launch_wide_one<2, 4>(a, b0, cols, grid, G * 32, L, smem, stream);
            else if (cg == 3) e = launch_wide_one<2, 3>(a, b0, cols, grid, G * 32, L, smem, stream);
            else if (cg == 2) e = launch_wide_one<2, 2>(a, b0, cols, grid, G * 32, L, smem, stream);
            else e = launch_wide_one<2, 1>(a, b0, cols, grid, G * 32, L, smem, stream);
        }
        if (e != cudaSuccess) return e;
        b0 += cols;
    }
    return cudaSuccess;
}

}  // namespace

// column groups (of four batch columns, one mma each) the kernel is instantiated for
static int col_groups(int cols) { return cols <= 4 ? 1 : 2; }
constexpr int kMaxCols = 8;      // 16 columns were measured: their activations leave room for 7 warps, no faster than two passes of 8

// Shared-memory map for P x G warps with S ring stages and `cols` activation columns; returns the bytes needed.
static uint32_t plan_smem(int bits, int K, int P, int G, int S, int cols, LutPlan &L)
{
    const int nwarps = P * G;
    const uint32_t chunk = 2u * (uint32_t)lut_atom_bytes(bits);
    L.P = P; L.G = G; L.S = S;
    L.bar_off = 1024;
    L.red_off = 2048;
    const uint32_t cg = (uint32_t)col_groups(cols);
    const uint32_t red_bytes = P > 1 ? (uint32_t)nwarps * kSlots * 32 * 4 * cg : 0u;  // no cross-warp sum when a warp owns whole tiles
    L.sbuf_off = (L.red_off + red_bytes + 127u) & ~127u;
    L.ring_off = L.sbuf_off + (uint32_t)nwarps * kScaleBufBytes;
    L.x_off = (L.ring_off + (uint32_t)nwarps * S * chunk + 127u) & ~127u;
    L.col_stride = (uint32_t)lut_slices(K) * kLutSlice * 2u + 16u;    // padded K in fp16; 16 mod 32 keeps two columns' 16-byte loads on different banks
    return L.x_off + (uint32_t)cols * L.col_stride;
}

struct Split { int P, G, slots, ctas, S, cols; };

// CTAs of one size class: `slots` of them fit an SM (registers at 80 per thread, shared memory), `ctas` are launched per
// SM.  (Classes with three or four slots and one of them left free for the first CTAs of the next launch in the stream
// were measured: the next launch gains nothing from moving in early, and the smaller CTAs lose 15 %.)
struct SizeClass { int slots, ctas, max_warps; uint32_t smem_cap; };
static const SizeClass kClasses[] = {
    {2, 2, 12, kSmemLimitHalf},
    {1, 1, kMaxWarps, kSmemLimit},
};

// Work split: P warps share a tile of 8 rows (each taking 1024-weight slices w, w+P, ..), G such groups per CTA, in the
// smallest size class the CTA fits.  Modelled time of a launch, in units of one chunk (8 rows x 1024 weights) of issue
// work per SM: what the busiest SM has to issue in whole rounds over the tiles (chunks per tile plus a charge per warp
// that visits the tile), stretched where fewer than 15 warps share the SM; all `want_cols` columns in one pass where
// shared memory allows.  Rings are two chunks deep: a third stage was never faster in sweeps over every feasible (P, G)
// on eighteen layer shapes (3072x3072 .. 57344x8192, 8192x28672), which is also where the constants come from: timed
// alone, launch after launch of one shape, the pick is within 3 % of the best split on average.  The worst case there
// (12288x4096, 17 %) is a shape whose best split alone is one CTA of 11 warps per SM; such light launches are avoided
// on purpose: between a launch of at most 12 warps per SM and one of 15 or more, in either order, about 2 us more pass
// than between two of a kind (measured on pairs of the 27B-class matrices: 27.8 against 23.3 us for qkv + o), and a
// token step alternates shapes.
static Split choose_split(int bits, int64_t N, int64_t K, int sms, int want_cols)
{
    const int nslices = (int)lut_slices(K);
    const int64_t ntiles = N / kLutAtomRows;
    double best = 1e300;
    Split sp = {1, 1, 1, 1, 2, 1};
    LutPlan tmp;
    for (int p = 1; p <= nslices && p <= kMaxWarps; ++p) {
        const int ns_max = (nslices + p - 1) / p;                                   // slices of warp 0
        for (int gg = 1; gg <= kMaxGroups && gg * p <= kMaxWarps; ++gg) {
            for (const SizeClass &sc : kClasses) {
                if (gg * p > sc.max_warps) continue;
                int cols = want_cols < kMaxCols ? want_cols : kMaxCols;
                while (cols > 1 && plan_smem(bits, (int)K, p, gg, 2, cols, tmp) > sc.smem_cap) --cols;
                if (plan_smem(bits, (int)K, p, gg, 2, cols, tmp) > sc.smem_cap) continue;
                if (cols < want_cols && sc.ctas > 1) continue;                      // rather one CTA per SM than a second pass
                // CTAs actually launched, CTAs on the busiest SM, rounds of the busiest group
                const int64_t need = (ntiles + gg - 1) / gg;
                const int64_t grid = need < (int64_t)sms * sc.ctas ? need : (int64_t)sms * sc.ctas;
                const int64_t rounds = (ntiles + grid * gg - 1) / (grid * gg);
                const int64_t ctas_on_sm = (grid + sms - 1) / sms;
                const double warps = (double)(ctas_on_sm * gg * p);
                const double per_tile = ((double)ns_max + 0.25) * p;                  // chunks + a charge per warp and tile
                const double stretch = warps < 15.0 ? 15.0 / warps : 1.0;
                // every further group of four columns adds an mma, four FFMA and its fragment loads to the eight lookups
                const int passes = (want_cols + cols - 1) / cols;
                const double cost = (double)passes * (1.0 + 0.2 * (col_groups(cols) - 1)) * (double)(ctas_on_sm * gg * rounds) * per_tile * stretch;
                if (cost < best) { best = cost; sp = {p, gg, sc.slots, sc.ctas, 2, cols}; }
                break;                                                              // the smallest class that fits
            }
        }
    }
    return sp;
}

template <int BITS>
static cudaError_t launch_bits(const GemvArgs &a, int b0, int cols, int grid, int threads, int slots, const LutPlan &L,
                               uint32_t smem, cudaStream_t stream)
{
    const int cg = col_groups(cols);
    if (slots == 2 && threads <= 384 && grid > 148) {
        // a single column with at most 8 warps per CTA: the variant that keeps up two of the four accumulator columns
        // (it needs more than 80 registers to gain from that)
        if (cols == 1 && threads <= 256) return launch_one<BITS, 256, 2, 1, true>(a, b0, cols, grid, threads, L, smem, stream);
        if (cg == 1) return launch_one<BITS, 384, 2, 1, false>(a, b0, cols, grid, threads, L, smem, stream);
        return launch_one<BITS, 384, 2, 2, false>(a, b0, cols, grid, threads, L, smem, stream);
    }
    if (cols == 1 && threads <= 640) return launch_one<BITS, 640, 1, 1, true>(a, b0, cols, grid, threads, L, smem, stream);
    if (threads <= 768) {
        if (cg == 1) return launch_one<BITS, 768, 1, 1, false>(a, b0, cols, grid, threads, L, smem, stream);
        return launch_one<BITS, 768, 1, 2, false>(a, b0, cols, grid, threads, L, smem, stream);
    }
    if (cg == 1) return launch_one<BITS, 1024, 1, 1, false>(a, b0, cols, grid, threads, L, smem, stream);
    return launch_one<BITS, 1024, 1, 2, false>(a, b0, cols, grid, threads, L, smem, stream);
}

// up to eight columns per pass
cudaError_t launch_gemv_lut(const GemvArgs &a, cudaStream_t stream)
{
    const int K = (int)a.K, N = (int)a.N, B = (int)a.B;
    if (a.bits != 2 && a.bits != 3) return cudaErrorInvalidValue;
    if (K > kLutMaxK) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // The tcgen05 kernel runs only where the caller asks for it (test hook): measured, it is the slower of the two
    // (23.7 against 16.3 us on 17408x5120; its header says why).
    if (a.kernel == 2) {
        const int wgs = gemv_lut_tc_warpgroups(a.bits, N, K, B, sms, true);
        if (wgs == 0) return cudaErrorInvalidValue;
        return launch_gemv_lut_tc(a, wgs, stream);
    }
    // batches above 8 on enough rows to give every SM several 16-row tiles: the kernel that walks K slice by slice
    // Batches above 8: one slice-by-slice pass over the weights per 32 columns instead of one pass per 8 columns, where
    // that is faster (measured: from 8192 rows on, and from 4096 rows on for 16 columns and more)
    if ((a.kernel == 3 || (a.kernel == 0 && a.force_P == 0 && B > 8 && (N >= 8192 || (B >= 16 && N >= 4096)))))
        return launch_wide(a, sms, stream);
    const int want_cols = B;                    // the split decides how many of them one pass takes
    Split sp = choose_split(a.bits, N, K, sms, want_cols);
    LutPlan L;
    if (a.force_P > 0 && a.force_G > 0) {
        if (a.force_P * a.force_G > 32 || a.force_G > kMaxGroups) return cudaErrorInvalidValue;
        sp.P = a.force_P; sp.G = a.force_G;
        sp.S = a.force_S > 0 ? a.force_S : 2;
        sp.cols = want_cols < 8 ? want_cols : 8;                 // every instantiation takes two column groups
        sp.slots = sp.ctas = 1;
        for (const SizeClass &sc : kClasses)                     // the smallest size class the forced split fits
            if (sp.P * sp.G <= sc.max_warps && plan_smem(a.bits, K, sp.P, sp.G, sp.S, sp.cols, L) <= sc.smem_cap) {
                sp.slots = sc.slots; sp.ctas = sc.ctas;
                break;
            }
        while (sp.cols > 1 && plan_smem(a.bits, K, sp.P, sp.G, sp.S, sp.cols, L) > kSmemLimit) --sp.cols;
    } else if (a.force_S > 0) {
        sp.S = a.force_S;
    }
    uint32_t smem_cap = kSmemLimit;
    for (const SizeClass &sc : kClasses) if (sc.slots == sp.slots) smem_cap = sc.smem_cap;
    if (plan_smem(a.bits, K, sp.P, sp.G, sp.S, sp.cols, L) > smem_cap) return cudaErrorInvalidValue;
    const int threads = sp.P * sp.G * 32;
    const int64_t need = ((int64_t)N / kLutAtomRows + sp.G - 1) / sp.G;
    const int grid = (int)(need < (int64_t)sms * sp.ctas ? need : (int64_t)sms * sp.ctas);
    L.wait_cycles = a.wait_cycles > 0 ? a.wait_cycles : tc::kWaitBudgetCycles;
    L.drop_first_copy = a.drop_first_copy;
    for (int b0 = 0; b0 < B; b0 += sp.cols) {
        const int cols = (B - b0 < sp.cols) ? (B - b0) : sp.cols;
        // Ask for at least so much shared memory that no more CTAs fit an SM than the split counts on: where a third
        // (second) CTA would fit, the hardware packs three (two) onto some SMs while others hold one, and the launch
        // takes as long as its fullest SM (measured: 17.3 against 12.9 us on 14336x4096 with 256 CTAs of 7 warps).
        uint32_t smem = L.x_off + (uint32_t)cols * L.col_stride;
        if (sp.ctas == 2 && grid > sms && smem < 76u * 1024u) smem = 76u * 1024u;
        const cudaError_t e = (a.bits == 3) ? launch_bits<3>(a, b0, cols, grid, threads, sp.slots, L, smem, stream)
                                            : launch_bits<2>(a, b0, cols, grid, threads, sp.slots, L, smem, stream);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace dq
