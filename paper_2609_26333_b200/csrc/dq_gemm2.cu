// NVFP4 x NVFP4 block-scaled GEMM, CTA-pair version (tcgen05 cta_group::2).
//   Y[m][n] = bf16( s_a * s_w * sum_blk dA[m][blk] dW[n][blk] sum_{k in blk} eA[m][k] eW[n][k] )
// (Sec. 2.3 prefill path; App. A.3 "NVFP4".)
//
// Two CTAs on neighbouring SMs form a cluster and compute one 256 x 256 output
// tile per step: each CTA stages its own 128 rows of A and its own half (128
// rows) of the W tile, so every SM reads half as many W bytes per flop as a lone
// CTA would.  The leader CTA issues the MMAs for the pair; accumulators (128 rows
// x 256 fp32 columns) sit in each CTA's TMEM.
//   warp 0      : TMA producer of this CTA's operand tiles and scale atoms; all loads
//                 signal barriers of the leader (scales and operands separately)
//   warp 1      : (leader) tcgen05.mma; commits release the smem stage in both CTAs and
//                 publish the accumulator to both
//   warps 2, 3  : (leader) tcgen05.cp of the stage's scale atoms into TMEM, one TMEM
//                 scale buffer per smem stage; the two warps take alternate k-steps.  Copies issued from their own thread
//                 run concurrently with the MMAs; issued from the MMA thread they
//                 serialise with them (measured: 490 us vs 240 us on 8192x17408x5120)
//   warps 4..11 : epilogue; TMEM -> registers, TMEM released at once, then scale, bf16
//                 convert, swizzled smem staging and TMA stores overlap the next tile's MMAs
// Every wait is bounded; a wait that runs out sets DQ_ERR_TIMEOUT and all roles
// of both CTAs leave through the common exit.
//
// Gated epilogue (EPI = 1; App. C.1: activation processing fused with the activation quantiser).  For the fused
// gate/up projection of a gated FFN whose weight rows are stored interleaved -- row 256 t + 128 h + 64 p + j holds
// gate (p = 0) or up (p = 1) of feature 128 t + 64 h + j -- every epilogue thread finds gate and up of 64 features
// of its row in its own registers.  It rounds both to bf16 (what the plain epilogue would have stored), forms
// bf16(SiLU(gate) * up), quantises the four 16-blocks to NVFP4 with the next layer's static input scale and writes
// 32 bytes of codes and one 32-bit word of block scales straight into the workspace of the down projection: the
// M x 2F bf16 matrix is neither written nor read back.
#include <cuda.h>

#include "dq_common.cuh"
#include "dq_quant.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

using namespace tc;

constexpr int BM = 128;                       // rows per CTA (pair tile: 256)

// Tile configuration: one 256 x 256 pair tile per step, one CTA per SM, the whole TMEM (256 accumulator columns +
// 5 scale buffers of 48).  (A 256 x 128 configuration with two CTAs of different pairs per SM, meant to hide the
// accumulator hand-off behind the other pair's MMAs, was measured 20 % slower on 8192 x 5120 x 17408 and is not
// kept.)
template <int BN_, int STAGES_, int EPI_WARPS_, int MIN_CTAS_>
struct Cfg {
    static constexpr int BN = BN_;
    static constexpr int kStages = STAGES_;
    static constexpr int kEpiWarps = EPI_WARPS_;
    static constexpr int kMinCtas = MIN_CTAS_;
    static constexpr int kKbPerStage = 4;                 // 64-element MMA k-steps per 256-element stage
    static constexpr int kSfbAtoms = BN / 128;            // 128-row scale atoms of the W tile
    static constexpr uint32_t A_BYTES = BM * 128;         // 16 KiB: 128 rows x 128 B of packed FP4
    static constexpr uint32_t B_BYTES = (BN / 2) * 128;   // this CTA's half of the W tile
    static constexpr uint32_t SFA_BYTES = kKbPerStage * 512;
    static constexpr uint32_t SFB_BYTES = kSfbAtoms * kKbPerStage * 512;
    static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;
    static constexpr uint32_t STG_WARP_BYTES = 32 * 128;                          // 32 rows x 64 bf16, one TMA-store box
    static constexpr uint32_t STG_OFF = kStages * STAGE_BYTES;                    // epilogue staging, 1024-byte aligned
    static constexpr uint32_t BAR_OFF = STG_OFF + kEpiWarps * STG_WARP_BYTES;
    static constexpr uint32_t SMEM_BYTES = BAR_OFF + 1024 + 256;
    static constexpr int kScaleWarps = 2;                          // warps 2 .. 1 + kScaleWarps
    static constexpr int kFirstEpiWarp = 2 + kScaleWarps;
    static constexpr int kThreads = 32 * (kFirstEpiWarp + kEpiWarps);
    static constexpr uint32_t kTmemSfBase = BN;                                   // accumulator: BN fp32 columns
    static constexpr uint32_t kTmemSfACols = 4 * kKbPerStage;
    static constexpr uint32_t kTmemSfBufCols = kTmemSfACols + 4 * kKbPerStage * kSfbAtoms;
    static constexpr uint32_t kTmemCols = (BN + kStages * kTmemSfBufCols) <= 256 ? 256 : 512;
    static_assert(kTmemSfBase + kStages * kTmemSfBufCols <= kTmemCols, "scale buffers must fit in TMEM");
    static_assert(STAGE_BYTES % 1024 == 0, "stages must stay 1024-byte aligned");
    static_assert(kEpiWarps == 4 * (BN / 128), "four epilogue warps (one per TMEM lane quarter) per 128 columns");
    // dense, A/B = E2M1, K-major, UE4M3 scales, N = BN, M = 256 across the pair
    static constexpr uint32_t kInstrDesc = (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
};
using WideCfg = Cfg<256, 5, 8, 1>;

constexpr uint32_t kDescHiSw128 = 64u | (1u << 14) | (2u << 29);   // SBO 1024 B, version 1, 128B swizzle
constexpr uint32_t kDescHiSf = 8u | (1u << 14);                    // SBO 128 B, version 1, no swizzle

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_remote_u32(uint32_t cluster_addr, uint32_t v)
{
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// pair-aware TMA tile load: data lands in this CTA, the transaction bytes are counted on `mbar_cluster`
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap *tmap, int c0, int c1,
                                             uint32_t mbar_cluster)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(mbar_cluster) : "memory");
}
__device__ __forceinline__ void tmem2_cp_sf(uint32_t taddr, uint32_t lo, uint32_t hi)
{
    asm volatile("{\n\t.reg .b64 d;\n\tmov.b64 d, {%1, %2};\n\t"
                 "tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], d;\n\t}" ::"r"(taddr), "r"(lo), "r"(hi) : "memory");
}
template <bool ACC>
__device__ __forceinline__ void mma2_nvf4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t sfa,
                                          uint32_t sfb, uint32_t idesc)
{
    asm volatile("{\n\t.reg .b64 da, db;\n\t.reg .pred p;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "setp.ne.b32 p, %7, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], da, db, %4, [%5], [%6], p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(sfa), "r"(sfb),
                   "r"(ACC ? 1u : 0u) : "memory");
}
// TMA store of one staged box (shared -> global); out-of-range rows / columns are clipped by the hardware
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *tmap, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(tmap), "r"(src), "r"(c0), "r"(c1) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// commit all MMAs issued so far; the arrival goes to the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void mma2_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}

// commit the copies / MMAs issued so far by this thread; arrival on a barrier of this CTA only
__device__ __forceinline__ void mma2_commit_local(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// bounded wait that also raises the partner's abort flag when it gives up
__device__ __forceinline__ bool mbar_wait2(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                           uint32_t peer_abort_addr)
{
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t it = 0;
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if ((++it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitBudgetCycles) {
                *abort_flag = 1;
                st_remote_u32(peer_abort_addr, 1u);
                return false;
            }
        }
    }
}

// pair-tile index -> (256-row block, 256-column block); m fastest inside groups of 8 so that the
// pairs running together share W column blocks and A row blocks in L2
__device__ __forceinline__ void tile_coords2(int t, int tiles_m, int tiles_n, int &mb, int &nb, int GM)
{
    const int per_group = GM * tiles_n;
    const int g = t / per_group;
    const int first_m = g * GM;
    const int gsz = min(GM, tiles_m - first_m);
    const int r = t - g * per_group;
    mb = first_m + r % gsz;
    nb = r / gsz;
}

// what the gated epilogue (EPI = 1) writes instead of Y
struct GatedOut {
    uint8_t *codes;          // [M][F/2] NVFP4 codes of bf16(SiLU(gate) * up)
    uint8_t *sf;             // their block scales in the MMA's layout
    float s;                 // static input scale of the layer that reads them
    int F;                   // features (N = 2F)
};

// MMA_ONLY (measurement): the same roles and barriers, but no operand or scale loads (the barriers are completed by
// hand), no scale copies into TMEM and no stores: what is left is the MMA issue sequence on whatever shared memory
// and TMEM hold, i.e. the tensor-core rate this kernel could reach if nothing else cost time.
template <bool MMA_ONLY, int EPI, class C>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(C::kThreads, C::kMinCtas)
gemm_nvfp4_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                       const __grid_constant__ CUtensorMap tmap_sfa, const __grid_constant__ CUtensorMap tmap_sfw,
                       const __grid_constant__ CUtensorMap tmap_y, const PackedHeader *__restrict__ hdr, float act_scale, __nv_bfloat16 *__restrict__ Y,
                       int64_t ldy, int M, int N, int K, StatusWord *status, int group_m, GatedOut gated)
{
    static_assert(EPI == 0 || C::BN == 256, "the gated epilogue is written for 256-column pair tiles");
    constexpr int BN = C::BN, kStages = C::kStages, kKbPerStage = C::kKbPerStage, kEpiWarps = C::kEpiWarps;
    constexpr int kSfbAtoms = C::kSfbAtoms;
    constexpr uint32_t A_BYTES = C::A_BYTES, B_BYTES = C::B_BYTES, SFA_BYTES = C::SFA_BYTES, SFB_BYTES = C::SFB_BYTES;
    constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES, STG_WARP_BYTES = C::STG_WARP_BYTES, STG_OFF = C::STG_OFF;
    constexpr uint32_t BAR_OFF = C::BAR_OFF, kTmemCols = C::kTmemCols, kTmemSfBase = C::kTmemSfBase;
    constexpr uint32_t kTmemSfBufCols = C::kTmemSfBufCols, kTmemSfACols = C::kTmemSfACols, kInstrDesc = C::kInstrDesc;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + BAR_OFF;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    auto sf_ready_bar = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
    auto sf_full_bar = [&](int s) { return bar_base + 8u * (3 * kStages + s); };
    const uint32_t tmem_full_bar = bar_base + 8u * (4 * kStages);
    const uint32_t tmem_empty_bar = bar_base + 8u * (4 * kStages + 1);
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(smem_gen + BAR_OFF + 8 * (4 * kStages + 2));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_ptr_smem + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t peer_abort = mapa(smem_u32(const_cast<int *>(abort_flag)), rank ^ 1u);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); mbar_init(sf_ready_bar(s), 1); mbar_init(sf_full_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 2 * kEpiWarps);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_ptr_smem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers exist before anyone signals across the pair
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr_smem;
    // Programmatic dependent launch: the set-up above may overlap the tail of the kernel before this one
    // (normally the activation quantiser, whose output this kernel reads); nothing is loaded or stored
    // before that kernel has completed.  A dependent kernel may start its own set-up from here on.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // measurement: the SM clock this launch really runs at (the clock a management query reports between launches is
    // not the clock under this load) -- cycles and global-timer nanoseconds of the first CTA, left in the status word
    long long clk0 = 0, ns0 = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        clk0 = clock64();
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns0));
    }

    const int tiles_m = (M + 2 * BM - 1) / (2 * BM);
    const int tiles_n = (N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int katoms = K / 64;
    const int num_ks = (katoms + kKbPerStage - 1) / kKbPerStage;
    const int pair = blockIdx.x >> 1;
    const int npairs = gridDim.x >> 1;
    const int gm = group_m;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int t = pair; t < num_tiles && ok; t += npairs) {
                int mb, nb;
                tile_coords2(t, tiles_m, tiles_n, mb, nb, gm);
                const int rowblk = mb * 2 + (int)rank;            // 128-row block of A this CTA owns
                for (int ks = 0; ks < num_ks; ++ks) {
                    if (!mbar_wait2(empty_bar(stage), phase ^ 1u, abort_flag, peer_abort)) { ok = false; break; }
                    const uint32_t sA = smem_base + stage * STAGE_BYTES;
                    const uint32_t sB = sA + A_BYTES;
                    const uint32_t sSFA = sB + B_BYTES;
                    const uint32_t sSFB = sSFA + SFA_BYTES;
                    // the small scale atoms go first and have their own barrier, so that their copy
                    // into TMEM overlaps the arrival of the operand tiles
                    const uint32_t leader_full = mapa(full_bar(stage), 0u);
                    const uint32_t leader_sf_full = mapa(sf_full_bar(stage), 0u);
                    if (rank == 0) {
                        mbar_expect_tx(sf_full_bar(stage), 2u * (SFA_BYTES + SFB_BYTES));
                        mbar_expect_tx(full_bar(stage), 2u * (A_BYTES + B_BYTES));
                    }
                    if (!MMA_ONLY) {
                        tma2_load_2d(sSFA, &tmap_sfa, 0, rowblk * katoms + ks * kKbPerStage, leader_sf_full);
#pragma unroll
                        for (int at = 0; at < kSfbAtoms; ++at)
                            tma2_load_2d(sSFB + (uint32_t)at * kKbPerStage * 512, &tmap_sfw, 0,
                                         (kSfbAtoms * nb + at) * katoms + ks * kKbPerStage, leader_sf_full);
                        tma2_load_2d(sA, &tmap_a, ks * 128, rowblk * BM, leader_full);
                        tma2_load_2d(sB, &tmap_w, ks * 128, nb * BN + (int)rank * (BN / 2), leader_full);
                    } else if (rank == 0) {
                        asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(sf_full_bar(stage)),
                                     "r"(2u * (SFA_BYTES + SFB_BYTES)) : "memory");
                        asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(full_bar(stage)),
                                     "r"(2u * (A_BYTES + B_BYTES)) : "memory");
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------- MMA issuer (leader CTA only)
        // The tensor pipe takes an MMA of this size every ~130 cycles, so this thread has about 520 cycles per stage
        // for everything it does, and a barrier probe alone is a round trip to shared memory.  The barriers of the
        // NEXT stage are therefore probed (without blocking) before the MMAs of this stage are issued and the answer
        // is read after them; the bounded blocking wait is only the fallback when the ring is not ahead.
        if (rank == 0 && lane == 0) {
            int stage = 0; uint32_t phase = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            bool seen = false;          // barriers of `stage` already seen complete by the look-ahead probe
            const uint32_t a_lo0 = ((smem_base & 0x3FFFFu) >> 4) | (1u << 16);
            for (int t = pair; t < num_tiles && ok; t += npairs) {
                if (!mbar_wait2(tmem_empty_bar, acc_phase ^ 1u, abort_flag, peer_abort)) { ok = false; break; }
                tc_fence_after();
                for (int ks = 0; ks < num_ks; ++ks) {
                    // operand tiles of this stage are in smem and its scales are in TMEM
                    if (!seen) {
                        if (!mbar_wait2(full_bar(stage), phase, abort_flag, peer_abort)) { ok = false; break; }
                        if (!mbar_wait2(sf_ready_bar(stage), phase, abort_flag, peer_abort)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const int nstage = (stage + 1 == kStages) ? 0 : stage + 1;
                    const uint32_t nphase = (stage + 1 == kStages) ? (phase ^ 1u) : phase;
                    const bool next_full = mbar_test(full_bar(nstage), nphase);
                    const bool next_sf = mbar_test(sf_ready_bar(nstage), nphase);
                    const int nkb = min(kKbPerStage, katoms - ks * kKbPerStage);
                    const uint32_t a_lo = a_lo0 + (uint32_t)stage * (STAGE_BYTES >> 4);
                    const uint32_t b_lo = a_lo + (A_BYTES >> 4);
                    const uint32_t t_sfa = tmem_base + kTmemSfBase + (uint32_t)stage * kTmemSfBufCols;
                    const uint32_t t_sfb = t_sfa + kTmemSfACols;
                    {
                        if (ks == 0) mma2_nvf4<false>(tmem_base, a_lo, b_lo, kDescHiSw128, t_sfa, t_sfb, kInstrDesc);
                        else mma2_nvf4<true>(tmem_base, a_lo, b_lo, kDescHiSw128, t_sfa, t_sfb, kInstrDesc);
#pragma unroll
                        for (int kb = 1; kb < kKbPerStage; ++kb) {
                            if (kb < nkb)
                                mma2_nvf4<true>(tmem_base, a_lo + 2u * kb, b_lo + 2u * kb, kDescHiSw128, t_sfa + 4u * kb,
                                                t_sfb + 4u * kSfbAtoms * kb, kInstrDesc);
                        }
                    }
                    mma2_commit_pair(empty_bar(stage));     // stage (smem and TMEM scales) reusable in both CTAs
                    seen = next_full && next_sf;
                    stage = nstage;
                    phase = nphase;
                }
                if (!ok) break;
                mma2_commit_pair(tmem_full_bar);
                acc_phase ^= 1u;
            }
        }
    } else if (warp < C::kFirstEpiWarp) {
        // ------------------------------- scale copies smem -> TMEM (leader CTA only)
        // One thread can issue only about one copy per 30 ns, and a stage needs 12 of them plus the
        // barrier round trips, which is more than the 0.4 us its MMAs take; so two threads take
        // alternate stages (warp 2 the even k-steps, warp 3 the odd ones).
        if (rank == 0 && lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            const uint32_t sf_lo0 = ((smem_base + A_BYTES + B_BYTES) & 0x3FFFFu) >> 4;
            uint32_t step = 0;
            for (int t = pair; t < num_tiles && ok; t += npairs) {
                for (int ks = 0; ks < num_ks; ++ks, ++step) {
                    if (step % (uint32_t)C::kScaleWarps == (uint32_t)(warp - 2)) {
                        if (!mbar_wait2(sf_full_bar(stage), phase, abort_flag, peer_abort)) { ok = false; break; }
                        tc_fence_after();
                        const int nkb = min(kKbPerStage, katoms - ks * kKbPerStage);
                        const uint32_t sfa_lo = sf_lo0 + (uint32_t)stage * (STAGE_BYTES >> 4);
                        const uint32_t sfb_lo = sfa_lo + (SFA_BYTES >> 4);
                        const uint32_t t_sfa = tmem_base + kTmemSfBase + (uint32_t)stage * kTmemSfBufCols;
                        const uint32_t t_sfb = t_sfa + kTmemSfACols;
                        if (!MMA_ONLY) {
#pragma unroll
                            for (int kb = 0; kb < kKbPerStage; ++kb) {
                                if (kb < nkb) {
                                    tmem2_cp_sf(t_sfa + 4u * kb, sfa_lo + 32u * kb, kDescHiSf);
#pragma unroll
                                    for (int at = 0; at < kSfbAtoms; ++at)
                                        tmem2_cp_sf(t_sfb + 4u * kSfbAtoms * kb + 4u * at,
                                                    sfb_lo + (uint32_t)at * (kKbPerStage * 512u >> 4) + 32u * kb, kDescHiSf);
                                }
                            }
                        }
                        mma2_commit_local(sf_ready_bar(stage));    // arrives once the copies have landed in both CTAs
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int ew = warp - C::kFirstEpiWarp;
        const int wq = warp & 3;                            // TMEM lane quarter this warp may read
        const int half = ew >> 2;                           // which 128 accumulator columns
        const float alpha = __fmul_rn(act_scale, hdr->s);
        const uint32_t leader_tmem_empty = mapa(tmem_empty_bar, 0u);
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int t = pair; t < num_tiles && ok; t += npairs) {
            int mb, nb;
            tile_coords2(t, tiles_m, tiles_n, mb, nb, gm);
            if (!mbar_wait2(tmem_full_bar, acc_phase, abort_flag, peer_abort)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16) + (uint32_t)(half * 128);
            // bf16 rows go through a swizzled staging box (32 rows x 64 columns per warp) and leave with
            // a TMA store, so that global memory sees full 128-byte lines instead of 16-byte pieces
            const int row0 = (mb * 2 + (int)rank) * BM + wq * 32;
            const int col0 = nb * BN + half * 128;
            const uint32_t stg = smem_base + STG_OFF + (uint32_t)ew * STG_WARP_BYTES;
            const uint32_t my_row = stg + (uint32_t)lane * 128u;
            const uint32_t sw = (uint32_t)(lane & 7);
            auto stage_box = [&](const uint32_t (&lo)[32], const uint32_t (&hi)[32], int box) {
                if (MMA_ONLY) return;
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // buffer free again
                __syncwarp();
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t (&v)[32] = (c < 4) ? lo : hi;
                    const int o = (c & 3) * 8;
                    sts_v4(my_row + (((uint32_t)c ^ sw) << 4),
                           pack_bf16x2(__uint_as_float(v[o + 0]) * alpha, __uint_as_float(v[o + 1]) * alpha),
                           pack_bf16x2(__uint_as_float(v[o + 2]) * alpha, __uint_as_float(v[o + 3]) * alpha),
                           pack_bf16x2(__uint_as_float(v[o + 4]) * alpha, __uint_as_float(v[o + 5]) * alpha),
                           pack_bf16x2(__uint_as_float(v[o + 6]) * alpha, __uint_as_float(v[o + 7]) * alpha));
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && row0 < M && col0 + box * 64 < N) tma_store_2d(&tmap_y, stg, col0 + box * 64, row0);
            };
            auto release_tmem = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(leader_tmem_empty);
            };
            // the whole 128-column slice at once, TMEM handed back before converting and storing
            uint32_t v0[32], v1[32], v2[32], v3[32];
            tmem_ld32(taddr, v0);
            tmem_ld32(taddr + 32u, v1);
            tmem_ld32(taddr + 64u, v2);
            tmem_ld32(taddr + 96u, v3);
            tmem_ld_wait();
            release_tmem();
            if (EPI == 0) {
                stage_box(v0, v1, 0);
                stage_box(v2, v3, 1);
            } else if (!MMA_ONLY) {
                // columns 0..63 of this warp's slice: gate, 64..127: up, of features f0 .. f0 + 63 of row `row`
                const int row = row0 + lane;
                const int f0 = nb * (BN / 2) + half * 64;
                const float rc6 = __frcp_rn(__fmul_rn(6.0f, gated.s));
                // G and U as the plain epilogue would have stored them, as packed bf16 pairs
                uint32_t g2[4][8], u2[4][8];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    g2[i >> 3][i & 7] = pack_bf16x2(__uint_as_float(v0[2 * i]) * alpha, __uint_as_float(v0[2 * i + 1]) * alpha);
                    g2[2 + (i >> 3)][i & 7] = pack_bf16x2(__uint_as_float(v1[2 * i]) * alpha, __uint_as_float(v1[2 * i + 1]) * alpha);
                    u2[i >> 3][i & 7] = pack_bf16x2(__uint_as_float(v2[2 * i]) * alpha, __uint_as_float(v2[2 * i + 1]) * alpha);
                    u2[2 + (i >> 3)][i & 7] = pack_bf16x2(__uint_as_float(v3[2 * i]) * alpha, __uint_as_float(v3[2 * i + 1]) * alpha);
                }
                uint32_t cw[8];
                uint32_t sfw = 0;
#pragma unroll
                for (int blk = 0; blk < 4; ++blk) {
                    uint32_t h[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) h[i] = silu_mul_bf16x2(g2[blk][i], u2[blk][i]);
                    uint2 c;
                    sfw |= quant_block_nvfp4_bf16(h, gated.s, rc6, c) << (8 * blk);
                    cw[2 * blk] = c.x;
                    cw[2 * blk + 1] = c.y;
                }
                if (row < M && f0 < gated.F) {
                    uint4 *dst = reinterpret_cast<uint4 *>(gated.codes + ((int64_t)row * (gated.F >> 4) + (f0 >> 4)) * 8);
                    dst[0] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
                    dst[1] = make_uint4(cw[4], cw[5], cw[6], cw[7]);
                    const int rr = row & 127;
                    const size_t off = ((size_t)(row >> 7) * (size_t)(gated.F >> 6) + (size_t)(f0 >> 6)) * 512 +
                                       (size_t)((rr & 31) * 16 + (rr >> 5) * 4);
                    *reinterpret_cast<uint32_t *>(gated.sf + off) = sfw;
                }
            }
            acc_phase ^= 1u;
        }
        if (EPI == 0 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores of this warp done
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        long long ns1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns1));
        status->gemm_cycles = (unsigned long long)(clock64() - clk0);
        status->gemm_ns = (unsigned long long)(ns1 - ns0);
    }
    cluster_sync_all();            // nobody leaves while the partner may still signal its barriers
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);       // let copies in flight land
        if (threadIdx.x == 0) {
            atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
            atomicExch(&status->detail, 0x20000 | (int)blockIdx.x);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool make_codes_tmap2(EncodeTiledFn enc, CUtensorMap *tm, const void *ptr, int64_t rows, int64_t K, uint32_t box_rows)
{
    cuuint64_t gdim[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)(K / 2)};
    cuuint32_t box[2] = {128u, box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// scale atoms as a matrix of 512-byte rows (128 x uint32); box = 4 consecutive k atoms
bool make_sf_tmap(EncodeTiledFn enc, CUtensorMap *tm, const void *ptr, int64_t atoms)
{
    cuuint64_t gdim[2] = {128u, (cuuint64_t)atoms};
    cuuint64_t gstride[1] = {512u};
    cuuint32_t box[2] = {128u, (cuuint32_t)4u};
    cuuint32_t estr[2] = {1u, 1u};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(ptr), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 output matrix [M][N] with row stride ldy; box = 64 columns x 32 rows, 128B swizzle
bool make_y_tmap(EncodeTiledFn enc, CUtensorMap *tm, void *ptr, int64_t M, int64_t N, int64_t ldy)
{
    cuuint64_t gdim[2] = {(cuuint64_t)N, (cuuint64_t)M};
    cuuint64_t gstride[1] = {(cuuint64_t)ldy * 2u};
    cuuint32_t box[2] = {64u, 32u};
    cuuint32_t estr[2] = {1u, 1u};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

template <class C>
static cudaError_t launch_pair_cfg(const GemmArgs &a, EncodeTiledFn enc, cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemm_nvfp4_pair_kernel<false, 0, C>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             C::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(gemm_nvfp4_pair_kernel<true, 0, C>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(gemm_nvfp4_pair_kernel<false, 1, C>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    constexpr int BN = C::BN;
    const int64_t katoms = a.K / 64;
    CUtensorMap tmap_a, tmap_w, tmap_sfa, tmap_sfw, tmap_y;
    if (!make_codes_tmap2(enc, &tmap_a, a.a_codes, a.M, a.K, BM)) return cudaErrorInvalidValue;
    if (!make_codes_tmap2(enc, &tmap_w, a.w_codes, a.N, a.K, BN / 2)) return cudaErrorInvalidValue;
    if (!make_sf_tmap(enc, &tmap_sfa, a.a_sf, ((a.M + 127) / 128) * katoms)) return cudaErrorInvalidValue;
    if (!make_sf_tmap(enc, &tmap_sfw, a.w_sf, ((a.N + 255) / 256) * 2 * katoms)) return cudaErrorInvalidValue;
    // the gated epilogue stores with plain instructions: its output map is never used, any valid map will do
    const bool gated = a.gated_codes != nullptr;
    if (gated) tmap_y = tmap_a;
    else if (!make_y_tmap(enc, &tmap_y, a.Y, a.M, a.N, a.ldy)) return cudaErrorInvalidValue;
    GatedOut go = {a.gated_codes, a.gated_sf, a.gated_scale, (int)(a.N / 2)};
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int tiles = (int)(((a.M + 2 * BM - 1) / (2 * BM)) * ((a.N + BN - 1) / BN));
    int pairs = sms / 2 * C::kMinCtas;
    if (tiles < pairs) pairs = tiles;
    // Tile order: groups of group_m row tiles sweep all column tiles, so that the A rows of a group stay in L2
    // while each W tile is read once per group.  Largest power of two whose A codes + scales fit about 48 MB.
    int group_m = 4;
    while (group_m < 64 && (double)(2 * group_m) * 256.0 * (double)a.K * 0.5625 <= 48.0e6) group_m *= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3((unsigned)C::kThreads);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (gated)
        return cudaLaunchKernelEx(&cfg, gemm_nvfp4_pair_kernel<false, 1, C>, tmap_a, tmap_w, tmap_sfa, tmap_sfw, tmap_y, a.hdr,
                                  a.act_scale, reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.M,
                                  (int)a.N, (int)a.K, a.status, group_m, go);
    if (a.mma_only)
        return cudaLaunchKernelEx(&cfg, gemm_nvfp4_pair_kernel<true, 0, C>, tmap_a, tmap_w, tmap_sfa, tmap_sfw, tmap_y, a.hdr,
                                  a.act_scale, reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.M,
                                  (int)a.N, (int)a.K, a.status, group_m, go);
    return cudaLaunchKernelEx(&cfg, gemm_nvfp4_pair_kernel<false, 0, C>, tmap_a, tmap_w, tmap_sfa, tmap_sfw, tmap_y, a.hdr,
                              a.act_scale, reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.M, (int)a.N,
                              (int)a.K, a.status, group_m, go);
}

}  // namespace

cudaError_t launch_gemm_nvfp4_pair(const GemmArgs &a, void *encode_fn, cudaStream_t stream)
{
    return launch_pair_cfg<WideCfg>(a, reinterpret_cast<EncodeTiledFn>(encode_fn), stream);
}

}  // namespace dq
