// NVFP4 x NVFP4 block-scaled GEMM for the prefill path on sm_100a (Sec. 2.3;
// App. A.3 "NVFP4": E2M1 values, 16-element blocks, E4M3 block scales, FP32
// tensor scales):
//   Y[m][n] = bf16( s_a * s_w * sum_blk dA[m][blk] dW[n][blk] sum_{k in blk} eA[m][k] eW[n][k] )
//
// One persistent CTA per SM, 128 x 256 output tiles, 256-element k-steps.
//   warp 0      : TMA producer (packed FP4 tiles, 128B swizzle) + bulk copies of the scale atoms
//   warp 1      : tcgen05.cp of the scales into TMEM and tcgen05.mma (kind::mxf4nvf4, block 16)
//   warps 2..5  : epilogue, TMEM -> registers -> bf16 -> global
// The fp32 accumulator lives in TMEM (256 columns); the per-stage scale factors
// occupy 2 x 48 further columns.  Every mbarrier wait is bounded: when it runs
// out the CTA records DQ_ERR_TIMEOUT in the status word and leaves normally.
#include <cuda.h>

#include "dq_common.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 256;                       // elements; 128 bytes of packed FP4 = one swizzle row
constexpr int kStages = 4;
constexpr int kKbPerStage = BK / 64;          // MMA k-steps (64 elements) per stage
constexpr uint32_t A_STAGE_BYTES = BM * 128;  // 16 KiB
constexpr uint32_t B_STAGE_BYTES = BN * 128;  // 32 KiB
constexpr uint32_t SFA_STAGE_BYTES = kKbPerStage * 512;
constexpr uint32_t SFB_STAGE_BYTES = 2 * kKbPerStage * 512;
constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES + SFA_STAGE_BYTES + SFB_STAGE_BYTES;
constexpr uint32_t SMEM_BYTES = kStages * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemSfBase = 256;         // accumulator uses columns [0, 256)
constexpr uint32_t kTmemSfBufCols = 48;       // 16 (A) + 32 (B) per stage, double buffered

static_assert(STAGE_BYTES % 1024 == 0, "stage must keep 1024-byte alignment for the 128B swizzle");

// instruction descriptor: dense, A/B = E2M1 (kind::mxf4nvf4), both K-major, scale type UE4M3,
// N >> 3 at bit 17, M >> 4 at bit 24, scale-factor ids 0, K = 64
constexpr uint32_t kInstrDesc = (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

using namespace tc;

// tile index -> (m block, n block): m fastest inside groups of 16 m-blocks so that
// the CTAs running at the same time share A row-blocks and W column-blocks in L2
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int &mb, int &nb)
{
    constexpr int GM = 16;
    const int per_group = GM * tiles_n;
    const int g = t / per_group;
    const int first_m = g * GM;
    const int gsz = min(GM, tiles_m - first_m);
    const int r = t - g * per_group;
    mb = first_m + r % gsz;
    nb = r / gsz;
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_nvfp4_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                  const uint8_t *__restrict__ a_sf, const uint8_t *__restrict__ w_sf,
                  const PackedHeader *__restrict__ hdr, float act_scale, __nv_bfloat16 *__restrict__ Y, int64_t ldy,
                  int M, int N, int K, StatusWord *status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    // per stage: [A 16K][B 32K][SFA 2K][SFB 4K]
    const uint32_t bar_base = smem_base + kStages * STAGE_BYTES;
    // barriers: full[kStages], empty[kStages], tmem_full, tmem_empty ; then tmem ptr, abort flag
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    const uint32_t tmem_full_bar = bar_base + 8u * (2 * kStages);
    const uint32_t tmem_empty_bar = bar_base + 8u * (2 * kStages + 1);
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(smem_gen + kStages * STAGE_BYTES + 8 * (2 * kStages + 2));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_ptr_smem + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_ptr_smem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr_smem;

    const int tiles_m = (M + BM - 1) / BM;
    const int tiles_n = (N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int katoms = K / 64;                                // 64-element k atoms in K
    const int num_ks = (katoms + kKbPerStage - 1) / kKbPerStage;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                int mb, nb;
                tile_coords(t, tiles_m, tiles_n, mb, nb);
                for (int ks = 0; ks < num_ks; ++ks) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const int nkb = min(kKbPerStage, katoms - ks * kKbPerStage);
                    const uint32_t sA = smem_base + stage * STAGE_BYTES;
                    const uint32_t sB = sA + A_STAGE_BYTES;
                    const uint32_t sSFA = sB + B_STAGE_BYTES;
                    const uint32_t sSFB = sSFA + SFA_STAGE_BYTES;
                    const uint32_t sf_bytes = (uint32_t)nkb * 512u;
                    mbar_expect_tx(full_bar(stage), A_STAGE_BYTES + B_STAGE_BYTES + 3u * sf_bytes);
                    tma_load_2d(sA, &tmap_a, ks * 128, mb * BM, full_bar(stage));
                    tma_load_2d(sB, &tmap_w, ks * 128, nb * BN, full_bar(stage));
                    const size_t koff = (size_t)ks * kKbPerStage * 512;
                    bulk_load(sSFA, a_sf + ((size_t)mb * katoms) * 512 + koff, sf_bytes, full_bar(stage));
                    bulk_load(sSFB, w_sf + ((size_t)(2 * nb) * katoms) * 512 + koff, sf_bytes, full_bar(stage));
                    bulk_load(sSFB + kKbPerStage * 512, w_sf + ((size_t)(2 * nb + 1) * katoms) * 512 + koff, sf_bytes,
                              full_bar(stage));
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            uint32_t acc_phase = 0;
            uint32_t sfbuf = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                if (!mbar_wait(tmem_empty_bar, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                for (int ks = 0; ks < num_ks; ++ks) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const int nkb = min(kKbPerStage, katoms - ks * kKbPerStage);
                    const uint32_t sA = smem_base + stage * STAGE_BYTES;
                    const uint32_t sB = sA + A_STAGE_BYTES;
                    const uint32_t sSFA = sB + B_STAGE_BYTES;
                    const uint32_t sSFB = sSFA + SFA_STAGE_BYTES;
                    const uint32_t t_sfa = tmem_base + kTmemSfBase + sfbuf * kTmemSfBufCols;
                    const uint32_t t_sfb = t_sfa + 16u;
                    for (int kb = 0; kb < nkb; ++kb) {
                        tmem_cp_sf(t_sfa + 4u * kb, make_desc_sf(sSFA + 512u * kb));
                        tmem_cp_sf(t_sfb + 8u * kb, make_desc_sf(sSFB + 512u * kb));
                        tmem_cp_sf(t_sfb + 8u * kb + 4u, make_desc_sf(sSFB + kKbPerStage * 512u + 512u * kb));
                    }
                    const uint64_t adesc = make_desc_sw128(sA);
                    const uint64_t bdesc = make_desc_sw128(sB);
                    for (int kb = 0; kb < nkb; ++kb) {
                        // one k-step is 64 elements = 32 bytes inside the 128-byte swizzle row
                        mma_nvf4(tmem_base, adesc + 2ull * kb, bdesc + 2ull * kb, kInstrDesc, t_sfa + 4u * kb,
                                 t_sfb + 8u * kb, (ks > 0 || kb > 0) ? 1u : 0u);
                    }
                    mma_commit(empty_bar(stage));          // frees the stage once these MMAs have read it
                    sfbuf ^= 1u;
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                mma_commit(tmem_full_bar);                 // accumulator complete
                acc_phase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int wq = warp & 3;                           // TMEM lane quarter this warp may read
        const float alpha = __fmul_rn(act_scale, hdr->s);
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
            int mb, nb;
            tile_coords(t, tiles_m, tiles_n, mb, nb);
            if (!mbar_wait(tmem_full_bar, acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const int row = mb * BM + wq * 32 + lane;
            __nv_bfloat16 *yrow = Y + (int64_t)row * ldy + (int64_t)nb * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(wq * 32) << 16) + (uint32_t)(c * 32), v);
                tmem_ld_wait();
                if (row < M) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int col = nb * BN + c * 32 + q * 8;
                        if (col < N) {
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(v[8 * q + 0]) * alpha, __uint_as_float(v[8 * q + 1]) * alpha);
                            o.y = pack_bf16x2(__uint_as_float(v[8 * q + 2]) * alpha, __uint_as_float(v[8 * q + 3]) * alpha);
                            o.z = pack_bf16x2(__uint_as_float(v[8 * q + 4]) * alpha, __uint_as_float(v[8 * q + 5]) * alpha);
                            o.w = pack_bf16x2(__uint_as_float(v[8 * q + 6]) * alpha, __uint_as_float(v[8 * q + 7]) * alpha);
                            *reinterpret_cast<uint4 *>(yrow + c * 32 + q * 8) = o;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tmem_empty_bar);
            acc_phase ^= 1u;
        }
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait ran out: give copies in flight time to land, then report
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        if (threadIdx.x == 0) {
            atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
            atomicExch(&status->detail, (int)blockIdx.x);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// packed FP4 codes as a byte matrix [rows][K/2]; box = 128 bytes x box_rows, 128B swizzle, zero fill outside
bool make_codes_tmap(CUtensorMap *tm, const void *ptr, int64_t rows, int64_t K, uint32_t box_rows)
{
    cuuint64_t gdim[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)(K / 2)};
    cuuint32_t box[2] = {128u, box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace

int gemm_init_driver_api()
{
    if (g_encode) return 0;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || fn == nullptr) return 1;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return 0;
}

cudaError_t launch_gemm_nvfp4(const GemmArgs &a, cudaStream_t stream)
{
    if (gemm_init_driver_api() != 0) return cudaErrorNotSupported;
    // more than one 128-row block: CTA pairs share the W tile; otherwise a lone CTA per tile
    // (the gated epilogue exists in the pair kernel only)
    if (a.M > BM || a.gated_codes) return launch_gemm_nvfp4_pair(a, reinterpret_cast<void *>(g_encode), stream);
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemm_nvfp4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    CUtensorMap tmap_a, tmap_w;
    if (!make_codes_tmap(&tmap_a, a.a_codes, a.M, a.K, BM)) return cudaErrorInvalidValue;
    if (!make_codes_tmap(&tmap_w, a.w_codes, a.N, a.K, BN)) return cudaErrorInvalidValue;
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int tiles = (int)(((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN));
    const int grid = tiles < sms ? tiles : sms;
    gemm_nvfp4_kernel<<<grid, kThreads, SMEM_BYTES, stream>>>(tmap_a, tmap_w, a.a_sf, a.w_sf, a.hdr, a.act_scale,
                                                             reinterpret_cast<__nv_bfloat16 *>(a.Y), a.ldy, (int)a.M,
                                                             (int)a.N, (int)a.K, a.status);
    return cudaGetLastError();
}

}  // namespace dq
