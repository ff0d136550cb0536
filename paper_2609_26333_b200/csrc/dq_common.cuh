// Shared declarations of the CUDA side: packed-buffer layout, device header,
// launcher prototypes.  Nothing here is shared with the CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/dq.h"

namespace dq {

constexpr int kBlock = 16;            // weights per block scale (App. A.3)
constexpr int kSfAtomRows = 128;      // rows of one scale-factor atom of the block-scaled MMA
constexpr int kSfAtomBytes = 512;     // 128 rows x 4 scales (64 k)
constexpr int kSfRowPad = 256;        // NVFP4 scale tiles padded to the GEMM's N tile
constexpr int kLutChunk = 128;        // weights per LUT3 device chunk (3 planes x 4 words)

// Device header at the start of the packed buffer (1 KiB reserved).
struct PackedHeader {
    unsigned int amax_bits;       // max|W| as fp32 bits (non-negative floats order like uints)
    float s;                      // tensor scale  s = max|W| / (6*448)
    float rc6;                    // 1 / (6 s)
    float pad0;
    float lut_levels[8];          // codebook as fp32
    float lut_thresholds[8];      // midpoints between consecutive levels (7 used)
    unsigned int lut_f16[8];      // codebook fp16 bit patterns
    int lut_zero_idx;
    unsigned int autocast_map;    // 8 nibbles: E2M1 code of each level
};
constexpr size_t kHeaderBytes = 1024;

struct PackedLayout {
    size_t nv_codes_off = 0, nv_codes_bytes = 0;     // uint8[N][K/2]
    size_t nv_sf_off = 0, nv_sf_bytes = 0;           // [ceil(N/256)*2][K/64][512] MMA scale layout
    size_t lut_planes_off = 0, lut_planes_bytes = 0; // uint32[N][K/128][3][4]
    size_t lut_sf_off = 0, lut_sf_bytes = 0;         // uint8[N][K/16] signed E4M3
    size_t total = 0;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline PackedLayout packed_layout(int64_t N, int64_t K, unsigned formats)
{
    PackedLayout L;
    size_t off = kHeaderBytes;
    if (formats & (DQ_FMT_NVFP4 | DQ_FMT_NVFP4_FROM_LUT3)) {
        L.nv_codes_off = off;
        L.nv_codes_bytes = (size_t)N * K / 2;
        off = align_up(off + L.nv_codes_bytes, 1024);
        L.nv_sf_off = off;
        L.nv_sf_bytes = align_up((size_t)N, kSfRowPad) * (size_t)(K / kBlock);
        off = align_up(off + L.nv_sf_bytes, 1024);
    }
    if (formats & (DQ_FMT_LUT3 | DQ_FMT_NVFP4_FROM_LUT3)) {
        L.lut_planes_off = off;
        L.lut_planes_bytes = (size_t)N * K / 8 * 3;
        off = align_up(off + L.lut_planes_bytes, 1024);
        L.lut_sf_off = off;
        L.lut_sf_bytes = (size_t)N * (K / kBlock);
        off = align_up(off + L.lut_sf_bytes, 1024);
    }
    L.total = off;
    return L;
}

// Byte offset of block scale (row r, 16-block b) inside the MMA scale layout:
// atoms of 128 rows x 4 scales, K-atoms fastest, then 128-row groups.
__host__ __device__ inline size_t sf_swizzled_offset(int64_t r, int64_t b, int64_t K)
{
    int64_t katoms = K / 64;
    int64_t atom = (r / 128) * katoms + (b / 4);
    int64_t rr = r % 128;
    return (size_t)atom * 512 + (size_t)(rr % 32) * 16 + (size_t)(rr / 32) * 4 + (size_t)(b % 4);
}

// Device status word: [0] = dq_status, [1] = detail.
struct StatusWord { int status; int detail; };

// ---- launchers (each enqueues on `stream`, returns a cudaError_t) ----
cudaError_t launch_pack_header(PackedHeader *hdr, const uint16_t *codebook_f16_host, cudaStream_t stream);
cudaError_t launch_absmax(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw, PackedHeader *hdr,
                          cudaStream_t stream);
cudaError_t launch_pack_nvfp4(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                              const PackedHeader *hdr, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream);
cudaError_t launch_pack_lut3(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                             const PackedHeader *hdr, uint32_t *planes_dev, uint8_t *lut_sf, cudaStream_t stream);
cudaError_t launch_autocast(const PackedHeader *hdr, const uint32_t *planes_dev, const uint8_t *lut_sf, int64_t N,
                            int64_t K, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream);
cudaError_t launch_export_nvfp4(const PackedHeader *hdr, const uint8_t *codes, const uint8_t *sf_swizzled, int64_t N,
                                int64_t K, uint8_t *codes_out, uint8_t *scales_out, float *s_out,
                                cudaStream_t stream);
cudaError_t launch_export_lut3(const PackedHeader *hdr, const uint32_t *planes_dev, const uint8_t *lut_sf, int64_t N,
                               int64_t K, uint32_t *planes_out, uint8_t *scales_out, float *s_out,
                               cudaStream_t stream);
// Activation quantiser: codes row-major [M][K/2]; scales either in the MMA layout
// (swizzled != 0) or canonical [M][K/16].
cudaError_t launch_quant_act(const void *A_bf16, int64_t M, int64_t K, int64_t lda, float act_scale, uint8_t *codes,
                             uint8_t *sf, int swizzled, cudaStream_t stream);

struct GemmArgs {
    const uint8_t *a_codes;  const uint8_t *a_sf;      // activations: [M][K/2], MMA scale layout
    const uint8_t *w_codes;  const uint8_t *w_sf;      // weights:     [N][K/2], MMA scale layout
    const PackedHeader *hdr;                           // tensor scale of the weights
    float act_scale;
    void *Y; int64_t ldy;
    int64_t M, N, K;
    StatusWord *status;
    int probe = 0;   // timing probes: 1 = no MMA, 2 = no loads, 4 = no scale copies (results are meaningless), 8 = force the 1-CTA kernel
};
cudaError_t launch_gemm_nvfp4(const GemmArgs &args, cudaStream_t stream);
cudaError_t launch_gemm_nvfp4_pair(const GemmArgs &args, void *encode_fn, cudaStream_t stream);
int gemm_init_driver_api();   // resolves the tensor-map encoder; 0 on success

struct GemvArgs {
    const uint32_t *planes; const uint8_t *sf; const PackedHeader *hdr;
    const void *X; int64_t ldx; int64_t B;
    void *Y; int64_t ldy;
    int64_t N, K;
};
cudaError_t launch_gemv_lut3(const GemvArgs &args, cudaStream_t stream);

}  // namespace dq
