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
constexpr size_t kLutTableBytes = 65536;   // 256 entries x 32 lane slots x (fp32, fp32): the decode kernel's shared-memory table

// LUT3 device layout: the weights of one row are cut into slices of 1024 (one per warp of the
// decode kernel); slice s of row r is one block of 448 bytes:
//   [word 0 of 32 triplets][word 1 of 32 triplets][word 2 of 32 triplets][scales: 64 signed E4M3 bytes]
// i.e. 3 index words + 2 scale bytes per 32 weights, 3.5 bit per weight (bit order: lut3_locate below).  A partial last slice is
// zero padded (zero scales, so the padding contributes nothing).
constexpr int kLutSlice = 1024;
constexpr int kLutBlockBytes = 448;
constexpr int kLutScaleOff = 384;
__host__ __device__ inline int64_t lut_slices(int64_t K) { return (K + kLutSlice - 1) / kLutSlice; }
// word p (0..2) of triplet j (32 weights) in row r; K/32 triplets per row
__host__ __device__ inline size_t lut_word_offset(int64_t r, int64_t j, int p, int64_t K)
{
    return (size_t)(r * lut_slices(K) + j / 32) * kLutBlockBytes + (size_t)p * 128 + (size_t)(j % 32) * 4;
}
// scale of 16-block b in row r
__host__ __device__ inline size_t lut_scale_offset(int64_t r, int64_t b, int64_t K)
{
    return (size_t)(r * lut_slices(K) + b / 64) * kLutBlockBytes + kLutScaleOff + (size_t)(b % 64);
}

struct PackedLayout {
    size_t nv_codes_off = 0, nv_codes_bytes = 0;     // uint8[N][K/2]
    size_t nv_sf_off = 0, nv_sf_bytes = 0;           // [ceil(N/256)*2][K/64][512] MMA scale layout
    size_t lut_table_off = 0;                        // 64 KiB decode lookup table (level pairs, one slot per lane)
    size_t lut_off = 0, lut_bytes = 0;               // [N][ceil(K/1024)] blocks of kLutBlockBytes (see below)
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
        L.lut_table_off = off;
        off += kLutTableBytes;
        L.lut_off = off;
        L.lut_bytes = (size_t)N * lut_slices(K) * kLutBlockBytes;
        off = align_up(off + L.lut_bytes, 1024);
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

// LUT3 device bit order.  Storage stays three 32-bit words per 32 weights (3 bit per weight), in the three
// 128-byte "plane" regions of a block, but the words are not bit-planes: words 0, 1, 2 hold the indices of
// weights 0-7, 8-15, 16-23 as nibbles (weight 8a + n in bits 4n .. 4n+2 of word a), and the spare top bit of
// the eight nibbles of word b holds bit b of the indices of weights 24-31 (weight 24 + n in bit 4n + 3).
// A decode kernel gets byte-permute selectors / pair indices for 24 weights with one AND per word and for the
// last eight with three shifts and three bitwise ops.  The canonical (export) layout is the bit-plane form.
__host__ __device__ inline void lut3_locate(int bit, int i, int &word, int &pos)
{
    if (i < 24) { word = i >> 3; pos = 4 * (i & 7) + bit; }
    else { word = bit; pos = 4 * (i - 24) + 3; }
}
// the four selector words of a word triplet: nibble n of word a is the index of weight 8a + n
__device__ __forceinline__ void lut3_selectors(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t (&sel)[4])
{
    sel[0] = w0 & 0x77777777u;
    sel[1] = w1 & 0x77777777u;
    sel[2] = w2 & 0x77777777u;
    sel[3] = ((w0 >> 3) & 0x11111111u) | ((w1 >> 2) & 0x22222222u) | ((w2 >> 1) & 0x44444444u);
}

// Device status word: [0] = dq_status, [1] = detail.
struct StatusWord { int status; int detail; };

// ---- launchers (each enqueues on `stream`, returns a cudaError_t) ----
cudaError_t launch_pack_header(PackedHeader *hdr, const uint16_t *codebook_f16_host, cudaStream_t stream);
cudaError_t launch_absmax(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw, PackedHeader *hdr,
                          cudaStream_t stream);
cudaError_t launch_pack_nvfp4(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                              const PackedHeader *hdr, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream);
cudaError_t launch_build_lut_table(const PackedHeader *hdr, uint8_t *table_dev, cudaStream_t stream);
cudaError_t launch_pack_lut3(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                             const PackedHeader *hdr, uint8_t *lut_dev, cudaStream_t stream);
cudaError_t launch_autocast(const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                            int64_t K, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream);
cudaError_t launch_export_nvfp4(const PackedHeader *hdr, const uint8_t *codes, const uint8_t *sf_swizzled, int64_t N,
                                int64_t K, uint8_t *codes_out, uint8_t *scales_out, float *s_out,
                                cudaStream_t stream);
cudaError_t launch_export_lut3(const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                               int64_t K, uint32_t *planes_out, uint8_t *scales_out, float *s_out,
                               cudaStream_t stream);
cudaError_t launch_pack_done(cudaStream_t stream);
cudaError_t launch_set_scale(PackedHeader *hdr, float s, cudaStream_t stream);
cudaError_t launch_import_nvfp4(const uint8_t *codes_in, const uint8_t *scales_in, int64_t N, int64_t K, uint8_t *codes,
                                uint8_t *sf_swizzled, cudaStream_t stream);
cudaError_t launch_import_lut3(const uint32_t *planes_in, const uint8_t *scales_in, int64_t N, int64_t K,
                               uint8_t *lut_dev, cudaStream_t stream);
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
    const uint8_t *lut; const PackedHeader *hdr;          // LUT3 blocks (planes + scales)
    const uint8_t *table = nullptr;                      // prebuilt 64 KiB pair table
    StatusWord *status = nullptr;
    const void *X; int64_t ldx; int64_t B;
    void *Y; int64_t ldy;
    int64_t N, K;
};
cudaError_t launch_gemv_lut3(const GemvArgs &args, cudaStream_t stream);              // CUDA cores: batch 1 and 2
cudaError_t launch_gemv_lut3_mma(const GemvArgs &args, cudaStream_t stream);          // tensor cores: eight columns per pass
bool gemv_lut3_mma_preferred(int64_t N, int64_t K, int64_t B);                          // which of the two dq_decode_linear takes

struct GemvNvArgs {
    const uint8_t *codes; const uint8_t *sf;              // NVFP4 view: [N][K/2] codes, MMA-layout scales
    const PackedHeader *hdr;
    StatusWord *status = nullptr;
    const void *X; int64_t ldx; int64_t B;
    void *Y; int64_t ldy;
    int64_t N, K;
};
cudaError_t launch_gemv_nvfp4(const GemvNvArgs &args, cudaStream_t stream);          // CUDA cores, pair-table lookups
cudaError_t launch_gemv_nvfp4_mma(const GemvNvArgs &args, cudaStream_t stream);      // tensor cores (mma.sync), no lookups
cudaError_t launch_fill_e2m1_table(cudaStream_t stream);   // value-pair table of the NVFP4 decode kernel

}  // namespace dq
