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
constexpr int kMaxDevices = 64;       // per-device one-time set-up flags
constexpr int kSfAtomRows = 128;      // rows of one scale-factor atom of the block-scaled MMA
constexpr int kSfAtomBytes = 512;     // 128 rows x 4 scales (64 k)
constexpr int kSfRowPad = 256;        // NVFP4 scale tiles padded to the GEMM's N tile

// Device header at the start of the packed buffer (1 KiB reserved).
struct PackedHeader {
    unsigned int amax_bits;       // max|W| as fp32 bits (non-negative floats order like uints)
    float s;                      // tensor scale  s = max|W| / (6*448)
    float rc6;                    // 1 / (6 s)
    float pad0;
    float lut_levels[8];          // LUT3 codebook as fp32
    float lut_thresholds[8];      // midpoints between consecutive levels (7 used)
    unsigned int lut_f16[8];      // LUT3 codebook, fp16 bit patterns
    int lut_zero_idx;
    unsigned int autocast_map;    // 8 nibbles: E2M1 code of each LUT3 level
    float lut2_levels[4];         // LUT2 codebook as fp32
    float lut2_thresholds[4];     // 3 used
    unsigned int lut2_f16[4];
    int lut2_zero_idx;
    int pad1[5];
    // codebooks as byte-permute tables: low bytes of levels 0-3, of levels 4-7, high bytes of levels 0-3, of levels 4-7
    unsigned int lut_prmt[4];
    unsigned int lut2_prmt[4];
};
static_assert(sizeof(PackedHeader) <= 1024 && offsetof(PackedHeader, lut_prmt) % 16 == 0, "header layout");
constexpr size_t kHeaderBytes = 1024;

// LUT device layout (LUT3 and LUT2).  The unit is an "atom": 8 consecutive rows x 512 consecutive weights,
//   [index words: BITS x 512 bytes][block scales: 8 rows x 32 signed E4M3 bytes]      1792 B (LUT3), 1280 B (LUT2)
// i.e. BITS + 0.5 bit per weight.  Atoms are ordered [16-row tile][1024-weight slice][row half][k half], so the
// two atoms of an (8 rows x 1024 weights) chunk are contiguous, and so are the four of a 16-row chunk.  A partial
// last slice is zero padded (zero scales: the padding contributes nothing).
// Inside an atom the index words are laid out for the fragment layout of mma.m16n8k16: lane (g, t), g = row of the
// atom, t = 0..3, owns weights 4t .. 4t+3 of every 16-weight block of its row (one mma contracts one block per
// row, lane t supplying its four weights), and reads them with one 16-byte load per index word "plane":
//   byte offset of word p (0..BITS-1) of lane (g, t), word group wi (0..3):  p * 512 + (4 g + t) * 16 + 4 wi.
// A word group (BITS words) holds 32 weights of the lane: its four weights of the eight blocks 8 wi .. 8 wi + 7 of
// the atom.  Selector word a (0..3) of a group serves blocks 8 wi + 2a (nibbles 0-3) and 8 wi + 2a + 1 (nibbles 4-7),
// nibble n holding the index of the lane's weight n % 4 of that block:
//   LUT3: selector a < 3 is stored word a with the top bit of every nibble cleared; those top bits hold selector 3
//         (bit b of its nibble n in bit 4n+3 of word b).
//   LUT2: selector a is the even (a even) or odd (a odd) 2-bit fields of word a / 2.
// Nibbles are what byte-permute takes as selectors, so a stored word becomes four looked-up weights per permute
// after one AND.  The canonical (export) layout is the bit-plane form of App. C.2.
constexpr int kLutAtomRows = 8;
constexpr int kLutAtomK = 512;
constexpr int kLutSlice = 1024;
constexpr int kLutAtomScaleBytes = 256;
constexpr int64_t kLutMaxK = 32768;       // the decode kernel keeps one fp16 activation row of K in shared memory
__host__ __device__ constexpr int lut_plane_bytes(int bits) { return bits * 512; }
__host__ __device__ constexpr int lut_atom_bytes(int bits) { return bits * 512 + kLutAtomScaleBytes; }
__host__ __device__ inline int64_t lut_slices(int64_t K) { return (K + kLutSlice - 1) / kLutSlice; }
// byte offset of the atom holding row r, weights 512 a .. 512 a + 511
__host__ __device__ inline size_t lut_atom_offset(int64_t r, int64_t a, int64_t K, int bits)
{
    const int64_t tile16 = r >> 4, rowhalf = (r >> 3) & 1;
    return (size_t)((((tile16 * lut_slices(K) + (a >> 1)) * 2 + rowhalf) * 2 + (a & 1))) * (size_t)lut_atom_bytes(bits);
}
// scale byte of 16-block b of row r
__host__ __device__ inline size_t lut_scale_offset(int64_t r, int64_t b, int64_t K, int bits)
{
    return lut_atom_offset(r, b >> 5, K, bits) + (size_t)lut_plane_bytes(bits) + (size_t)(r & 7) * 32 + (size_t)(b & 31);
}
// word p of the group of lane (r % 8, t) that holds its weights of blocks 8 q .. 8 q + 7 of row r (q = k / 128)
__host__ __device__ inline size_t lut_word_offset(int64_t r, int64_t q, int t, int p, int64_t K, int bits)
{
    return lut_atom_offset(r, q >> 2, K, bits) + (size_t)p * 512 + (size_t)((r & 7) * 4 + t) * 16 + (size_t)(q & 3) * 4;
}
// where index bit `bit` of the lane's weight n4 (0..3) of block bb (0..7) of a word group lives
template <int BITS>
__host__ __device__ inline void lut_locate(int bb, int n4, int bit, int &word, int &pos)
{
    const int a = bb >> 1, nib = (bb & 1) * 4 + n4;
    if (BITS == 3) {
        if (a < 3) { word = a; pos = 4 * nib + bit; }
        else { word = bit; pos = 4 * nib + 3; }
    } else {
        word = a >> 1;
        pos = 4 * nib + 2 * (a & 1) + bit;
    }
}
// the four selector words of a word group
template <int BITS>
__device__ __forceinline__ void lut_selectors(const uint32_t (&w)[BITS], uint32_t (&sel)[4])
{
    if (BITS == 3) {
        sel[0] = w[0] & 0x77777777u;
        sel[1] = w[1] & 0x77777777u;
        sel[2] = w[BITS - 1] & 0x77777777u;
        sel[3] = ((w[0] >> 3) & 0x11111111u) | ((w[1] >> 2) & 0x22222222u) | ((w[BITS - 1] >> 1) & 0x44444444u);
    } else {
        sel[0] = w[0] & 0x33333333u;
        sel[1] = (w[0] >> 2) & 0x33333333u;
        sel[2] = w[1] & 0x33333333u;
        sel[3] = (w[1] >> 2) & 0x33333333u;
    }
}

struct PackedLayout {
    size_t nv_codes_off = 0, nv_codes_bytes = 0;     // uint8[N][K/2]
    size_t nv_sf_off = 0, nv_sf_bytes = 0;           // [ceil(N/256)*2][K/64][512] MMA scale layout
    size_t lut_off = 0, lut_bytes = 0;               // LUT3 atoms
    size_t lut2_off = 0, lut2_bytes = 0;             // LUT2 atoms
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
        L.lut_off = off;
        L.lut_bytes = (size_t)(N / 16) * lut_slices(K) * 4 * lut_atom_bytes(3);
        off = align_up(off + L.lut_bytes, 1024);
    }
    if (formats & DQ_FMT_LUT2) {
        L.lut2_off = off;
        L.lut2_bytes = (size_t)(N / 16) * lut_slices(K) * 4 * lut_atom_bytes(2);
        off = align_up(off + L.lut2_bytes, 1024);
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

// Device status word: [0] = dq_status, [1] = detail; then, for measurement, what the last pair-GEMM launch took on the
// SM of its first CTA: SM clock cycles and nanoseconds of the global timer from the CTA's start to its end.
struct StatusWord { int status; int detail; unsigned long long gemm_cycles; unsigned long long gemm_ns; };

bool handle_on_current_device(const dq_weights *w);      // defined beside the handle (dq_api.cu)

// ---- launchers (each enqueues on `stream`, returns a cudaError_t) ----
cudaError_t launch_pack_header(PackedHeader *hdr, const uint16_t *codebook_f16_host, cudaStream_t stream);
cudaError_t launch_absmax(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw, PackedHeader *hdr,
                          cudaStream_t stream);
cudaError_t launch_pack_nvfp4(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                              const PackedHeader *hdr, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream);
// bits = 3 (LUT3) or 2 (LUT2) in the four LUT launchers below
cudaError_t launch_pack_lut(int bits, const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                            const PackedHeader *hdr, uint8_t *lut_dev, cudaStream_t stream);
cudaError_t launch_autocast(const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                            int64_t K, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream);
cudaError_t launch_export_nvfp4(const PackedHeader *hdr, const uint8_t *codes, const uint8_t *sf_swizzled, int64_t N,
                                int64_t K, uint8_t *codes_out, uint8_t *scales_out, float *s_out,
                                cudaStream_t stream);
cudaError_t launch_export_lut(int bits, const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                              int64_t K, uint32_t *planes_out, uint8_t *scales_out, float *s_out,
                              cudaStream_t stream);
cudaError_t launch_pack_done(cudaStream_t stream);
cudaError_t launch_set_scale(PackedHeader *hdr, float s, cudaStream_t stream);
cudaError_t launch_import_nvfp4(const uint8_t *codes_in, const uint8_t *scales_in, int64_t N, int64_t K, uint8_t *codes,
                                uint8_t *sf_swizzled, cudaStream_t stream);
cudaError_t launch_import_lut(int bits, const uint32_t *planes_in, const uint8_t *scales_in, int64_t N, int64_t K,
                              uint8_t *lut_dev, cudaStream_t stream);
// Activation quantiser: codes row-major [M][K/2]; scales either in the MMA layout
// (swizzled != 0) or canonical [M][K/16].
cudaError_t launch_quant_act(const void *A_bf16, int64_t M, int64_t K, int64_t lda, float act_scale, uint8_t *codes,
                             uint8_t *sf, int swizzled, cudaStream_t stream);

// fused activation processing + quantiser (dq_fused_quant.cu); outputs as launch_quant_act
cudaError_t launch_rmsnorm_quant(const void *X_bf16, int64_t M, int64_t K, int64_t ldx, const void *gamma_bf16, float eps,
                                 float act_scale, uint8_t *codes, uint8_t *sf, int swizzled, cudaStream_t stream);
cudaError_t launch_silu_mul_quant(const void *GU_bf16, int64_t M, int64_t F, int64_t ldgu, float act_scale, uint8_t *codes,
                                  uint8_t *sf, int swizzled, cudaStream_t stream);
cudaError_t launch_silu_probe(const void *g_bf16, int64_t n, float *out, cudaStream_t stream);

struct GemmArgs {
    const uint8_t *a_codes;  const uint8_t *a_sf;      // activations: [M][K/2], MMA scale layout
    const uint8_t *w_codes;  const uint8_t *w_sf;      // weights:     [N][K/2], MMA scale layout
    const PackedHeader *hdr;                           // tensor scale of the weights
    float act_scale;
    void *Y; int64_t ldy;
    int64_t M, N, K;
    StatusWord *status;
    bool mma_only = false;   // measurement: MMA issue sequence only (pair kernel; no loads, scale copies or stores)
    // gated epilogue (pair kernel only): W is a fused gate/up matrix with interleaved rows, and instead of Y the kernel
    // writes NVFP4(bf16(SiLU(gate) * up)) with input scale gated_scale: codes [M][N/4], block scales in the MMA's layout
    uint8_t *gated_codes = nullptr; uint8_t *gated_sf = nullptr; float gated_scale = 0.0f;
};
cudaError_t launch_gemm_nvfp4(const GemmArgs &args, cudaStream_t stream);
cudaError_t launch_gemm_nvfp4_pair(const GemmArgs &args, void *encode_fn, cudaStream_t stream);
int gemm_init_driver_api();   // resolves the tensor-map encoder; 0 on success

struct GemvArgs {
    int bits = 3;                                         // 3 = LUT3, 2 = LUT2
    const uint8_t *lut; const PackedHeader *hdr;          // atoms (index words + scales)
    StatusWord *status = nullptr;
    const void *X; int64_t ldx; int64_t B;
    void *Y; int64_t ldy;
    int64_t N, K;
    // test hooks: warps per row group, row groups per CTA, ring depth (0 = chosen by the launcher), wait budget in
    // clock cycles (0 = default)
    int force_P = 0, force_G = 0, force_S = 0;
    long long wait_cycles = 0;
    int drop_first_copy = 0;                              // one warp's first copy is never requested (its wait must run out)
    int kernel = 0;                                       // 0 = chosen by the launcher, 1 = mma.sync kernel, 2 = tcgen05 kernel (batch 1), 3 = slice-by-slice kernel (batches above 8)
};
cudaError_t launch_gemv_lut(const GemvArgs &args, cudaStream_t stream);     // picks one of the two kernels below
// tcgen05 kernel (batch 1): number of warpgroups it would run this shape with, 0 where it does not take it
int gemv_lut_tc_warpgroups(int bits, int64_t N, int64_t K, int64_t B, int sms, bool any_size);
cudaError_t launch_gemv_lut_tc(const GemvArgs &args, int warpgroups, cudaStream_t stream);

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
cudaError_t launch_fill_e2m1_table(cudaStream_t stream);
// read-only streaming sum with 128-bit loads (measurement): 8 bytes of result at out_dev
cudaError_t launch_stream_read(const void *src_dev, size_t bytes, void *out_dev, cudaStream_t stream);   // value-pair table of the NVFP4 decode kernel

}  // namespace dq
