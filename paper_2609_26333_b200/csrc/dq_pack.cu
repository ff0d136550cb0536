// Packers and quantisers: tensor scale, NVFP4 and LUT3 round-to-nearest,
// LUT3 -> NVFP4 autocast, canonical export, and the activation quantiser of the
// prefill path.  (App. A.3 "Quantization formats", Sec. 2.3, App. C.2 storage.)
//
// Quantiser arithmetic is fp32 with explicit round-to-nearest intrinsics so the
// compiler cannot contract or reorder it:
//   rc6 = 1/(6 s);  t = extreme * rc6;  d = E4M3(t);  r = 1/(s * dec(d));  y = x * r
#include "dq_common.cuh"

namespace dq {

// ---------------------------------------------------------------- converts

__device__ __forceinline__ uint32_t f32_to_e4m3(float t)
{
    // cvt packs two values; the second operand lands in the low byte
    unsigned short out;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(out) : "f"(0.0f), "f"(t));
    return out & 0xFFu;
}

__device__ __forceinline__ float e4m3_to_f32(uint32_t b)
{
    unsigned short in = (unsigned short)(b & 0xFFu);
    unsigned int h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(in));
    return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

// two floats -> one byte of E2M1 codes, `lo` in the low nibble
__device__ __forceinline__ uint32_t f32x2_to_e2m1x2(float lo, float hi)
{
    unsigned short out;
    asm("{\n\t.reg .b8 t;\n\tcvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\tcvt.u16.u8 %0, t;\n\t}"
        : "=h"(out) : "f"(hi), "f"(lo));
    return out & 0xFFu;
}

template <bool FP32IN>
__device__ __forceinline__ void load16(const void *base, int64_t row, int64_t k0, int64_t ld, float (&x)[16])
{
    if (FP32IN) {
        const float4 *p = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(base) + row * ld + k0);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float4 v = __ldg(p + j);
            x[4 * j] = v.x; x[4 * j + 1] = v.y; x[4 * j + 2] = v.z; x[4 * j + 3] = v.w;
        }
    } else {
        const uint4 *p = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(base) + row * ld + k0);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            uint4 v = __ldg(p + j);
            uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                x[8 * j + 2 * q] = __uint_as_float(w[q] << 16);
                x[8 * j + 2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
            }
        }
    }
}

// NVFP4 round-to-nearest of one 16-block: returns the E4M3 scale byte, writes 8 code bytes.
__device__ __forceinline__ uint32_t quant_block_nvfp4(const float (&x)[16], float s, float rc6, uint2 &codes)
{
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) a = fmaxf(a, fabsf(x[i]));
    const float t = __fmul_rn(a, rc6);
    const uint32_t d8 = f32_to_e4m3(t);
    codes = make_uint2(0u, 0u);
    if ((d8 & 0x7Fu) != 0u) {
        const float r = __frcp_rn(__fmul_rn(s, e4m3_to_f32(d8)));
        uint32_t w0 = 0, w1 = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            w0 |= f32x2_to_e2m1x2(__fmul_rn(x[2 * j], r), __fmul_rn(x[2 * j + 1], r)) << (8 * j);
            w1 |= f32x2_to_e2m1x2(__fmul_rn(x[8 + 2 * j], r), __fmul_rn(x[8 + 2 * j + 1], r)) << (8 * j);
        }
        codes = make_uint2(w0, w1);
    }
    return d8;
}

// ------------------------------------------------------------------ header

struct Codebook8 { unsigned short h[8]; };

__global__ void pack_header_kernel(PackedHeader *hdr, Codebook8 cb)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    hdr->amax_bits = 0u;
    hdr->s = 1.0f;
    hdr->rc6 = 0.0f;
    int zero_idx = 0;
    unsigned int amap = 0;
    for (int j = 0; j < 8; ++j) {
        float g = __half2float(__ushort_as_half(cb.h[j]));
        hdr->lut_levels[j] = g;
        hdr->lut_f16[j] = cb.h[j];
        if (g == 0.0f) zero_idx = j;
        amap |= (f32x2_to_e2m1x2(g, 0.0f) & 0xFu) << (4 * j);
    }
    for (int j = 0; j < 7; ++j)
        hdr->lut_thresholds[j] = __fmul_rn(__fadd_rn(hdr->lut_levels[j], hdr->lut_levels[j + 1]), 0.5f);
    hdr->lut_thresholds[7] = __int_as_float(0x7f800000);
    hdr->lut_zero_idx = zero_idx;
    hdr->autocast_map = amap;
}

cudaError_t launch_pack_header(PackedHeader *hdr, const uint16_t *codebook_f16_host, cudaStream_t stream)
{
    Codebook8 cb;
    for (int j = 0; j < 8; ++j) cb.h[j] = codebook_f16_host[j];
    pack_header_kernel<<<1, 32, 0, stream>>>(hdr, cb);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ absmax

template <bool FP32IN>
__global__ void absmax_kernel(const void *W, int64_t N, int64_t K, int64_t ldw, PackedHeader *hdr)
{
    const int64_t nb = K / 16;
    const int64_t total = N * nb;
    float a = 0.0f;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        float x[16];
        load16<FP32IN>(W, i / nb, (i % nb) * 16, ldw, x);
#pragma unroll
        for (int j = 0; j < 16; ++j) a = fmaxf(a, fabsf(x[j]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    __shared__ float red[32];
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x < 32) {
        a = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
        if (threadIdx.x == 0) atomicMax(&hdr->amax_bits, __float_as_uint(a));
    }
}

__global__ void finalize_scale_kernel(PackedHeader *hdr)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const float amax = __uint_as_float(hdr->amax_bits);
    const float s = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, 2688.0f);      // 6 * 448
    hdr->s = s;
    hdr->rc6 = __frcp_rn(__fmul_rn(6.0f, s));
}

cudaError_t launch_absmax(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw, PackedHeader *hdr,
                          cudaStream_t stream)
{
    const int64_t total = N * (K / 16);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (w_dtype == DQ_DT_FP32) absmax_kernel<true><<<blocks, 256, 0, stream>>>(W, N, K, ldw, hdr);
    else absmax_kernel<false><<<blocks, 256, 0, stream>>>(W, N, K, ldw, hdr);
    finalize_scale_kernel<<<1, 32, 0, stream>>>(hdr);
    return cudaGetLastError();
}

// -------------------------------------------------------------- NVFP4 pack

template <bool FP32IN>
__global__ void pack_nvfp4_kernel(const void *W, int64_t N, int64_t K, int64_t ldw, const PackedHeader *hdr,
                                  uint8_t *codes, uint8_t *sf)
{
    const int64_t nb = K / 16;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * nb) return;
    const int64_t r = i / nb, b = i % nb;
    float x[16];
    load16<FP32IN>(W, r, b * 16, ldw, x);
    uint2 c;
    const uint32_t d8 = quant_block_nvfp4(x, hdr->s, hdr->rc6, c);
    *reinterpret_cast<uint2 *>(codes + r * (K / 2) + b * 8) = c;
    sf[sf_swizzled_offset(r, b, K)] = (uint8_t)d8;
}

cudaError_t launch_pack_nvfp4(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                              const PackedHeader *hdr, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream)
{
    const int64_t total = N * (K / 16);
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (w_dtype == DQ_DT_FP32) pack_nvfp4_kernel<true><<<blocks, 256, 0, stream>>>(W, N, K, ldw, hdr, codes, sf_swizzled);
    else pack_nvfp4_kernel<false><<<blocks, 256, 0, stream>>>(W, N, K, ldw, hdr, codes, sf_swizzled);
    return cudaGetLastError();
}

// ------------------------------------------------------- decode pair table

// Image of the decode kernel's shared-memory table, built once at pack time: entry e (a byte holding the
// indices of two neighbouring weights as nibbles, idx_b << 4 | idx_a) -> (G[idx_a], G[idx_b]) as fp32,
// replicated into one 8-byte slot per lane (entry stride 256 bytes).
__global__ void build_lut_table_kernel(const PackedHeader *hdr, uint8_t *table)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 256 * 32) return;
    const int e = i >> 5, l = i & 31;
    const int ia = e & 7, ib = (e >> 4) & 7;
    *reinterpret_cast<float2 *>(table + e * 256 + l * 8) = make_float2(hdr->lut_levels[ia], hdr->lut_levels[ib]);
}

cudaError_t launch_build_lut_table(const PackedHeader *hdr, uint8_t *table_dev, cudaStream_t stream)
{
    build_lut_table_kernel<<<32, 256, 0, stream>>>(hdr, table_dev);
    return cudaGetLastError();
}

// --------------------------------------------------------------- LUT3 pack

// One thread quantises 32 consecutive weights (two 16-blocks) and emits one word of each bit-plane.
template <bool FP32IN>
__global__ void pack_lut3_kernel(const void *W, int64_t N, int64_t K, int64_t ldw, const PackedHeader *hdr,
                                 uint8_t *lut)
{
    const int64_t nw = K / 32;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * nw) return;
    const int64_t r = i / nw, j = i % nw;
    const float s = hdr->s, rc6 = hdr->rc6;
    float T[7];
#pragma unroll
    for (int q = 0; q < 7; ++q) T[q] = hdr->lut_thresholds[q];
    const int zero_idx = hdr->lut_zero_idx;
    uint32_t wd[3] = {0u, 0u, 0u};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float x[16];
        load16<FP32IN>(W, r, j * 32 + h * 16, ldw, x);
        // the block's maximum-magnitude weight with its sign; equal magnitudes: the positive one
        float m = x[0];
#pragma unroll
        for (int q = 1; q < 16; ++q) {
            const float v = x[q];
            if (fabsf(v) > fabsf(m) || (fabsf(v) == fabsf(m) && v > m)) m = v;
        }
        uint32_t d8 = f32_to_e4m3(__fmul_rn(m, rc6));
        if ((d8 & 0x7Fu) == 0u) d8 = 0u;
        lut[lut_scale_offset(r, j * 2 + h, K)] = (uint8_t)d8;
        const float rr = (d8 != 0u) ? __frcp_rn(__fmul_rn(s, e4m3_to_f32(d8))) : 0.0f;
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            int idx = zero_idx;
            if (d8 != 0u) {
                const float y = __fmul_rn(x[q], rr);
                idx = 0;
#pragma unroll
                for (int l = 0; l < 7; ++l) idx += (y > T[l]) ? 1 : 0;
            }
            const int i = h * 16 + q;
#pragma unroll
            for (int b = 0; b < 3; ++b) {
                int word, pos;
                lut3_locate(b, i, word, pos);                      // all indices are compile-time constants here
                wd[word] |= (uint32_t)((idx >> b) & 1) << pos;
            }
        }
    }
    // device layout: 448-byte blocks per (row, 1024-weight slice); bit order inside the word triplet per lut3_locate
#pragma unroll
    for (int p = 0; p < 3; ++p) *reinterpret_cast<uint32_t *>(lut + lut_word_offset(r, j, p, K)) = wd[p];
}

cudaError_t launch_pack_lut3(const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                             const PackedHeader *hdr, uint8_t *lut_dev, cudaStream_t stream)
{
    const int64_t total = N * (K / 32);
    const unsigned blocks = (unsigned)((total + 127) / 128);
    if (w_dtype == DQ_DT_FP32) pack_lut3_kernel<true><<<blocks, 128, 0, stream>>>(W, N, K, ldw, hdr, lut_dev);
    else pack_lut3_kernel<false><<<blocks, 128, 0, stream>>>(W, N, K, ldw, hdr, lut_dev);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- autocast

// NVFP4 view of the LUT3 codes (Sec. 2.3): level -> nearest E2M1 value, element signs
// flipped under a negative block scale, block scale |d|, same tensor scale.
// One thread per word triplet (32 weights).  A selector byte holds the indices of a weight pair as nibbles;
// a small shared-memory table maps such a byte to the byte of two E2M1 codes, in three variants: positive
// scale, negative scale (sign bits of non-zero codes flipped), zero scale (all codes zero).  Pair q of the
// triplet is byte q % 4 of selector word q / 4 and output byte q of the row's 16 code bytes.
__global__ void __launch_bounds__(256) autocast_kernel(const PackedHeader *hdr, const uint8_t *lut, int64_t N,
                                                       int64_t K, uint8_t *codes, uint8_t *sf)
{
    __shared__ uint8_t table[3][128];               // [variant][idx_b << 4 | idx_a] -> two E2M1 codes
    const uint32_t amap = hdr->autocast_map;
    for (int i = threadIdx.x; i < 3 * 128; i += blockDim.x) {
        const int v = i >> 7, e = i & 127;
        uint32_t ca = (amap >> (4 * (e & 7))) & 0xFu, cb = (amap >> (4 * ((e >> 4) & 7))) & 0xFu;
        if (v == 1) { if (ca & 7u) ca ^= 8u; if (cb & 7u) cb ^= 8u; }
        if (v == 2) { ca = 0u; cb = 0u; }
        table[v][e] = (uint8_t)(ca | (cb << 4));
    }
    __syncthreads();
    const int nw = (int)(K / 32);
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * nw) return;
    const int64_t r = i / nw;
    const int j = (int)(i - r * nw);
    const uint32_t w0 = *reinterpret_cast<const uint32_t *>(lut + lut_word_offset(r, j, 0, K));
    const uint32_t w1 = *reinterpret_cast<const uint32_t *>(lut + lut_word_offset(r, j, 1, K));
    const uint32_t w2 = *reinterpret_cast<const uint32_t *>(lut + lut_word_offset(r, j, 2, K));
    const uint32_t d2 = *reinterpret_cast<const unsigned short *>(lut + lut_scale_offset(r, j * 2, K));
    uint32_t sel[4], out[4];
    lut3_selectors(w0, w1, w2, sel);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t d8 = (g < 2) ? (d2 & 0xFFu) : (d2 >> 8);            // pairs 0..7 are block 0, 8..15 block 1
        const uint8_t *tab = table[d8 == 0u ? 2 : ((d8 & 0x80u) ? 1 : 0)];
        const uint32_t u = sel[g];
        out[g] = (uint32_t)tab[u & 0xFFu] | ((uint32_t)tab[(u >> 8) & 0xFFu] << 8) |
                 ((uint32_t)tab[(u >> 16) & 0xFFu] << 16) | ((uint32_t)tab[u >> 24] << 24);
    }
    *reinterpret_cast<uint4 *>(codes + r * (K / 2) + (int64_t)j * 16) = make_uint4(out[0], out[1], out[2], out[3]);
    sf[sf_swizzled_offset(r, j * 2, K)] = (uint8_t)(d2 & 0x7Fu);
    sf[sf_swizzled_offset(r, j * 2 + 1, K)] = (uint8_t)((d2 >> 8) & 0x7Fu);
}

cudaError_t launch_autocast(const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                            int64_t K, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream)
{
    const int64_t total = N * (K / 32);
    autocast_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(hdr, lut_dev, N, K, codes, sf_swizzled);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ export

__global__ void export_nvfp4_kernel(const PackedHeader *hdr, const uint8_t *codes, const uint8_t *sf, int64_t N,
                                    int64_t K, uint8_t *codes_out, uint8_t *scales_out, float *s_out)
{
    const int64_t nb = K / 16;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0 && s_out) *s_out = hdr->s;
    if (i >= N * nb) return;
    const int64_t r = i / nb, b = i % nb;
    *reinterpret_cast<uint2 *>(codes_out + r * (K / 2) + b * 8) =
        *reinterpret_cast<const uint2 *>(codes + r * (K / 2) + b * 8);
    scales_out[r * nb + b] = sf[sf_swizzled_offset(r, b, K)];
}

cudaError_t launch_export_nvfp4(const PackedHeader *hdr, const uint8_t *codes, const uint8_t *sf_swizzled, int64_t N,
                                int64_t K, uint8_t *codes_out, uint8_t *scales_out, float *s_out,
                                cudaStream_t stream)
{
    const int64_t total = N * (K / 16);
    export_nvfp4_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(hdr, codes, sf_swizzled, N, K,
                                                                             codes_out, scales_out, s_out);
    return cudaGetLastError();
}

__global__ void export_lut3_kernel(const PackedHeader *hdr, const uint8_t *lut, int64_t N,
                                   int64_t K, uint32_t *planes_out, uint8_t *scales_out, float *s_out)
{
    const int64_t nw = K / 32;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0 && s_out) *s_out = hdr->s;
    if (i >= N * nw) return;
    const int64_t r = i / nw, j = i % nw;
    uint32_t wd[3];
#pragma unroll
    for (int p = 0; p < 3; ++p) wd[p] = *reinterpret_cast<const uint32_t *>(lut + lut_word_offset(r, j, p, K));
#pragma unroll
    for (int p = 0; p < 3; ++p) {
        uint32_t c = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            int word, pos;
            lut3_locate(p, i, word, pos);
            c |= ((wd[word] >> pos) & 1u) << i;                                      // canonical: LSB-first bit-planes
        }
        planes_out[(r * 3 + p) * nw + j] = c;
    }
    scales_out[r * (K / 16) + 2 * j] = lut[lut_scale_offset(r, 2 * j, K)];
    scales_out[r * (K / 16) + 2 * j + 1] = lut[lut_scale_offset(r, 2 * j + 1, K)];
}

cudaError_t launch_export_lut3(const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                               int64_t K, uint32_t *planes_out, uint8_t *scales_out, float *s_out,
                               cudaStream_t stream)
{
    const int64_t total = N * (K / 32);
    export_lut3_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(hdr, lut_dev, N, K, planes_out,
                                                                            scales_out, s_out);
    return cudaGetLastError();
}

// Last launch of every pack / import: does nothing.  The decode kernel is launched so that its set-up may
// overlap the kernel before it in the stream; with this launch in between, that kernel is never one that
// writes the packed buffer.
__global__ void pack_done_kernel() {}
cudaError_t launch_pack_done(cudaStream_t stream)
{
    pack_done_kernel<<<1, 32, 0, stream>>>();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ import

// Canonical codes / scales (the layouts of the export) -> device layouts.  Inverse of the export kernels.
__global__ void import_nvfp4_kernel(const uint8_t *codes_in, const uint8_t *scales_in, int64_t N, int64_t K,
                                    uint8_t *codes, uint8_t *sf)
{
    const int64_t nb = K / 16;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * nb) return;
    const int64_t r = i / nb, b = i % nb;
    *reinterpret_cast<uint2 *>(codes + r * (K / 2) + b * 8) =
        *reinterpret_cast<const uint2 *>(codes_in + r * (K / 2) + b * 8);
    sf[sf_swizzled_offset(r, b, K)] = scales_in[r * nb + b];
}

__global__ void import_lut3_kernel(const uint32_t *planes_in, const uint8_t *scales_in, int64_t N, int64_t K,
                                   uint8_t *lut)
{
    const int64_t nw = K / 32;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * nw) return;
    const int64_t r = i / nw, j = i % nw;
    uint32_t wd[3] = {0u, 0u, 0u};
#pragma unroll
    for (int p = 0; p < 3; ++p) {
        const uint32_t c = planes_in[(r * 3 + p) * nw + j];                        // canonical: LSB-first bit-planes
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            int word, pos;
            lut3_locate(p, i, word, pos);
            wd[word] |= ((c >> i) & 1u) << pos;
        }
    }
#pragma unroll
    for (int p = 0; p < 3; ++p) *reinterpret_cast<uint32_t *>(lut + lut_word_offset(r, j, p, K)) = wd[p];
    lut[lut_scale_offset(r, 2 * j, K)] = scales_in[r * (K / 16) + 2 * j];
    lut[lut_scale_offset(r, 2 * j + 1, K)] = scales_in[r * (K / 16) + 2 * j + 1];
}

__global__ void set_scale_kernel(PackedHeader *hdr, float s)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    hdr->s = s;
    hdr->rc6 = __frcp_rn(__fmul_rn(6.0f, s));
    hdr->amax_bits = __float_as_uint(__fmul_rn(s, 2688.0f));
}

cudaError_t launch_set_scale(PackedHeader *hdr, float s, cudaStream_t stream)
{
    set_scale_kernel<<<1, 32, 0, stream>>>(hdr, s);
    return cudaGetLastError();
}

cudaError_t launch_import_nvfp4(const uint8_t *codes_in, const uint8_t *scales_in, int64_t N, int64_t K, uint8_t *codes,
                                uint8_t *sf_swizzled, cudaStream_t stream)
{
    const int64_t total = N * (K / 16);
    import_nvfp4_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(codes_in, scales_in, N, K, codes,
                                                                             sf_swizzled);
    return cudaGetLastError();
}

cudaError_t launch_import_lut3(const uint32_t *planes_in, const uint8_t *scales_in, int64_t N, int64_t K,
                               uint8_t *lut_dev, cudaStream_t stream)
{
    const int64_t total = N * (K / 32);
    import_lut3_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(planes_in, scales_in, N, K, lut_dev);
    return cudaGetLastError();
}

// --------------------------------------------------- activation quantiser

// eight floats -> four bytes of E2M1 codes (element 0 in the low nibble of byte 0)
__device__ __forceinline__ uint32_t f32x8_to_e2m1x8(float f0, float f1, float f2, float f3, float f4, float f5, float f6,
                                                    float f7)
{
    uint32_t r;
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
        : "=r"(r) : "f"(f0), "f"(f1), "f"(f2), "f"(f3), "f"(f4), "f"(f5), "f"(f6), "f"(f7));
    return r;
}

// NVFP4 round-to-nearest of one 16-block held as eight packed bf16 pairs; same arithmetic as
// quant_block_nvfp4 (the block maximum is exact in bf16, so taking it on packed pairs changes nothing)
__device__ __forceinline__ uint32_t quant_block_nvfp4_bf16(const uint32_t (&w)[8], float s, float rc6, uint2 &codes)
{
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t a;
        asm("abs.bf16x2 %0, %1;" : "=r"(a) : "r"(w[i]));
        if (i == 0) m = a;
        else asm("max.bf16x2 %0, %0, %1;" : "+r"(m) : "r"(a));
    }
    const float a = fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
    const float t = __fmul_rn(a, rc6);
    const uint32_t d8 = f32_to_e4m3(t);
    codes = make_uint2(0u, 0u);
    if ((d8 & 0x7Fu) != 0u) {
        const float r = __frcp_rn(__fmul_rn(s, e4m3_to_f32(d8)));
        float y[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            y[2 * i] = __fmul_rn(__uint_as_float(w[i] << 16), r);
            y[2 * i + 1] = __fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), r);
        }
        codes.x = f32x8_to_e2m1x8(y[0], y[1], y[2], y[3], y[4], y[5], y[6], y[7]);
        codes.y = f32x8_to_e2m1x8(y[8], y[9], y[10], y[11], y[12], y[13], y[14], y[15]);
    }
    return d8;
}

// bf16 -> NVFP4 with a static tensor scale (App. A.3 "NVFP4").  One thread per
// 16-block: 32 B in, 8 B of codes out; four neighbouring lanes (one 64-wide k
// atom) merge their scale bytes into one 32-bit store of the MMA scale layout.
template <bool SWIZZLED>
__global__ void __launch_bounds__(256) quant_act_kernel(const __nv_bfloat16 *A, int M, int nb, int64_t lda,
                                                        float s, uint8_t *codes, uint8_t *sf)
{
    // launched with programmatic stream serialization (hides the launch latency behind the previous
    // kernel); that kernel may produce A or still read the workspace, so wait for it before anything else
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // 64 blocks of one row per 64 threads, four rows per CTA: no division, 32-bit index arithmetic
    const int b = blockIdx.y * 64 + threadIdx.x;
    const int r = blockIdx.x * 4 + threadIdx.y;
    const bool live = (b < nb) && (r < M);
    const float rc6 = __frcp_rn(__fmul_rn(6.0f, s));
    uint32_t d8 = 0;
    if (live) {
        const uint4 *p = reinterpret_cast<const uint4 *>(A + (int64_t)r * lda + b * 16);
        const uint4 v0 = __ldg(p), v1 = __ldg(p + 1);
        const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        uint2 c;
        d8 = quant_block_nvfp4_bf16(w, s, rc6, c);
        *reinterpret_cast<uint2 *>(codes + ((int64_t)r * nb + b) * 8) = c;
    }
    // K % 64 == 0, so lanes 4q..4q+3 always hold the four blocks of one k atom of one row
    uint32_t w = d8 << (8 * (threadIdx.x & 3));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    if (live && (threadIdx.x & 3) == 0) {
        if (SWIZZLED) {
            // atom (r / 128, b / 4) of 512 bytes; row rr of the atom at (rr % 32) * 16 + (rr / 32) * 4
            const int rr = r & 127;
            const size_t off = ((size_t)(r >> 7) * (size_t)(nb >> 2) + (size_t)(b >> 2)) * 512 + (size_t)((rr & 31) * 16 + (rr >> 5) * 4);
            *reinterpret_cast<uint32_t *>(sf + off) = w;
        } else {
            *reinterpret_cast<uint32_t *>(sf + (int64_t)r * nb + b) = w;
        }
    }
}

cudaError_t launch_quant_act(const void *A_bf16, int64_t M, int64_t K, int64_t lda, float act_scale, uint8_t *codes,
                             uint8_t *sf, int swizzled, cudaStream_t stream)
{
    const int nb = (int)(K / 16);
    const int m = (int)M;
    const __nv_bfloat16 *A = reinterpret_cast<const __nv_bfloat16 *>(A_bf16);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((m + 3) / 4), (unsigned)((nb + 63) / 64));
    cfg.blockDim = dim3(64, 4);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (swizzled) return cudaLaunchKernelEx(&cfg, quant_act_kernel<true>, A, m, nb, lda, act_scale, codes, sf);
    return cudaLaunchKernelEx(&cfg, quant_act_kernel<false>, A, m, nb, lda, act_scale, codes, sf);
}

}  // namespace dq
