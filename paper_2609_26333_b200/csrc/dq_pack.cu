// Packers and quantisers: tensor scale, NVFP4 and LUT3 round-to-nearest,
// LUT3 -> NVFP4 autocast, canonical export, and the activation quantiser of the
// prefill path.  (App. A.3 "Quantization formats", Sec. 2.3, App. C.2 storage.)
//
// Quantiser arithmetic is fp32 with explicit round-to-nearest intrinsics so the
// compiler cannot contract or reorder it:
//   rc6 = 1/(6 s);  t = extreme * rc6;  d = E4M3(t);  r = 1/(s * dec(d));  y = x * r
#include "dq_common.cuh"
#include "dq_quant.cuh"

namespace dq {

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
    // LUT2A16 grid (App. A.3 "LUT formats"), rounded to fp16
    const float grid2[4] = {-3.6517f, 0.0f, 2.5227f, 6.0f};
    for (int j = 0; j < 4; ++j) {
        const __half h = __float2half_rn(grid2[j]);
        hdr->lut2_f16[j] = __half_as_ushort(h);
        hdr->lut2_levels[j] = __half2float(h);
        if (hdr->lut2_levels[j] == 0.0f) hdr->lut2_zero_idx = j;
    }
    for (int j = 0; j < 3; ++j)
        hdr->lut2_thresholds[j] = __fmul_rn(__fadd_rn(hdr->lut2_levels[j], hdr->lut2_levels[j + 1]), 0.5f);
    hdr->lut2_thresholds[3] = __int_as_float(0x7f800000);
    for (int q = 0; q < 4; ++q) { hdr->lut_prmt[q] = 0u; hdr->lut2_prmt[q] = 0u; }
    for (int j = 0; j < 8; ++j) {
        hdr->lut_prmt[j >> 2] |= (hdr->lut_f16[j] & 0xFFu) << (8 * (j & 3));
        hdr->lut_prmt[2 + (j >> 2)] |= ((hdr->lut_f16[j] >> 8) & 0xFFu) << (8 * (j & 3));
    }
    for (int j = 0; j < 4; ++j) {
        hdr->lut2_prmt[0] |= (hdr->lut2_f16[j] & 0xFFu) << (8 * j);
        hdr->lut2_prmt[2] |= ((hdr->lut2_f16[j] >> 8) & 0xFFu) << (8 * j);
    }
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

// ---------------------------------------------------------------- LUT pack

template <bool FP32IN>
__device__ __forceinline__ void load4(const void *base, int64_t row, int64_t k0, int64_t ld, float (&x)[4])
{
    if (FP32IN) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(base) + row * ld + k0));
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(base) + row * ld + k0));
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xFFFF0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xFFFF0000u);
    }
}

// the larger magnitude of two signed values; equal magnitudes: the positive one
__device__ __forceinline__ float signed_extreme(float m, float v)
{
    return (fabsf(v) > fabsf(m) || (fabsf(v) == fabsf(m) && v > m)) ? v : m;
}

// LUT3 / LUT2 round-to-nearest (App. A.3 "LUT formats").  Four neighbouring threads (t = 0..3) quantise the 128
// weights 128 q .. 128 q + 127 of one row: thread t holds weights 4t .. 4t+3 of each of the eight 16-blocks, which is
// exactly what its word group of the device layout stores; the block extreme is found across the four threads.
template <bool FP32IN, int BITS>
__global__ void __launch_bounds__(128) pack_lut_kernel(const void *W, int64_t N, int64_t K, int64_t ldw,
                                                       const PackedHeader *hdr, uint8_t *lut)
{
    const int64_t nq = K / 128;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t quad = i >> 2;
    const int t = (int)(i & 3);
    const bool live = quad < N * nq;                      // whole quads are live or not; shuffles stay inside a quad
    const int64_t r = live ? quad / nq : 0, q = live ? quad % nq : 0;
    const float s = hdr->s, rc6 = hdr->rc6;
    constexpr int NT = (1 << BITS) - 1;
    float T[NT];
#pragma unroll
    for (int l = 0; l < NT; ++l) T[l] = (BITS == 3) ? hdr->lut_thresholds[l] : hdr->lut2_thresholds[l];
    const int zero_idx = (BITS == 3) ? hdr->lut_zero_idx : hdr->lut2_zero_idx;
    uint32_t wd[BITS];
#pragma unroll
    for (int p = 0; p < BITS; ++p) wd[p] = 0u;
    uint32_t sc_lo = 0u, sc_hi = 0u;
#pragma unroll
    for (int bb = 0; bb < 8; ++bb) {
        float x[4];
        load4<FP32IN>(W, r, q * 128 + bb * 16 + t * 4, ldw, x);
        // the block's maximum-magnitude weight with its sign; equal magnitudes: the positive one
        float m = signed_extreme(signed_extreme(x[0], x[1]), signed_extreme(x[2], x[3]));
        m = signed_extreme(m, __shfl_xor_sync(0xffffffffu, m, 1));
        m = signed_extreme(m, __shfl_xor_sync(0xffffffffu, m, 2));
        uint32_t d8 = f32_to_e4m3(__fmul_rn(m, rc6));
        if ((d8 & 0x7Fu) == 0u) d8 = 0u;
        if (bb < 4) sc_lo |= d8 << (8 * bb); else sc_hi |= d8 << (8 * (bb - 4));
        const float rr = (d8 != 0u) ? __frcp_rn(__fmul_rn(s, e4m3_to_f32(d8))) : 0.0f;
#pragma unroll
        for (int n4 = 0; n4 < 4; ++n4) {
            int idx = zero_idx;
            if (d8 != 0u) {
                const float y = __fmul_rn(x[n4], rr);
                idx = 0;
#pragma unroll
                for (int l = 0; l < NT; ++l) idx += (y > T[l]) ? 1 : 0;
            }
#pragma unroll
            for (int b = 0; b < BITS; ++b) {
                int word, pos;
                lut_locate<BITS>(bb, n4, b, word, pos);            // compile-time constants after unrolling
                wd[word] |= (uint32_t)((idx >> b) & 1) << pos;
            }
        }
    }
    if (!live) return;
#pragma unroll
    for (int p = 0; p < BITS; ++p) *reinterpret_cast<uint32_t *>(lut + lut_word_offset(r, q, t, p, K, BITS)) = wd[p];
    if (t == 0) *reinterpret_cast<uint2 *>(lut + lut_scale_offset(r, q * 8, K, BITS)) = make_uint2(sc_lo, sc_hi);
}

cudaError_t launch_pack_lut(int bits, const void *W, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                            const PackedHeader *hdr, uint8_t *lut_dev, cudaStream_t stream)
{
    const int64_t total = N * (K / 128) * 4;
    const unsigned blocks = (unsigned)((total + 127) / 128);
    const bool f32 = (w_dtype == DQ_DT_FP32);
    if (bits == 3) {
        if (f32) pack_lut_kernel<true, 3><<<blocks, 128, 0, stream>>>(W, N, K, ldw, hdr, lut_dev);
        else pack_lut_kernel<false, 3><<<blocks, 128, 0, stream>>>(W, N, K, ldw, hdr, lut_dev);
    } else {
        if (f32) pack_lut_kernel<true, 2><<<blocks, 128, 0, stream>>>(W, N, K, ldw, hdr, lut_dev);
        else pack_lut_kernel<false, 2><<<blocks, 128, 0, stream>>>(W, N, K, ldw, hdr, lut_dev);
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------- autocast

// NVFP4 view of the LUT3 codes (Sec. 2.3): level -> nearest E2M1 value, element signs
// flipped under a negative block scale, block scale |d|, same tensor scale.
// One thread per word group (32 weights: four of each of eight blocks).  A selector byte holds the indices of a
// weight pair as nibbles; a small shared-memory table maps such a byte to the byte of two E2M1 codes, in three
// variants: positive scale, negative scale (sign bits of non-zero codes flipped), zero scale (all codes zero).
// Selector word a holds blocks 2a (low half) and 2a+1 (high half); the thread's four codes of a block are two
// consecutive bytes of the row's code bytes.
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
    const int64_t nq = K / 128;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t quad = i >> 2;
    const int t = (int)(i & 3);
    if (quad >= N * nq) return;
    const int64_t r = quad / nq, q = quad % nq;
    uint32_t w[3], sel[4];
#pragma unroll
    for (int p = 0; p < 3; ++p) w[p] = *reinterpret_cast<const uint32_t *>(lut + lut_word_offset(r, q, t, p, K, 3));
    lut_selectors<3>(w, sel);
    const uint2 d8x8 = *reinterpret_cast<const uint2 *>(lut + lut_scale_offset(r, q * 8, K, 3));
#pragma unroll
    for (int bb = 0; bb < 8; ++bb) {
        const uint32_t d8 = ((bb < 4 ? d8x8.x : d8x8.y) >> (8 * (bb & 3))) & 0xFFu;
        const uint8_t *tab = table[d8 == 0u ? 2 : ((d8 & 0x80u) ? 1 : 0)];
        const uint32_t u = (sel[bb >> 1] >> (16 * (bb & 1))) & 0xFFFFu;
        const unsigned short two = (unsigned short)((uint32_t)tab[u & 0xFFu] | ((uint32_t)tab[u >> 8] << 8));
        *reinterpret_cast<unsigned short *>(codes + r * (K / 2) + q * 64 + bb * 8 + t * 2) = two;
        if (t == (bb & 3)) sf[sf_swizzled_offset(r, q * 8 + bb, K)] = (uint8_t)(d8 & 0x7Fu);
    }
}

cudaError_t launch_autocast(const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                            int64_t K, uint8_t *codes, uint8_t *sf_swizzled, cudaStream_t stream)
{
    const int64_t total = N * (K / 128) * 4;
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

// index of weight k of row r, read from the device layout
template <int BITS>
__device__ __forceinline__ int lut_read_index(const uint8_t *lut, int64_t r, int64_t k, int64_t K)
{
    const int64_t q = k >> 7;
    const int bb = (int)((k >> 4) & 7), t = (int)((k >> 2) & 3), n4 = (int)(k & 3);
    int idx = 0;
#pragma unroll
    for (int b = 0; b < BITS; ++b) {
        int word, pos;
        lut_locate<BITS>(bb, n4, b, word, pos);
        const uint32_t w = *reinterpret_cast<const uint32_t *>(lut + lut_word_offset(r, q, t, word, K, BITS));
        idx |= (int)((w >> pos) & 1u) << b;
    }
    return idx;
}

template <int BITS>
__global__ void export_lut_kernel(const PackedHeader *hdr, const uint8_t *lut, int64_t N,
                                  int64_t K, uint32_t *planes_out, uint8_t *scales_out, float *s_out)
{
    const int64_t nw = K / 32;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0 && s_out) *s_out = hdr->s;
    if (i >= N * nw) return;
    const int64_t r = i / nw, j = i % nw;
    uint32_t c[BITS];
#pragma unroll
    for (int p = 0; p < BITS; ++p) c[p] = 0u;
    for (int e = 0; e < 32; ++e) {
        const int idx = lut_read_index<BITS>(lut, r, j * 32 + e, K);
#pragma unroll
        for (int p = 0; p < BITS; ++p) c[p] |= (uint32_t)((idx >> p) & 1) << e;      // canonical: LSB-first bit-planes
    }
#pragma unroll
    for (int p = 0; p < BITS; ++p) planes_out[(r * BITS + p) * nw + j] = c[p];
    scales_out[r * (K / 16) + 2 * j] = lut[lut_scale_offset(r, 2 * j, K, BITS)];
    scales_out[r * (K / 16) + 2 * j + 1] = lut[lut_scale_offset(r, 2 * j + 1, K, BITS)];
}

cudaError_t launch_export_lut(int bits, const PackedHeader *hdr, const uint8_t *lut_dev, int64_t N,
                              int64_t K, uint32_t *planes_out, uint8_t *scales_out, float *s_out,
                              cudaStream_t stream)
{
    const int64_t total = N * (K / 32);
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (bits == 3) export_lut_kernel<3><<<blocks, 256, 0, stream>>>(hdr, lut_dev, N, K, planes_out, scales_out, s_out);
    else export_lut_kernel<2><<<blocks, 256, 0, stream>>>(hdr, lut_dev, N, K, planes_out, scales_out, s_out);
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

// one thread per word group, as in the packer
template <int BITS>
__global__ void import_lut_kernel(const uint32_t *planes_in, const uint8_t *scales_in, int64_t N, int64_t K,
                                  uint8_t *lut)
{
    const int64_t nq = K / 128, nw = K / 32;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t quad = i >> 2;
    const int t = (int)(i & 3);
    if (quad >= N * nq) return;
    const int64_t r = quad / nq, q = quad % nq;
    uint32_t wd[BITS];
#pragma unroll
    for (int p = 0; p < BITS; ++p) wd[p] = 0u;
#pragma unroll
    for (int bb = 0; bb < 8; ++bb) {
        // weights 16 bb + 4 t .. + 3 of the 128: bits 16 (bb % 2) + 4 t .. of canonical word 4 q + bb / 2
        uint32_t c[BITS];
#pragma unroll
        for (int p = 0; p < BITS; ++p) c[p] = planes_in[(r * BITS + p) * nw + q * 4 + (bb >> 1)] >> (16 * (bb & 1) + 4 * t);
#pragma unroll
        for (int n4 = 0; n4 < 4; ++n4)
#pragma unroll
            for (int b = 0; b < BITS; ++b) {
                int word, pos;
                lut_locate<BITS>(bb, n4, b, word, pos);
                wd[word] |= ((c[b] >> n4) & 1u) << pos;
            }
    }
#pragma unroll
    for (int p = 0; p < BITS; ++p) *reinterpret_cast<uint32_t *>(lut + lut_word_offset(r, q, t, p, K, BITS)) = wd[p];
    if (t == 0) {
#pragma unroll
        for (int bb = 0; bb < 8; ++bb) lut[lut_scale_offset(r, q * 8 + bb, K, BITS)] = scales_in[r * (K / 16) + q * 8 + bb];
    }
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

cudaError_t launch_import_lut(int bits, const uint32_t *planes_in, const uint8_t *scales_in, int64_t N, int64_t K,
                              uint8_t *lut_dev, cudaStream_t stream)
{
    const int64_t total = N * (K / 128) * 4;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (bits == 3) import_lut_kernel<3><<<blocks, 256, 0, stream>>>(planes_in, scales_in, N, K, lut_dev);
    else import_lut_kernel<2><<<blocks, 256, 0, stream>>>(planes_in, scales_in, N, K, lut_dev);
    return cudaGetLastError();
}

// ------------------------------------------------------ measurement kernel

// Read-only streaming sum with 128-bit loads: the practical ceiling of a kernel that only reads (the decode
// kernels' roofline is quoted against the copy bandwidth; this number shows what a pure reader reaches).
__global__ void __launch_bounds__(512) stream_read_kernel(const uint4 *__restrict__ src, size_t n16, unsigned long long *out)
{
    uint32_t acc = 0;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n16; i += 4 * stride) {          // four independent loads in flight per thread
        const uint4 a = __ldg(src + i), b = __ldg(src + i + stride), c = __ldg(src + i + 2 * stride), d = __ldg(src + i + 3 * stride);
        acc += (a.x ^ a.y ^ a.z ^ a.w) + (b.x ^ b.y ^ b.z ^ b.w) + (c.x ^ c.y ^ c.z ^ c.w) + (d.x ^ d.y ^ d.z ^ d.w);
    }
    for (; i < n16; i += stride) {
        const uint4 a = __ldg(src + i);
        acc += a.x ^ a.y ^ a.z ^ a.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0 && acc == 0x9E3779B9u) atomicAdd(out, 1ull);     // keeps the loads alive; almost never taken
}

cudaError_t launch_stream_read(const void *src_dev, size_t bytes, void *out_dev, cudaStream_t stream)
{
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    stream_read_kernel<<<sms * 4, 512, 0, stream>>>(reinterpret_cast<const uint4 *>(src_dev), bytes / 16,
                                                    reinterpret_cast<unsigned long long *>(out_dev));
    return cudaGetLastError();
}

// --------------------------------------------------- activation quantiser

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
