// Device routines shared by the quantising kernels: format converts and the NVFP4 round-to-nearest of one
// 16-element block (App. A.3 "NVFP4-esque two-level scaling", "NVFP4").  fp32 arithmetic with explicit
// round-to-nearest intrinsics so the compiler cannot contract or reorder it:
//   t = extreme * rc6;  d = E4M3(t);  r = 1/(s * dec(d));  y = x * r
#pragma once

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

// SiLU(g) = g / (1 + exp(-g)) in a fixed fp32 sequence (the same one a CPU evaluation can follow bit for bit):
//   exp(-g) = 2^t, t = -g log2(e): n = rint(t clamped to +-126), f = fma(g, -L_hi, -n), f = fma(g, -L_lo, f),
//   p = degree-7 Taylor polynomial of 2^f by fused multiply-adds, e = p * 2^n;  silu = g / (1 + e) by IEEE divide.
__device__ __forceinline__ float silu_f32(float g)
{
    const float L_HI = 1.4426950216293335f, L_LO = 1.925963033500256e-08f;      // log2(e) = L_HI + L_LO
    const float t = __fmul_rn(g, -L_HI);
    const float n = rintf(fminf(fmaxf(t, -126.0f), 126.0f));
    float f = __fmaf_rn(g, -L_HI, -n);
    f = __fmaf_rn(g, -L_LO, f);
    f = fminf(fmaxf(f, -1.0f), 1.0f);
    float p = 1.5252733804059841e-05f;
    p = __fmaf_rn(p, f, 0.00015403530393381608f);
    p = __fmaf_rn(p, f, 0.0013333558146428443f);
    p = __fmaf_rn(p, f, 0.009618129107628477f);
    p = __fmaf_rn(p, f, 0.05550410866482158f);
    p = __fmaf_rn(p, f, 0.2402265069591007f);
    p = __fmaf_rn(p, f, 0.6931471805599453f);
    p = __fmaf_rn(p, f, 1.0f);
    const float e = __fmul_rn(p, __int_as_float(((int)n + 127) << 23));
    return __fdiv_rn(g, __fadd_rn(1.0f, e));
}

// two floats -> packed bf16 pair, round to nearest even, `lo` in the low half
__device__ __forceinline__ uint32_t pack_bf16_rn(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// h = bf16( SiLU(g) * u ) on packed bf16 pairs
__device__ __forceinline__ uint32_t silu_mul_bf16x2(uint32_t g2, uint32_t u2)
{
    const float lo = __fmul_rn(silu_f32(__uint_as_float(g2 << 16)), __uint_as_float(u2 << 16));
    const float hi = __fmul_rn(silu_f32(__uint_as_float(g2 & 0xFFFF0000u)), __uint_as_float(u2 & 0xFFFF0000u));
    return pack_bf16_rn(lo, hi);
}

}  // namespace dq
