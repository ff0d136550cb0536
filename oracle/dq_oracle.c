/*
 * dq_oracle.c -- plain, slow CPU oracle for the format-disaggregated quantized
 * linear layer ("Disaggregated Quantization", App. A.3 "Quantization formats",
 * Sec. 2.3, App. C.2 "Kernel specification").
 *
 * THIS IS TEST INFRASTRUCTURE.  Only the tests, the smoke check and the bench's
 * CPU-baseline leg may call it.  It shares no code, header, table or constant
 * generator with the CUDA path and is never a fallback for it.
 *
 * What it computes, in the paper's order:
 *   1. two-level scaling (App. A.3 "NVFP4-esque two-level scaling"):
 *        s   = max|W| / (6*448)                      one FP32 scale per tensor
 *        d_b = E4M3( extreme_b / (6*s) )             one FP8-E4M3 scale per 16
 *              elements along the contraction dimension
 *   2. NVFP4 (App. A.3 "NVFP4"): element code = nearest E2M1 value of
 *        x / (s*d_b), magnitudes {0,.5,1,1.5,2,3,4,6} with sign.
 *   3. LUT3 (App. A.3 "LUT formats"): the block scale carries the sign of the
 *        block's maximum-magnitude element, so that element normalises to +6;
 *        element index = nearest level of the 8-level grid; indices stored
 *        bit-planed as int32 over (N, 3, K/32) (App. C.2).
 *      LUT2 (same passage): the same rule with the 4-level grid, 2 bit-planes.
 *   4. autocast LUT3 -> NVFP4 (Sec. 2.3): re-quantise the LUT3 weights to NVFP4.
 *   5. dequantise x^ = s * d_b * level and fp64 products  Y = A^ W^T.
 *
 * Readings where the paper is silent (all stated again in the design notes):
 *   - quantiser arithmetic is FP32, round-to-nearest, reciprocal-multiply:
 *       rc6 = 1/(6*s);  t = extreme*rc6;  d = E4M3(t);  r = 1/(s*dec(d));  y = x*r
 *   - E4M3 (e4m3fn: bias 7, no inf, max 448) and E2M1 encodes are
 *     round-to-nearest-even with saturation to the largest finite value
 *   - LUT3: nearest level, a value exactly halfway goes to the lower level
 *   - equal largest magnitudes with both signs in a block: the positive one
 *     gives the scale its sign
 *   - a block whose scale rounds to zero stores zero codes (LUT3: the index of
 *     the 0.0 level); an all-zero tensor gets s = 1
 *   - bit i (LSB = 0) of word j of plane p is bit p of idx[32*j + i]
 *   - the 8 LUT3 levels are the paper's 4-decimal values rounded to fp16
 *
 * Parity pins (tests/test_oracle_*.py): E2M1 value set printed in the paper,
 * codec round trips, brute-force nearest, block-scale / absmax invariants,
 * exact round trip of representable tensors, Lloyd stationarity of the LUT3
 * grid (App. A.3: the grids minimise expected squared error), storage cost
 * b+0.5 bit, exact-integer dot products.  The paper prints no numeric example
 * of a quantised block or of a product: GEMM/GEMV values are "parity
 * unpinned" against the paper itself and pinned by exact integer arithmetic.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define DQO_BLOCK 16

/* ------------------------------------------------------------------ codecs */

/* E2M1 (1 sign, 2 exponent, 1 mantissa bit, bias 1): App. A.3 "NVFP4" prints
 * the magnitude grid {0, 0.5, 1, 1.5, 2, 3, 4, 6}. */
float dqo_e2m1_decode(uint8_t code)
{
    int sign = (code >> 3) & 1;
    int e = (code >> 1) & 3;
    int m = code & 1;
    float v = (e == 0) ? 0.5f * (float)m : ldexpf(1.0f + 0.5f * (float)m, e - 1);
    return sign ? -v : v;
}

/* Round-to-nearest-even onto the E2M1 grid, saturating at 6; the sign bit is
 * kept even when the magnitude rounds to zero; NaN gives +6 (0x7). */
uint8_t dqo_e2m1_encode(float y)
{
    if (isnan(y)) return 0x7;
    uint8_t sign = signbit(y) ? 0x8 : 0x0;
    float a = fabsf(y);
    if (a >= 6.0f) return sign | 0x7;
    int e2;                       /* a = f * 2^e2, f in [0.5, 1) */
    if (a == 0.0f) return sign;
    (void)frexpf(a, &e2);
    int E = e2 - 1;               /* a in [2^E, 2^(E+1)) */
    if (E < 0) {                  /* subnormal range: step 0.5 */
        float q = nearbyintf(a * 2.0f);          /* 0, 1 or 2 */
        if (q >= 2.0f) return sign | 0x2;        /* rounds up to 1.0 */
        return sign | (uint8_t)q;
    }
    /* normal: step 2^(E-1), q in {2,3,4} */
    float q = nearbyintf(ldexpf(a, 1 - E));
    if (q >= 4.0f) { E += 1; q = 2.0f; }
    if (E > 2) return sign | 0x7;
    return sign | (uint8_t)(((E + 1) << 1) | ((int)q - 2));
}

/* E4M3 "fn" (bias 7, 3 mantissa bits, no infinities, 0x7F/0xFF = NaN, max 448:
 * the 448 of App. A.3's  s = max|W|/(6*448)). */
float dqo_e4m3_decode(uint8_t b)
{
    int sign = b >> 7;
    int e = (b >> 3) & 0xF;
    int m = b & 7;
    float v;
    if (e == 0xF && m == 7) v = NAN;
    else if (e == 0) v = ldexpf((float)m, -9);
    else v = ldexpf(1.0f + (float)m / 8.0f, e - 7);
    return sign ? -v : v;
}

/* Round-to-nearest-even onto the E4M3 grid, saturating at +-448. */
uint8_t dqo_e4m3_encode(float t)
{
    uint8_t sign = signbit(t) ? 0x80 : 0x00;
    if (isnan(t)) return sign | 0x7F;
    float a = fabsf(t);
    if (a > 448.0f) return sign | 0x7E;
    if (a == 0.0f) return sign;
    int e2;
    (void)frexpf(a, &e2);
    int E = e2 - 1;               /* a in [2^E, 2^(E+1)) */
    if (E < -6) {                 /* subnormal: step 2^-9 */
        float q = nearbyintf(ldexpf(a, 9));      /* 0 .. 8 */
        return sign | (uint8_t)q;                /* q == 8 is 0x08 = 2^-6 */
    }
    float q = nearbyintf(ldexpf(a, 3 - E));      /* 8 .. 16 */
    if (q >= 16.0f) { E += 1; q = 8.0f; }
    return sign | (uint8_t)(((E + 7) << 3) | ((int)q - 8));
}

/* IEEE binary16 <-> float, round-to-nearest-even (codebook precision). */
float dqo_f16_decode(uint16_t h)
{
    int sign = h >> 15;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    float v;
    if (e == 0x1F) v = m ? NAN : INFINITY;
    else if (e == 0) v = ldexpf((float)m, -24);
    else v = ldexpf(1.0f + (float)m / 1024.0f, e - 15);
    return sign ? -v : v;
}

uint16_t dqo_f16_encode(float x)
{
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    if (isnan(x)) return sign | 0x7E00;
    float a = fabsf(x);
    if (a >= 65520.0f) return sign | 0x7C00;
    if (a == 0.0f) return sign;
    int e2;
    (void)frexpf(a, &e2);
    int E = e2 - 1;
    if (E < -14) {
        float q = nearbyintf(ldexpf(a, 24));     /* 0 .. 1024 */
        return sign | (uint16_t)q;
    }
    float q = nearbyintf(ldexpf(a, 10 - E));     /* 1024 .. 2048 */
    if (q >= 2048.0f) { E += 1; q = 1024.0f; }
    return sign | (uint16_t)(((E + 15) << 10) | ((int)q - 1024));
}

/* bfloat16 <-> float (activations and checkpoints are bf16). */
float dqo_bf16_decode(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

uint16_t dqo_bf16_encode(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    if (isnan(x)) return (uint16_t)((u >> 16) | 0x40);
    uint32_t lsb = (u >> 16) & 1;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* The paper's LUT3A16 grid (App. A.3 "LUT formats"), rounded to fp16. */
static const float DQO_LUT3_PAPER_GRID[8] = {
    -4.7038f, -2.8698f, -1.3696f, 0.0f, 1.2204f, 2.5285f, 4.0473f, 6.0f
};

void dqo_lut3_default_codebook(uint16_t codebook_f16[8])
{
    for (int j = 0; j < 8; ++j) codebook_f16[j] = dqo_f16_encode(DQO_LUT3_PAPER_GRID[j]);
}

/* The paper's LUT2A16 grid (App. A.3 "LUT formats": 4 levels, 2.5 bit per weight), rounded to fp16. */
static const float DQO_LUT2_PAPER_GRID[4] = { -3.6517f, 0.0f, 2.5227f, 6.0f };

void dqo_lut2_default_codebook(uint16_t codebook_f16[4])
{
    for (int j = 0; j < 4; ++j) codebook_f16[j] = dqo_f16_encode(DQO_LUT2_PAPER_GRID[j]);
}

/* ----------------------------------------------------------- global scale */

/* App. A.3: s = max|W| / (6*448); fused layers pass the concatenated matrix. */
float dqo_absmax(const float *x, int64_t rows, int64_t K, int64_t ld)
{
    float amax = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            float a = fabsf(x[r * ld + k]);
            if (a > amax) amax = a;
        }
    return amax;
}

float dqo_global_scale(float amax)
{
    if (amax == 0.0f) return 1.0f;
    return amax / 2688.0f;        /* 6 * 448 */
}

/* ------------------------------------------------------------- quantisers */

/* NVFP4 round-to-nearest of a rows x K matrix (row stride ld, K % 16 == 0)
 * with a given tensor scale s (weights: dqo_global_scale; activations: the
 * static input scale of App. A.3 "NVFP4").
 *   codes  : uint8[rows][K/2], element 2j in the low nibble, 2j+1 in the high
 *   scales : uint8[rows][K/16], E4M3, sign bit clear                        */
void dqo_quant_nvfp4(const float *x, int64_t rows, int64_t K, int64_t ld, float s,
                     uint8_t *codes, uint8_t *scales)
{
    const float rc6 = 1.0f / (6.0f * s);
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < K / DQO_BLOCK; ++b) {
            const float *xb = x + r * ld + b * DQO_BLOCK;
            float a = 0.0f;
            for (int i = 0; i < DQO_BLOCK; ++i) {
                float v = fabsf(xb[i]);
                if (v > a) a = v;
            }
            float t = a * rc6;
            uint8_t d = dqo_e4m3_encode(t);
            scales[r * (K / DQO_BLOCK) + b] = d;
            uint8_t c[DQO_BLOCK];
            if ((d & 0x7F) == 0) {
                for (int i = 0; i < DQO_BLOCK; ++i) c[i] = 0;
            } else {
                float rr = 1.0f / (s * dqo_e4m3_decode(d));
                for (int i = 0; i < DQO_BLOCK; ++i) {
                    float y = xb[i] * rr;
                    c[i] = dqo_e2m1_encode(y);
                }
            }
            uint8_t *out = codes + r * (K / 2) + b * (DQO_BLOCK / 2);
            for (int i = 0; i < DQO_BLOCK / 2; ++i)
                out[i] = (uint8_t)(c[2 * i] | (c[2 * i + 1] << 4));
        }
    }
}

/* LUT3 round-to-nearest (K % 32 == 0).
 *   codebook_f16 : 8 fp16 levels, strictly increasing, containing 0 and 6
 *   planes : uint32[rows][3][K/32] bit-planes (App. C.2)
 *   scales : uint8[rows][K/16] signed E4M3, zero stored as 0x00            */
void dqo_quant_lut3(const float *x, int64_t rows, int64_t K, int64_t ld, float s,
                    const uint16_t codebook_f16[8], uint32_t *planes, uint8_t *scales)
{
    float G[8], T[7];
    int zero_idx = 0;
    for (int j = 0; j < 8; ++j) {
        G[j] = dqo_f16_decode(codebook_f16[j]);
        if (G[j] == 0.0f) zero_idx = j;
    }
    for (int j = 0; j < 7; ++j) T[j] = (G[j] + G[j + 1]) * 0.5f;   /* exact in fp32 */
    const float rc6 = 1.0f / (6.0f * s);
    const int64_t W = K / 32;
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        uint32_t *pl = planes + r * 3 * W;
        for (int64_t j = 0; j < 3 * W; ++j) pl[j] = 0;
        for (int64_t b = 0; b < K / DQO_BLOCK; ++b) {
            const float *xb = x + r * ld + b * DQO_BLOCK;
            /* the block's maximum-magnitude element, with its sign */
            float m = xb[0];
            for (int i = 1; i < DQO_BLOCK; ++i) {
                float v = xb[i];
                if (fabsf(v) > fabsf(m) || (fabsf(v) == fabsf(m) && v > m)) m = v;
            }
            float t = m * rc6;
            uint8_t d = dqo_e4m3_encode(t);
            if ((d & 0x7F) == 0) d = 0;
            scales[r * (K / DQO_BLOCK) + b] = d;
            for (int i = 0; i < DQO_BLOCK; ++i) {
                int idx = zero_idx;
                if (d != 0) {
                    float rr = 1.0f / (s * dqo_e4m3_decode(d));
                    float y = xb[i] * rr;
                    idx = 0;
                    for (int j = 0; j < 7; ++j) idx += (y > T[j]);
                }
                int64_t k = b * DQO_BLOCK + i;
                for (int p = 0; p < 3; ++p)
                    pl[p * W + k / 32] |= (uint32_t)((idx >> p) & 1) << (k % 32);
            }
        }
    }
}

/* LUT2 round-to-nearest (App. A.3 "LUT formats"; K % 32 == 0): the same rule as LUT3 with the
 * 4-level grid -- signed block scale from the block's maximum-magnitude element (so that element
 * normalises to +6), nearest level, a value exactly halfway goes to the lower level.
 *   codebook_f16 : 4 fp16 levels, strictly increasing, containing 0 and 6
 *   planes : uint32[rows][2][K/32] bit-planes (App. C.2 storage with b = 2)
 *   scales : uint8[rows][K/16] signed E4M3, zero stored as 0x00            */
void dqo_quant_lut2(const float *x, int64_t rows, int64_t K, int64_t ld, float s,
                    const uint16_t codebook_f16[4], uint32_t *planes, uint8_t *scales)
{
    float G[4], T[3];
    int zero_idx = 0;
    for (int j = 0; j < 4; ++j) {
        G[j] = dqo_f16_decode(codebook_f16[j]);
        if (G[j] == 0.0f) zero_idx = j;
    }
    for (int j = 0; j < 3; ++j) T[j] = (G[j] + G[j + 1]) * 0.5f;   /* exact in fp32 */
    const float rc6 = 1.0f / (6.0f * s);
    const int64_t W = K / 32;
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        uint32_t *pl = planes + r * 2 * W;
        for (int64_t j = 0; j < 2 * W; ++j) pl[j] = 0;
        for (int64_t b = 0; b < K / DQO_BLOCK; ++b) {
            const float *xb = x + r * ld + b * DQO_BLOCK;
            float m = xb[0];
            for (int i = 1; i < DQO_BLOCK; ++i) {
                float v = xb[i];
                if (fabsf(v) > fabsf(m) || (fabsf(v) == fabsf(m) && v > m)) m = v;
            }
            float t = m * rc6;
            uint8_t d = dqo_e4m3_encode(t);
            if ((d & 0x7F) == 0) d = 0;
            scales[r * (K / DQO_BLOCK) + b] = d;
            for (int i = 0; i < DQO_BLOCK; ++i) {
                int idx = zero_idx;
                if (d != 0) {
                    float rr = 1.0f / (s * dqo_e4m3_decode(d));
                    float y = xb[i] * rr;
                    idx = 0;
                    for (int j = 0; j < 3; ++j) idx += (y > T[j]);
                }
                int64_t k = b * DQO_BLOCK + i;
                for (int p = 0; p < 2; ++p)
                    pl[p * W + k / 32] |= (uint32_t)((idx >> p) & 1) << (k % 32);
            }
        }
    }
}

/* Sec. 2.3 autocast: the NVFP4 view of LUT3 weights.  Each level maps to its
 * nearest E2M1 value; a negative block scale flips the element signs and the
 * NVFP4 block scale is |d_b| (the LUT3 block extreme is exactly 6*|d_b|*s, so
 * NVFP4's own block-scale rule gives |d_b| back); the tensor scale is kept. */
void dqo_autocast_lut3_to_nvfp4(const uint32_t *planes, const uint8_t *lut_scales,
                                int64_t rows, int64_t K, const uint16_t codebook_f16[8],
                                uint8_t *codes, uint8_t *scales)
{
    uint8_t map[8];
    for (int j = 0; j < 8; ++j) map[j] = dqo_e2m1_encode(dqo_f16_decode(codebook_f16[j]));
    const int64_t W = K / 32;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t k = 0; k < K; k += 2) {
            uint8_t c2[2];
            for (int u = 0; u < 2; ++u) {
                int64_t kk = k + u;
                int idx = 0;
                for (int p = 0; p < 3; ++p)
                    idx |= (int)((planes[(r * 3 + p) * W + kk / 32] >> (kk % 32)) & 1u) << p;
                uint8_t d = lut_scales[r * (K / DQO_BLOCK) + kk / DQO_BLOCK];
                uint8_t c = map[idx];
                if ((d & 0x80) && (c & 0x7)) c ^= 0x8;
                if ((d & 0x7F) == 0) c = 0;
                c2[u] = c;
            }
            codes[r * (K / 2) + k / 2] = (uint8_t)(c2[0] | (c2[1] << 4));
        }
        for (int64_t b = 0; b < K / DQO_BLOCK; ++b)
            scales[r * (K / DQO_BLOCK) + b] = lut_scales[r * (K / DQO_BLOCK) + b] & 0x7F;
    }
}

/* ------------------------------------------- activation processing + quantiser */

/* The paper's prefill stack fuses activation processing with the NVFP4 activation quantiser (App. C.1
 * "we fuse compatible projections and activation processing"; the per-component latency table counts the
 * quantiser inside "norms").  It gives no arithmetic for the fused operators.  Reading used here: the fused
 * operator produces exactly what the two unfused steps would -- the processed activation rounded to bf16
 * (the dtype activations travel in), then dqo_quant_nvfp4 with the static input scale -- with the fp32
 * arithmetic of the processing step fixed as follows so that it can be reproduced bit for bit:
 *
 * RMSNorm:  ss  = sum_k x_k^2      in fp32: x_k^2 summed in order inside each 16-element block, the block sums
 *                                  combined 32 blocks at a time by a balanced binary tree (neighbours first), the
 *                                  group sums added in increasing order
 *           r   = 1 / sqrt(ss / K + eps)                      (fp32 divide, add, square root, reciprocal)
 *           h_k = bf16( (x_k * r) * gamma_k )
 * SiLU(gate) * up:  silu(g) = g / (1 + e),  e = 2^t,  t = clamp(g * (-log2 e), -126, 126), evaluated as
 *           n = rint(t), f = fma(g, -L_hi, -n) then f = fma(g, -L_lo, f) with log2 e = L_hi + L_lo (so that the
 *           reduction keeps full precision for large |g|), p = degree-7 polynomial in f with the Taylor
 *           coefficients of 2^f (fused multiply-adds, highest degree first), e = p * 2^n;   h = bf16( silu(g) * u ).
 * Outputs are fp32 arrays holding bf16 values. */
static float dqo_round_to_bf16(float v) { return dqo_bf16_decode(dqo_bf16_encode(v)); }

void dqo_rmsnorm_bf16(const float *x, int64_t rows, int64_t K, int64_t ld, const float *gamma, float eps, float *h)
{
    const int64_t nb = K / DQO_BLOCK;
    const int64_t ngroups = (nb + 31) / 32;
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const float *xr = x + r * ld;
        float total = 0.0f;
        for (int64_t g = 0; g < ngroups; ++g) {
            float v[32];
            for (int i = 0; i < 32; ++i) {
                int64_t b = g * 32 + i;
                float bs = 0.0f;
                if (b < nb)
                    for (int k = 0; k < DQO_BLOCK; ++k) { float sq = xr[b * DQO_BLOCK + k] * xr[b * DQO_BLOCK + k]; bs = bs + sq; }
                v[i] = bs;
            }
            for (int step = 1; step < 32; step *= 2)          /* neighbours first */
                for (int i = 0; i < 32; i += 2 * step) v[i] = v[i] + v[i + step];
            total = total + v[0];
        }
        float mean = total / (float)K;
        float rr = 1.0f / sqrtf(mean + eps);
        for (int64_t k = 0; k < K; ++k) {
            float t = xr[k] * rr;
            h[r * K + k] = dqo_round_to_bf16(t * gamma[k]);
        }
    }
}

float dqo_silu_f32(float g)
{
    static const float C[8] = { 1.0f, 0.6931471805599453f, 0.2402265069591007f, 0.05550410866482158f,
                                0.009618129107628477f, 0.0013333558146428443f, 0.00015403530393381608f,
                                1.5252733804059841e-05f };
    const float L_HI = 1.4426950216293335f, L_LO = 1.925963033500256e-08f;      /* log2(e) = L_HI + L_LO */
    float t = g * -L_HI;
    float n = nearbyintf(fminf(fmaxf(t, -126.0f), 126.0f));
    float f = fmaf(g, -L_HI, -n);
    f = fmaf(g, -L_LO, f);
    f = fminf(fmaxf(f, -1.0f), 1.0f);                 /* only clamped arguments (|g| > 87) leave [-0.5, 0.5] */
    float p = C[7];
    for (int i = 6; i >= 0; --i) p = fmaf(p, f, C[i]);
    float e = ldexpf(p, (int)n);
    return g / (1.0f + e);
}

/* gate_up: rows x 2F (gate in columns [0, F), up in [F, 2F): the output of a fused gate/up projection) */
void dqo_silu_mul_bf16(const float *gate_up, int64_t rows, int64_t F, int64_t ld, float *h)
{
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < F; ++k) {
            float sv = dqo_silu_f32(gate_up[r * ld + k]);
            h[r * F + k] = dqo_round_to_bf16(sv * gate_up[r * ld + F + k]);
        }
}

/* ------------------------------------------------------------ dequantise */

/* x^ = s * d_b * level, evaluated in double from exactly representable factors. */
void dqo_dequant_nvfp4(const uint8_t *codes, const uint8_t *scales, int64_t rows, int64_t K,
                       float s, double *out)
{
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = codes[r * (K / 2) + k / 2];
            uint8_t c = (k & 1) ? (byte >> 4) : (byte & 0xF);
            double d = (double)dqo_e4m3_decode(scales[r * (K / DQO_BLOCK) + k / DQO_BLOCK]);
            out[r * K + k] = (double)s * d * (double)dqo_e2m1_decode(c);
        }
}

void dqo_dequant_lut3(const uint32_t *planes, const uint8_t *scales, int64_t rows, int64_t K,
                      float s, const uint16_t codebook_f16[8], double *out)
{
    const int64_t W = K / 32;
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            int idx = 0;
            for (int p = 0; p < 3; ++p)
                idx |= (int)((planes[(r * 3 + p) * W + k / 32] >> (k % 32)) & 1u) << p;
            double d = (double)dqo_e4m3_decode(scales[r * (K / DQO_BLOCK) + k / DQO_BLOCK]);
            out[r * K + k] = (double)s * d * (double)dqo_f16_decode(codebook_f16[idx]);
        }
}

void dqo_dequant_lut2(const uint32_t *planes, const uint8_t *scales, int64_t rows, int64_t K,
                      float s, const uint16_t codebook_f16[4], double *out)
{
    const int64_t W = K / 32;
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            int idx = 0;
            for (int p = 0; p < 2; ++p)
                idx |= (int)((planes[(r * 2 + p) * W + k / 32] >> (k % 32)) & 1u) << p;
            double d = (double)dqo_e4m3_decode(scales[r * (K / DQO_BLOCK) + k / DQO_BLOCK]);
            out[r * K + k] = (double)s * d * (double)dqo_f16_decode(codebook_f16[idx]);
        }
}

/* -------------------------------------------------------------- products */

/* Y[m][n] = sum_k A[m][k] * W[n][k]  and  Sabs[m][n] = sum_k |A[m][k] * W[n][k]|
 * in double, k ascending (y = x W^T, Sec. 1.1).  Sabs may be NULL. */
void dqo_matmul_nt(const double *A, int64_t M, int64_t K, const double *W, int64_t N,
                   double *Y, double *Sabs)
{
    #pragma omp parallel for schedule(static)
    for (int64_t mn = 0; mn < M * N; ++mn) {
        int64_t m = mn / N, n = mn % N;
        double acc = 0.0, sab = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double p = A[m * K + k] * W[n * K + k];
            acc += p;
            sab += fabs(p);
        }
        Y[mn] = acc;
        if (Sabs) Sabs[mn] = sab;
    }
}

int dqo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
