/*
 * dq.h -- C ABI of the format-disaggregated quantized linear layer for NVIDIA
 * B200 (sm_100a).
 *
 * One stored weight matrix W (N x K, out-features x in-features, K contiguous)
 * is packed once and then served by two phase-specific kernels ("Disaggregated
 * Quantization", Sec. 2.3 and Fig. 2b): prefill runs a block-scaled NVFP4 x
 * NVFP4 GEMM on tensor cores after quantising the bf16 activations on the fly,
 * decode runs a weight-only LUT3 mat-vec against raw bf16 activations.
 *
 * Conventions for every entry point
 *   - returns a dq_status code, never throws, aborts or exits;
 *   - pointers named *_dev are device pointers on the current CUDA device,
 *     pointers named *_host are host pointers; the caller owns every buffer;
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream); work is
 *     enqueued on it and the call returns without synchronising;
 *   - nothing is allocated on the device; scratch comes from the caller;
 *   - shapes: K % 128 == 0, N % 16 == 0, and K <= 32768 for a handle that holds a
 *     LUT encoding (else DQ_ERR_SHAPE); row strides in
 *     elements, multiples of 8; device pointers 16-byte aligned, `packed_dev`
 *     and `workspace_dev` 1024-byte aligned (else DQ_ERR_ALIGN);
 *   - a handle belongs to the device that was current when it was packed; calls that
 *     use it with another device current return DQ_ERR_INVALID_ARG;
 *   - NaN/Inf in tensors give unspecified values, never a fault;
 *   - the device must be compute capability 10.0 (else DQ_ERR_ARCH).
 */
#ifndef DQ_H_
#define DQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dq_weights dq_weights;   /* opaque host-side handle */

enum dq_status {
    DQ_OK = 0,
    DQ_ERR_INVALID_ARG = 1,
    DQ_ERR_SHAPE = 2,
    DQ_ERR_ALIGN = 3,
    DQ_ERR_WORKSPACE = 4,
    DQ_ERR_ARCH = 5,
    DQ_ERR_CUDA = 6,
    DQ_ERR_TIMEOUT = 7,
    DQ_ERR_INTERNAL = 8
};

/* weight encodings held by a handle (bit mask) */
enum dq_format {
    DQ_FMT_NVFP4 = 1,            /* NVFP4 round-to-nearest of the master weights   */
    DQ_FMT_LUT3 = 2,             /* LUT3 round-to-nearest of the master weights    */
    DQ_FMT_NVFP4_FROM_LUT3 = 4,  /* NVFP4 view re-quantised from the LUT3 codes    */
    DQ_FMT_LUT2 = 8              /* LUT2 round-to-nearest of the master weights    */
};

enum dq_dtype { DQ_DT_BF16 = 0, DQ_DT_FP32 = 1 };

/* Library version (major*10000 + minor*100 + patch). */
int dq_version(void);
const char *dq_status_string(int status);

/*
 * Size of the device buffer dq_pack_weights needs for the requested encodings.
 * Storage follows App. A.3 "Storage cost": NVFP4 4.5 bit, LUT3 3.5 bit and LUT2 2.5 bit
 * per weight (codes plus one FP8 scale per 16 weights), plus a 1 KiB header, padding of
 * the NVFP4 scale tiles to 256 rows and of LUT rows to a multiple of 1024 weights.
 * `formats` must contain at most one of DQ_FMT_NVFP4 / DQ_FMT_NVFP4_FROM_LUT3;
 * DQ_FMT_NVFP4_FROM_LUT3 implies DQ_FMT_LUT3.
 */
int dq_packed_bytes(int64_t N, int64_t K, unsigned formats, size_t *bytes_host);

/*
 * Pack a (fused) weight matrix (App. A.3 "NVFP4-esque two-level scaling",
 * "NVFP4", "LUT formats"; App. C.2 storage).
 *   tensor scale  s = max|W| / (6*448) over the whole matrix given (layers an
 *                 engine fuses are passed concatenated so they share s);
 *   block scale   d_b = E4M3(extreme_b / (6 s)) per 16 weights along K; for LUT3
 *                 it carries the sign of the block's maximum-magnitude weight;
 *   NVFP4 code    nearest E2M1 value of w / (s d_b);
 *   LUT3 index    nearest level of the 8-entry fp16 codebook, stored bit-planed;
 *   LUT2 index    nearest level of the paper's 4-level LUT2A16 grid {-3.6517, 0, 2.5227, 6}
 *                 rounded to fp16, same signed block scale rule.
 *   DQ_FMT_NVFP4_FROM_LUT3 derives the NVFP4 codes from the LUT3 indices
 *   (Sec. 2.3 autocast) instead of from W.
 * W_dev: device, row-major, row stride ldw elements, dtype per `w_dtype`.
 * lut3_codebook_f16_host: 8 fp16 bit patterns, strictly increasing, containing
 *   0.0 and with maximum 6.0; NULL selects the paper's LUT3A16 grid rounded to fp16.
 * packed_dev: device buffer of at least dq_packed_bytes bytes; must stay alive
 *   and unmodified while the handle is used.
 * *out_host receives a handle owned by the caller (dq_free_weights). The handle
 * is immutable and may be used from several streams once the pack has finished
 * on `stream`.
 */
int dq_pack_weights(const void *W_dev, int w_dtype, int64_t N, int64_t K, int64_t ldw,
                    unsigned formats, const uint16_t *lut3_codebook_f16_host,
                    void *packed_dev, size_t packed_bytes, void *stream,
                    dq_weights **out_host);

/* Frees the host handle only; the packed device buffer belongs to the caller. */
int dq_free_weights(dq_weights *w);

/* Scratch dq_prefill_linear needs for M tokens: NVFP4 activation codes + scales, and for a
 * handle packed with DQ_FMT_LUT3 only also the NVFP4 view of the weights (see below). */
int dq_prefill_workspace_bytes(const dq_weights *w, int64_t M, size_t *bytes_host);

/*
 * Prefill linear (Sec. 1.1 "compute-bound prefill", Sec. 2.3, App. C.1):
 *   Y[m][n] = bf16( sum_k A^[m][k] * W^[n][k] ),
 * where A^ is the NVFP4 round-to-nearest of A with the static per-tensor input
 * scale `act_global_scale` (App. A.3 "NVFP4": s_a in  a^ = s_a * d_b * e2m1) and
 * W^ the handle's NVFP4 weights; block-scaled FP4 tensor-core GEMM, fp32
 * accumulation.
 * A handle packed with DQ_FMT_LUT3 alone stores one 3.5-bit matrix for both phases
 * (Sec. 2.3 "format-disaggregated LUT3"; the paper describes this on-the-fly cast but
 * does not build it): every prefill call first casts the LUT3 codes to NVFP4 into the
 * workspace (integer code map, block scale |d_b|, same tensor scale; the result equals
 * the DQ_FMT_NVFP4_FROM_LUT3 view bit for bit) and then runs the same GEMM.  The cast
 * is part of dq_prefill_quantize when the two stages are called separately.
 * A_dev: M x K bf16, row stride lda; Y_dev: M x N bf16, row stride ldy.
 * act_global_scale must be finite and > 0.  M >= 1.
 * workspace_dev: at least dq_prefill_workspace_bytes(M) bytes, private to this
 * call until it has finished on `stream`.
 */
int dq_prefill_linear(const dq_weights *w, const void *A_dev, int64_t M, int64_t lda,
                      float act_global_scale, void *Y_dev, int64_t ldy,
                      void *workspace_dev, size_t workspace_bytes, void *stream);

/*
 * The two stages of dq_prefill_linear as separate calls, for callers that time or
 * overlap them: dq_prefill_quantize writes the NVFP4 activations (App. A.3 "NVFP4",
 * static input scale) into the workspace, dq_prefill_gemm multiplies them with the
 * handle's NVFP4 weights (Sec. 2.3).  Arguments as in dq_prefill_linear; the same
 * M, workspace and act_global_scale must be passed to both.
 */
int dq_prefill_quantize(const dq_weights *w, const void *A_dev, int64_t M, int64_t lda,
                        float act_global_scale, void *workspace_dev, size_t workspace_bytes,
                        void *stream);
int dq_prefill_gemm(const dq_weights *w, int64_t M, float act_global_scale, void *Y_dev, int64_t ldy,
                    const void *workspace_dev, size_t workspace_bytes, void *stream);

/*
 * The activation stage of the prefill linear fused with the operator in front of it, so that the normalised or gated
 * activation never travels through HBM (App. C.1: the paper's prefill stack fuses activation processing with the
 * activation quantiser; its per-component latency table counts the quantiser inside "norms").  Each call replaces
 * dq_prefill_quantize and is followed by dq_prefill_gemm with the same M, workspace and act_global_scale.
 *   dq_prefill_rmsnorm_quantize:  A = bf16( X * r * gamma ),  r = 1 / sqrt(mean_k(X^2) + eps) per row,
 *       X_dev: M x K bf16 (row stride ldx), gamma_dev: K bf16 (16-byte aligned), eps >= 0; K <= 131072.
 *   dq_prefill_silu_mul_quantize: A = bf16( SiLU(G) * U ),  SiLU(g) = g / (1 + exp(-g)),
 *       GU_dev: M x 2K bf16 (row stride ldgu >= 2K), G in columns [0, K), U in [K, 2K): the output of a fused
 *       gate/up projection feeding the down projection `w`.
 * A is what the two unfused steps would produce (the operator's result rounded to bf16); it is quantised exactly as
 * dq_prefill_quantize quantises (App. A.3 "NVFP4", static input scale).  The fp32 arithmetic of r and of exp is
 * fixed (stated at the top of csrc/dq_fused_quant.cu), so codes and scales are reproducible bit for bit.
 */
int dq_prefill_rmsnorm_quantize(const dq_weights *w, const void *X_dev, int64_t M, int64_t ldx,
                                const void *gamma_dev, float eps, float act_global_scale,
                                void *workspace_dev, size_t workspace_bytes, void *stream);
int dq_prefill_silu_mul_quantize(const dq_weights *w, const void *GU_dev, int64_t M, int64_t ldgu,
                                 float act_global_scale, void *workspace_dev, size_t workspace_bytes,
                                 void *stream);

/*
 * The gate/up projection of a gated FFN with the gating and the next layer's activation quantiser in the GEMM's
 * epilogue (App. C.1: activation processing fused with the quantiser; Sec. 2.3 prefill path):
 *   H = bf16( SiLU(G) * U ),  [G | U] = bf16( A^ W_gate_up^T ),   out_workspace <- NVFP4(H) with out_global_scale,
 * i.e. what dq_prefill_gemm on w_gate_up followed by dq_prefill_silu_mul_quantize for w_down produces, without the
 * M x 2F bf16 matrix ever going to memory.  Call order for the whole FFN:
 *   dq_prefill_quantize (or dq_prefill_rmsnorm_quantize) for w_gate_up into `workspace`, this call,
 *   dq_prefill_gemm(w_down, M, out_global_scale, Y, ldy, out_workspace, ...).
 * w_gate_up: 2F x K, one tensor (one global scale), with its rows INTERLEAVED so that a 256-row tile holds gate and
 *   up of the same 128 features: row 256 t + 128 h + 64 p + j (h, p in {0, 1}, j < 64) is the gate (p = 0) or up
 *   (p = 1) row of feature 128 t + 64 h + j.  The caller permutes the rows before dq_pack_weights; the handle does
 *   not record the order, and the same handle passed to dq_prefill_gemm gives the columns in this order.
 * w_down: N_out x F (F a multiple of 128, as every packed K); only its shape, and for a DQ_FMT_LUT3-only handle its
 *   call-time NVFP4 cast, are used here.  w_gate_up's N must equal 2 * w_down's K, else DQ_ERR_SHAPE.
 * workspace: the quantised input, as for dq_prefill_gemm(w_gate_up, M, act_global_scale, ...).
 * out_workspace: at least dq_prefill_workspace_bytes(w_down, M) bytes, 1024-byte aligned, not overlapping
 *   `workspace` (DQ_ERR_INVALID_ARG); written by this call, then read by dq_prefill_gemm(w_down, ...).
 * Arithmetic: G and U are rounded to bf16 exactly as dq_prefill_gemm would store them, SiLU and the quantiser are those
 * of dq_prefill_silu_mul_quantize; for M > 128 codes and scales equal the two-call path bit for bit.
 */
int dq_prefill_gemm_silu_mul_quantize(const dq_weights *w_gate_up, int64_t M, float act_global_scale,
                                      const void *workspace_dev, size_t workspace_bytes,
                                      const dq_weights *w_down, float out_global_scale,
                                      void *out_workspace_dev, size_t out_workspace_bytes, void *stream);

/*
 * dq_prefill_linear without a caller-provided workspace.  (The paper has no counterpart: this
 * entry point exists for integration, not for the method.)
 * It is meant for callers that cannot allocate device memory where they call from -- an engine
 * whose memory pool already owns all of HBM, code running inside another process's allocator
 * regime, or a thread that must not hit the device-wide synchronisation inside cudaMalloc and
 * cudaFree.  The scratch is an array built into the library (8 MiB per GPU that loads it, held
 * until the process exits); no cudaMalloc, cudaFree or allocating library routine is called.
 * Limit: dq_prefill_workspace_bytes(w, M) must not exceed 8 MiB (8388608 bytes), i.e. roughly
 * M * K <= 14.9 M elements; larger problems return DQ_ERR_WORKSPACE and nothing is launched.
 * The first call on a device looks up the array's device address (once per device, with that
 * device current); make that first call before starting any stream capture.
 * All calls on a device share the one array: two calls whose GPU work overlaps (different
 * streams without ordering) race on it and give wrong results; calls ordered on one stream, or
 * by events, are safe.  The array keeps the previous call's contents; the call clears the part
 * it reads without rewriting.
 * Other arguments, results and status codes as dq_prefill_linear.
 */
int dq_prefill_linear_static(const dq_weights *w, const void *A_dev, int64_t M, int64_t lda,
                             float act_global_scale, void *Y_dev, int64_t ldy, void *stream);

/*
 * Decode linear (Sec. 1.1 "memory-bound decode", App. C.2 "Kernel specification"):
 *   Y[b][n] = bf16( sum_k X[b][k] * W~[n][k] ),  W~ = s * d_b * codebook[idx],
 * a weight-only mat-vec / skinny GEMM on the handle's LUT3 weights with raw bf16
 * activations.  1 <= B <= 64.
 * Arithmetic: the products codebook[idx] * x are formed exactly (fp16 levels and the
 * activations, scaled by one power of two into fp16, on tensor cores) and summed in fp32 per
 * 16-weight block; the block sum is multiplied by d_b and accumulated in fp32; s is applied to
 * the total.  Nothing is rounded before the fp32 accumulation, so the error per output is a few
 * fp32 rounding errors of sum_k |x w| plus the bf16 rounding of the result, for any activation
 * pattern.  An activation more than 2^28 times smaller in magnitude than the largest activation
 * it shares a power-of-two scale with loses low bits or reads as zero: that is the largest of the
 * same pass (up to eight rows of X), or, for batches above 8 on matrices of 8192 rows and more (4096 and
 * more from batch 16 on), of the same 1024-element slice of K of the same pass (up to 32 rows of X).
 * X_dev: B x K bf16, row stride ldx; Y_dev: B x N bf16, row stride ldy.
 */
int dq_decode_linear(const dq_weights *w, const void *X_dev, int64_t B, int64_t ldx,
                     void *Y_dev, int64_t ldy, void *stream);

/*
 * The same decode on the handle's LUT2 weights (App. A.3 "LUT formats": 4 levels, 2.5 bit per
 * weight; App. C.2; Table 1's LUT2 rows).  Needs DQ_FMT_LUT2 in the handle.  Arguments, arithmetic
 * and limits as dq_decode_linear.
 */
int dq_decode_linear_lut2(const dq_weights *w, const void *X_dev, int64_t B, int64_t ldx,
                          void *Y_dev, int64_t ldy, void *stream);

/*
 * The same decode on the handle's NVFP4 view (weight-only NVFP4A16, Sec. 2.3 and Table 1
 * "format-disaggregated NVFP4": one stored 4.5-bit matrix serves the tensor-core prefill and
 * this mat-vec):
 *   Y[b][n] = bf16( sum_k X[b][k] * W^[n][k] ),  W^ = s * d_b * e2m1(code),
 * raw bf16 activations, fp32 accumulation.  Needs DQ_FMT_NVFP4 or DQ_FMT_NVFP4_FROM_LUT3 in the
 * handle (DQ_ERR_INVALID_ARG otherwise).  Arguments and limits as dq_decode_linear.
 */
int dq_decode_linear_nvfp4(const dq_weights *w, const void *X_dev, int64_t B, int64_t ldx,
                           void *Y_dev, int64_t ldy, void *stream);

/* ---- host-buffer entry points (the paper has no counterpart; they exist to use and to measure the path
 *      end to end through this interface, copies included) ---- */

/*
 * dq_prefill_linear on host memory: A_host (M x K bf16, row stride lda) is copied to the device, the
 * prefill linear runs, Y_host (M x N bf16, row stride ldy) receives the result.  M is cut into row
 * chunks; the copy in of the next chunk and the copy out of the previous one overlap the kernels of the
 * current one on two internal streams per device (created at the first call on that device, which
 * therefore must not happen during a stream capture; these calls are not capturable at all).
 * A_host and Y_host should be pinned (cudaHostAlloc / cudaHostRegister), else the copies serialise.
 * staging_dev: caller-owned device buffer of at least dq_prefill_host_staging_bytes(w, M) bytes
 * (device copies of A and Y plus the prefill workspace of one chunk), 1024-byte aligned.
 * On return everything is queued; `stream` is complete when Y_host is.  All calls on one device share
 * the internal streams and events: issue them from one thread, ordered on the caller's streams.
 */
int dq_prefill_host_staging_bytes(const dq_weights *w, int64_t M, size_t *bytes_host);
int dq_prefill_linear_host(const dq_weights *w, const void *A_host, int64_t M, int64_t lda,
                           float act_global_scale, void *Y_host, int64_t ldy, void *staging_dev,
                           size_t staging_bytes, void *stream);

/*
 * dq_decode_linear on host memory (X_host B x K, Y_host B x N, bf16): copy in, mat-vec, copy out on
 * `stream`.  staging_dev: at least roundup(2*B*K, 1024) + 2*B*N bytes, 1024-byte aligned.
 */
int dq_decode_linear_host(const dq_weights *w, const void *X_host, int64_t B, int64_t ldx, void *Y_host,
                          int64_t ldy, void *staging_dev, size_t staging_bytes, void *stream);

/* ---- parity hooks: canonical encodings, compared bit for bit with the oracle ---- */

/*
 * Copy one encoding of the handle into canonical layout (all device pointers):
 *   DQ_FMT_NVFP4 / DQ_FMT_NVFP4_FROM_LUT3:
 *     codes  uint8[N][K/2]  element 2j in the low nibble, 2j+1 in the high nibble,
 *            code = sign<<3 | index into {0,.5,1,1.5,2,3,4,6} (App. A.3 "NVFP4")
 *     scales uint8[N][K/16] E4M3
 *   DQ_FMT_LUT3 (b = 3) / DQ_FMT_LUT2 (b = 2):
 *     codes  uint32[N][b][K/32] bit-planes (App. C.2): bit i (LSB = 0) of word j of
 *            plane p is bit p of the index of weight 32*j + i
 *     scales uint8[N][K/16] signed E4M3, zero stored as 0x00
 *   global_scale_dev: one float, the tensor scale s.
 */
int dq_export_canonical(const dq_weights *w, unsigned format, void *codes_dev, void *scales_dev,
                        float *global_scale_dev, void *stream);

/*
 * The inverse: build a handle from canonical encodings (layouts as above, device pointers), e.g.
 * weights quantised elsewhere with the same formats (App. A.3).  `formats` as in dq_pack_weights:
 * DQ_FMT_NVFP4 needs nvfp4_codes_dev / nvfp4_scales_dev, DQ_FMT_LUT3 and DQ_FMT_NVFP4_FROM_LUT3
 * need lut3_planes_dev / lut3_scales_dev (unused pointers may be NULL); global_scale is the tensor
 * scale s (finite, > 0), shared by both encodings.  packed_dev / packed_bytes / ownership as in
 * dq_pack_weights.  No value check is made on the codes: every bit pattern decodes to something.
 * DQ_FMT_LUT2 is imported on its own with dq_import_canonical_lut2 (passing it here: DQ_ERR_INVALID_ARG).
 */
int dq_import_canonical(int64_t N, int64_t K, unsigned formats, const void *nvfp4_codes_dev,
                        const void *nvfp4_scales_dev, const void *lut3_planes_dev,
                        const void *lut3_scales_dev, float global_scale,
                        const uint16_t *lut3_codebook_f16_host, void *packed_dev, size_t packed_bytes,
                        void *stream, dq_weights **out_host);

/*
 * A DQ_FMT_LUT2 handle from canonical LUT2 encodings (planes uint32[N][2][K/32], scales uint8[N][K/16] signed E4M3,
 * device pointers; App. A.3 "LUT formats", the 4-level grid) and the tensor scale.  The result decodes with
 * dq_decode_linear_lut2.  Other arguments, ownership and status codes as dq_import_canonical.
 */
int dq_import_canonical_lut2(int64_t N, int64_t K, const void *lut2_planes_dev, const void *lut2_scales_dev,
                             float global_scale, void *packed_dev, size_t packed_bytes, void *stream,
                             dq_weights **out_host);

/*
 * The activation quantiser of dq_prefill_linear on its own (App. A.3 "NVFP4",
 * static input scale), writing canonical layout:
 *   codes uint8[M][K/2], scales uint8[M][K/16].
 */
int dq_quantize_activations(const void *A_dev, int64_t M, int64_t K, int64_t lda,
                            float act_global_scale, void *codes_dev, void *scales_dev,
                            void *stream);

/*
 * The fused quantisers of dq_prefill_rmsnorm_quantize / dq_prefill_silu_mul_quantize on their own, writing canonical
 * layout (codes uint8[M][K/2], scales uint8[M][K/16]; K = F for the gated form).  Arguments as there.
 */
int dq_rmsnorm_quantize_activations(const void *X_dev, int64_t M, int64_t K, int64_t ldx,
                                    const void *gamma_dev, float eps, float act_global_scale,
                                    void *codes_dev, void *scales_dev, void *stream);
int dq_silu_mul_quantize_activations(const void *GU_dev, int64_t M, int64_t F, int64_t ldgu,
                                     float act_global_scale, void *codes_dev, void *scales_dev,
                                     void *stream);

/*
 * Measurement hook: how long the last CTA-pair GEMM launch on the current device (dq_prefill_gemm with M > 128,
 * dq_prefill_gemm_silu_mul_quantize, dq_bench_gemm_mma_only) ran on the SM of its first CTA, in SM clock cycles
 * (clock64) and in nanoseconds of the global timer; their ratio is the SM clock under that load, which on a
 * power-capped part is lower than what a management query reports between launches.  Synchronises `stream`.
 * Both values are 0 before the first such launch.
 */
int dq_bench_gemm_clocks(void *stream, unsigned long long *sm_cycles_host, unsigned long long *ns_host);

/*
 * Test hook: out[i] = SiLU(g[i]) in fp32 exactly as the gated quantisers evaluate it (dq_prefill_silu_mul_quantize,
 * dq_prefill_gemm_silu_mul_quantize; App. C.1 fused activation processing), for n bf16 values on the device.  There
 * are only 65536 inputs, so a test can compare the fixed fp32 sequence with a CPU evaluation for every one of them.
 */
int dq_test_silu(const void *g_dev, int64_t n, float *out_dev, void *stream);

/*
 * Reads the library's device status word for the current device (synchronises
 * `stream`).  Kernels never trap or spin without bound: a wait that runs out
 * records DQ_ERR_TIMEOUT and a detail code here and the kernel returns.
 * The word is cleared by the read.
 */
int dq_get_status(void *stream, int *status_host, int *detail_host);

/* Shape queries on a handle. */
int dq_weights_shape(const dq_weights *w, int64_t *N_host, int64_t *K_host, unsigned *formats_host);

/* ---- test hooks (the paper has no counterpart; not for production callers) ---- */

/*
 * A decode call with its launch parameters forced, so that tests reach every work split and the
 * bounded-wait exit of the kernels without touching global state.
 *   format  DQ_FMT_LUT3 / DQ_FMT_LUT2: the LUT decode kernel with `warps_per_group` warps sharing an
 *           8-row tile, `groups_per_cta` such groups per CTA, `ring_stages` bulk-copy stages per
 *           warp (each 0 = the launcher's choice; their product must fit 32 warps, stages 2..8) and
 *           a device-side wait budget of `wait_cycles` SM clocks (0 = the default of about two
 *           seconds).  variant 1 additionally leaves out one bulk copy (the first atom of warp 0 of
 *           CTA 0), so that the wait for it runs out after `wait_cycles`: the kernel returns normally,
 *           writes partial output and records DQ_ERR_TIMEOUT for dq_get_status.  variant 2 is the
 *           same kernel as variant 0.  variant 3 (B = 1 only; DQ_ERR_INVALID_ARG where the row is
 *           too long for its shared-memory layout, about K > 12288) runs the tcgen05 kernel instead:
 *           levels stored to tensor memory, one tcgen05.mma per 16-weight block, the same exact
 *           arithmetic; measured slower than the default kernel, it is kept for comparison and is
 *           not what dq_decode_linear launches.  The three split arguments do not apply to it.
 *           variant 4 runs the kernel that dq_decode_linear takes for batches above 8 on matrices
 *           of 8192 rows and more (up to 32 columns in one pass over the weights, 16-row
 *           tiles, K walked in slices of 1024 with a power-of-two activation scale per slice) on
 *           any shape and batch; groups_per_cta (1..9) then sets its warps per CTA.
 *   format  DQ_FMT_NVFP4 / DQ_FMT_NVFP4_FROM_LUT3: the NVFP4A16 decode; variant 0 = the tensor-core
 *           kernel dq_decode_linear_nvfp4 runs, 1 = the CUDA-core kernel kept for comparison.
 * Other arguments as dq_decode_linear.
 */
int dq_test_decode_linear(const dq_weights *w, unsigned format, int variant, int warps_per_group,
                          int groups_per_cta, int ring_stages, long long wait_cycles, const void *X_dev,
                          int64_t B, int64_t ldx, void *Y_dev, int64_t ldy, void *stream);

/* ---- measurement hooks (the paper has no counterpart; they give bench.py its two measured ceilings) ---- */

/*
 * The prefill GEMM kernel reduced to its tensor-core instruction stream: same launch, roles and barriers as
 * dq_prefill_gemm for M > 128, but no operand or scale loads, no scale copies and no stores (Y_dev is not
 * written; the products are computed on whatever shared memory holds).  2*M*N*K divided by its time is the
 * block-scaled FP4 rate this kernel's MMA sequence reaches on this GPU at the clock it runs at: the measured
 * FP4 tensor peak the roofline fraction is quoted against beside the nominal figure.  M must exceed 128;
 * arguments otherwise as dq_prefill_gemm (the workspace need not have been filled).
 */
int dq_bench_gemm_mma_only(const dq_weights *w, int64_t M, void *Y_dev, int64_t ldy,
                           const void *workspace_dev, size_t workspace_bytes, void *stream);

/*
 * Reads `bytes` bytes at src_dev once with 128-bit loads and nothing else (a grid of 4 CTAs per SM): bytes
 * divided by its time is the practical read-only streaming ceiling for the decode kernels.  out_dev: 8 bytes
 * of device memory (a counter that keeps the loads alive), src_dev 16-byte aligned.
 */
int dq_bench_stream_read(const void *src_dev, size_t bytes, void *out_dev, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* DQ_H_ */
