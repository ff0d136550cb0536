// C ABI (include/dq.h): argument checks, handle bookkeeping and kernel launches.
// No device allocation, no synchronisation except in dq_get_status.
#include <cmath>
#include <cstring>
#include <new>

#include "dq_common.cuh"

namespace dq {
__device__ StatusWord g_status_word;
}

struct dq_weights {
    uint32_t magic;
    int device;
    int64_t N, K;
    unsigned formats;
    uint8_t *base;
    dq::PackedLayout layout;
};

namespace {

constexpr uint32_t kMagic = 0x44515731u;   // "DQW1"

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_arch()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DQ_ERR_CUDA;
    int major = 0, minor = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess) return DQ_ERR_CUDA;
    if (major != 10 || minor != 0) return DQ_ERR_ARCH;
    return DQ_OK;
}

int check_shape(int64_t N, int64_t K, unsigned formats)
{
    if (N <= 0 || K <= 0) return DQ_ERR_SHAPE;
    if (K % 128 != 0 || N % 16 != 0) return DQ_ERR_SHAPE;
    if (N > (1ll << 30) || K > (1ll << 30)) return DQ_ERR_SHAPE;
    // the LUT decode kernel keeps a whole activation row in shared memory
    if ((formats & (DQ_FMT_LUT3 | DQ_FMT_LUT2 | DQ_FMT_NVFP4_FROM_LUT3)) && K > dq::kLutMaxK) return DQ_ERR_SHAPE;
    return DQ_OK;
}

int check_formats(unsigned formats)
{
    const unsigned all = DQ_FMT_NVFP4 | DQ_FMT_LUT3 | DQ_FMT_NVFP4_FROM_LUT3 | DQ_FMT_LUT2;
    if (formats == 0 || (formats & ~all)) return DQ_ERR_INVALID_ARG;
    if ((formats & DQ_FMT_NVFP4) && (formats & DQ_FMT_NVFP4_FROM_LUT3)) return DQ_ERR_INVALID_ARG;
    return DQ_OK;
}

bool valid_handle(const dq_weights *w) { return w != nullptr && w->magic == kMagic; }

// the handle's buffers live on the device it was packed on; a call made with another device current
// would hand that device's kernels foreign pointers
bool on_handle_device(const dq_weights *w)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == w->device;
}

// Prefill workspace: NVFP4 activations (codes, MMA-layout scales); for a handle that stores only
// LUT3 the NVFP4 view of the weights (codes, MMA-layout scales) follows, rebuilt on every call.
}  // namespace

namespace dq {
// for the entry points that live in other files: is this a live handle whose buffers are on the current device?
bool handle_on_current_device(const dq_weights *w) { return valid_handle(w) && on_handle_device(w); }
}  // namespace dq

namespace {

struct WsLayout { size_t a_sf = 0, w_codes = 0, w_sf = 0, w_sf_bytes = 0, total = 0; };
bool has_nvfp4_view(const dq_weights *w) { return (w->formats & (DQ_FMT_NVFP4 | DQ_FMT_NVFP4_FROM_LUT3)) != 0; }
WsLayout ws_layout(const dq_weights *w, int64_t M)
{
    WsLayout L;
    L.a_sf = dq::align_up((size_t)M * w->K / 2, 1024);
    const size_t sf = dq::align_up((size_t)M, dq::kSfAtomRows) * (size_t)(w->K / dq::kBlock);
    L.total = L.a_sf + dq::align_up(sf, 1024);
    if (!has_nvfp4_view(w)) {
        L.w_codes = L.total;
        L.w_sf = L.w_codes + dq::align_up((size_t)w->N * w->K / 2, 1024);
        L.w_sf_bytes = dq::align_up((size_t)w->N, dq::kSfRowPad) * (size_t)(w->K / dq::kBlock);
        L.total = L.w_sf + dq::align_up(L.w_sf_bytes, 1024);
    }
    return L;
}

dq::StatusWord *status_word_ptr()
{
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, dq::g_status_word) != cudaSuccess) return nullptr;
    return reinterpret_cast<dq::StatusWord *>(p);
}

// default codebook: the paper's LUT3A16 grid (App. A.3 "LUT formats") rounded to fp16
void default_codebook(uint16_t cb[8])
{
    const float grid[8] = {-4.7038f, -2.8698f, -1.3696f, 0.0f, 1.2204f, 2.5285f, 4.0473f, 6.0f};
    for (int j = 0; j < 8; ++j) cb[j] = __half_as_ushort(__float2half_rn(grid[j]));
}

bool valid_codebook(const uint16_t cb[8])
{
    bool has_zero = false;
    float prev = 0.0f;
    for (int j = 0; j < 8; ++j) {
        const float g = __half2float(__ushort_as_half(cb[j]));
        if (!std::isfinite(g)) return false;
        if (j > 0 && !(g > prev)) return false;
        if (g == 0.0f) { has_zero = true; if (cb[j] != 0) return false; }
        prev = g;
    }
    return has_zero && prev == 6.0f;
}

}  // namespace

extern "C" {

int dq_version(void) { return 100; }

const char *dq_status_string(int status)
{
    switch (status) {
        case DQ_OK: return "ok";
        case DQ_ERR_INVALID_ARG: return "invalid argument";
        case DQ_ERR_SHAPE: return "unsupported shape (need K % 128 == 0, N % 16 == 0; K <= 32768 for LUT formats)";
        case DQ_ERR_ALIGN: return "misaligned pointer or stride";
        case DQ_ERR_WORKSPACE: return "buffer too small";
        case DQ_ERR_ARCH: return "device is not compute capability 10.0";
        case DQ_ERR_CUDA: return "CUDA runtime error";
        case DQ_ERR_TIMEOUT: return "device-side wait ran out";
        case DQ_ERR_INTERNAL: return "internal error";
        default: return "unknown status";
    }
}

int dq_packed_bytes(int64_t N, int64_t K, unsigned formats, size_t *bytes_host)
{
    if (!bytes_host) return DQ_ERR_INVALID_ARG;
    int st = check_formats(formats);
    if (st != DQ_OK) return st;
    st = check_shape(N, K, formats);
    if (st != DQ_OK) return st;
    *bytes_host = dq::packed_layout(N, K, formats).total;
    return DQ_OK;
}

int dq_pack_weights(const void *W_dev, int w_dtype, int64_t N, int64_t K, int64_t ldw, unsigned formats,
                    const uint16_t *lut3_codebook_f16_host, void *packed_dev, size_t packed_bytes, void *stream,
                    dq_weights **out_host)
{
    if (!W_dev || !packed_dev || !out_host) return DQ_ERR_INVALID_ARG;
    if (w_dtype != DQ_DT_BF16 && w_dtype != DQ_DT_FP32) return DQ_ERR_INVALID_ARG;
    int st = check_formats(formats);
    if (st != DQ_OK) return st;
    st = check_shape(N, K, formats);
    if (st != DQ_OK) return st;
    if (ldw < K || ldw % 8 != 0) return DQ_ERR_ALIGN;
    if (!aligned(W_dev, 16) || !aligned(packed_dev, 1024)) return DQ_ERR_ALIGN;
    uint16_t cb[8];
    if (lut3_codebook_f16_host) std::memcpy(cb, lut3_codebook_f16_host, sizeof(cb));
    else default_codebook(cb);
    if (!valid_codebook(cb)) return DQ_ERR_INVALID_ARG;
    st = check_arch();
    if (st != DQ_OK) return st;
    if (formats & DQ_FMT_NVFP4_FROM_LUT3) formats |= DQ_FMT_LUT3;
    const dq::PackedLayout L = dq::packed_layout(N, K, formats);
    if (packed_bytes < L.total) return DQ_ERR_WORKSPACE;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint8_t *base = reinterpret_cast<uint8_t *>(packed_dev);
    dq::PackedHeader *hdr = reinterpret_cast<dq::PackedHeader *>(base);
    if (cudaMemsetAsync(base, 0, dq::kHeaderBytes, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_pack_header(hdr, cb, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_absmax(W_dev, w_dtype, N, K, ldw, hdr, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (L.nv_sf_bytes) {
        if (cudaMemsetAsync(base + L.nv_sf_off, 0, L.nv_sf_bytes, s) != cudaSuccess) return DQ_ERR_CUDA;
    }
    if (formats & DQ_FMT_NVFP4) {
        if (dq::launch_pack_nvfp4(W_dev, w_dtype, N, K, ldw, hdr, base + L.nv_codes_off, base + L.nv_sf_off, s) !=
            cudaSuccess)
            return DQ_ERR_CUDA;
    }
    if (formats & DQ_FMT_LUT3) {
        if (K % dq::kLutSlice != 0) {       // partial last slice: padding must read as zero
            if (cudaMemsetAsync(base + L.lut_off, 0, L.lut_bytes, s) != cudaSuccess) return DQ_ERR_CUDA;
        }
        if (dq::launch_pack_lut(3, W_dev, w_dtype, N, K, ldw, hdr, base + L.lut_off, s) != cudaSuccess)
            return DQ_ERR_CUDA;
    }
    if (formats & DQ_FMT_LUT2) {
        if (K % dq::kLutSlice != 0) {
            if (cudaMemsetAsync(base + L.lut2_off, 0, L.lut2_bytes, s) != cudaSuccess) return DQ_ERR_CUDA;
        }
        if (dq::launch_pack_lut(2, W_dev, w_dtype, N, K, ldw, hdr, base + L.lut2_off, s) != cudaSuccess)
            return DQ_ERR_CUDA;
    }
    if (formats & DQ_FMT_NVFP4_FROM_LUT3) {
        if (dq::launch_autocast(hdr, base + L.lut_off, N, K, base + L.nv_codes_off, base + L.nv_sf_off, s) !=
            cudaSuccess)
            return DQ_ERR_CUDA;
    }
    if ((formats & (DQ_FMT_NVFP4 | DQ_FMT_NVFP4_FROM_LUT3)) && dq::launch_fill_e2m1_table(s) != cudaSuccess)
        return DQ_ERR_CUDA;
    if (dq::launch_pack_done(s) != cudaSuccess) return DQ_ERR_CUDA;
    dq_weights *w = new (std::nothrow) dq_weights;
    if (!w) return DQ_ERR_INTERNAL;
    w->magic = kMagic;
    cudaGetDevice(&w->device);
    w->N = N;
    w->K = K;
    w->formats = formats;
    w->base = base;
    w->layout = L;
    *out_host = w;
    return DQ_OK;
}

int dq_import_canonical(int64_t N, int64_t K, unsigned formats, const void *nvfp4_codes_dev,
                        const void *nvfp4_scales_dev, const void *lut3_planes_dev, const void *lut3_scales_dev,
                        float global_scale, const uint16_t *lut3_codebook_f16_host, void *packed_dev,
                        size_t packed_bytes, void *stream, dq_weights **out_host)
{
    if (!packed_dev || !out_host) return DQ_ERR_INVALID_ARG;
    int st = check_formats(formats);
    if (st != DQ_OK) return st;
    st = check_shape(N, K, formats);
    if (st != DQ_OK) return st;
    if (!(global_scale > 0.0f) || !std::isfinite(global_scale)) return DQ_ERR_INVALID_ARG;
    if (formats & DQ_FMT_LUT2) return DQ_ERR_INVALID_ARG;          // LUT2 is packed from master weights only
    if (formats & DQ_FMT_NVFP4_FROM_LUT3) formats |= DQ_FMT_LUT3;
    if ((formats & DQ_FMT_NVFP4) && (!nvfp4_codes_dev || !nvfp4_scales_dev)) return DQ_ERR_INVALID_ARG;
    if ((formats & DQ_FMT_LUT3) && (!lut3_planes_dev || !lut3_scales_dev)) return DQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 1024)) return DQ_ERR_ALIGN;
    if ((formats & DQ_FMT_NVFP4) && (!aligned(nvfp4_codes_dev, 8))) return DQ_ERR_ALIGN;
    if ((formats & DQ_FMT_LUT3) && (!aligned(lut3_planes_dev, 4))) return DQ_ERR_ALIGN;
    uint16_t cb[8];
    if (lut3_codebook_f16_host) std::memcpy(cb, lut3_codebook_f16_host, sizeof(cb));
    else default_codebook(cb);
    if (!valid_codebook(cb)) return DQ_ERR_INVALID_ARG;
    st = check_arch();
    if (st != DQ_OK) return st;
    const dq::PackedLayout L = dq::packed_layout(N, K, formats);
    if (packed_bytes < L.total) return DQ_ERR_WORKSPACE;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint8_t *base = reinterpret_cast<uint8_t *>(packed_dev);
    dq::PackedHeader *hdr = reinterpret_cast<dq::PackedHeader *>(base);
    if (cudaMemsetAsync(base, 0, dq::kHeaderBytes, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_pack_header(hdr, cb, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_set_scale(hdr, global_scale, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (L.nv_sf_bytes && cudaMemsetAsync(base + L.nv_sf_off, 0, L.nv_sf_bytes, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (formats & DQ_FMT_NVFP4) {
        if (dq::launch_import_nvfp4(reinterpret_cast<const uint8_t *>(nvfp4_codes_dev),
                                    reinterpret_cast<const uint8_t *>(nvfp4_scales_dev), N, K, base + L.nv_codes_off,
                                    base + L.nv_sf_off, s) != cudaSuccess)
            return DQ_ERR_CUDA;
    }
    if (formats & DQ_FMT_LUT3) {
        if (K % dq::kLutSlice != 0 && cudaMemsetAsync(base + L.lut_off, 0, L.lut_bytes, s) != cudaSuccess)
            return DQ_ERR_CUDA;
        if (dq::launch_import_lut(3, reinterpret_cast<const uint32_t *>(lut3_planes_dev),
                                  reinterpret_cast<const uint8_t *>(lut3_scales_dev), N, K, base + L.lut_off, s) !=
            cudaSuccess)
            return DQ_ERR_CUDA;
    }
    if (formats & DQ_FMT_NVFP4_FROM_LUT3) {
        if (dq::launch_autocast(hdr, base + L.lut_off, N, K, base + L.nv_codes_off, base + L.nv_sf_off, s) !=
            cudaSuccess)
            return DQ_ERR_CUDA;
    }
    if ((formats & (DQ_FMT_NVFP4 | DQ_FMT_NVFP4_FROM_LUT3)) && dq::launch_fill_e2m1_table(s) != cudaSuccess)
        return DQ_ERR_CUDA;
    if (dq::launch_pack_done(s) != cudaSuccess) return DQ_ERR_CUDA;
    dq_weights *w = new (std::nothrow) dq_weights;
    if (!w) return DQ_ERR_INTERNAL;
    w->magic = kMagic;
    cudaGetDevice(&w->device);
    w->N = N;
    w->K = K;
    w->formats = formats;
    w->base = base;
    w->layout = L;
    *out_host = w;
    return DQ_OK;
}

int dq_import_canonical_lut2(int64_t N, int64_t K, const void *lut2_planes_dev, const void *lut2_scales_dev,
                             float global_scale, void *packed_dev, size_t packed_bytes, void *stream,
                             dq_weights **out_host)
{
    if (!packed_dev || !out_host || !lut2_planes_dev || !lut2_scales_dev) return DQ_ERR_INVALID_ARG;
    const unsigned formats = DQ_FMT_LUT2;
    int st = check_shape(N, K, formats);
    if (st != DQ_OK) return st;
    if (!(global_scale > 0.0f) || !std::isfinite(global_scale)) return DQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 1024) || !aligned(lut2_planes_dev, 4)) return DQ_ERR_ALIGN;
    uint16_t cb[8];
    default_codebook(cb);                                  // header field of the LUT3 grid; the LUT2 grid is fixed
    st = check_arch();
    if (st != DQ_OK) return st;
    const dq::PackedLayout L = dq::packed_layout(N, K, formats);
    if (packed_bytes < L.total) return DQ_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint8_t *base = reinterpret_cast<uint8_t *>(packed_dev);
    dq::PackedHeader *hdr = reinterpret_cast<dq::PackedHeader *>(base);
    if (cudaMemsetAsync(base, 0, dq::kHeaderBytes, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_pack_header(hdr, cb, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_set_scale(hdr, global_scale, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (K % dq::kLutSlice != 0 && cudaMemsetAsync(base + L.lut2_off, 0, L.lut2_bytes, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_import_lut(2, reinterpret_cast<const uint32_t *>(lut2_planes_dev),
                              reinterpret_cast<const uint8_t *>(lut2_scales_dev), N, K, base + L.lut2_off, s) != cudaSuccess)
        return DQ_ERR_CUDA;
    if (dq::launch_pack_done(s) != cudaSuccess) return DQ_ERR_CUDA;
    dq_weights *w = new (std::nothrow) dq_weights;
    if (!w) return DQ_ERR_INTERNAL;
    w->magic = kMagic;
    cudaGetDevice(&w->device);
    w->N = N;
    w->K = K;
    w->formats = formats;
    w->base = base;
    w->layout = L;
    *out_host = w;
    return DQ_OK;
}

int dq_free_weights(dq_weights *w)
{
    if (!valid_handle(w)) return DQ_ERR_INVALID_ARG;
    w->magic = 0;
    delete w;
    return DQ_OK;
}

int dq_weights_shape(const dq_weights *w, int64_t *N_host, int64_t *K_host, unsigned *formats_host)
{
    if (!valid_handle(w)) return DQ_ERR_INVALID_ARG;
    if (N_host) *N_host = w->N;
    if (K_host) *K_host = w->K;
    if (formats_host) *formats_host = w->formats;
    return DQ_OK;
}

int dq_prefill_workspace_bytes(const dq_weights *w, int64_t M, size_t *bytes_host)
{
    if (!valid_handle(w) || !bytes_host || M < 1) return DQ_ERR_INVALID_ARG;
    *bytes_host = ws_layout(w, M).total;
    return DQ_OK;
}

static int prefill_checks(const dq_weights *w, int64_t M, float act_global_scale, const void *workspace_dev,
                          size_t workspace_bytes)
{
    if (!valid_handle(w) || !workspace_dev) return DQ_ERR_INVALID_ARG;
    if (!on_handle_device(w)) return DQ_ERR_INVALID_ARG;
    if (!has_nvfp4_view(w) && !(w->formats & DQ_FMT_LUT3)) return DQ_ERR_INVALID_ARG;
    if (M < 1 || M > (1ll << 24)) return DQ_ERR_INVALID_ARG;
    if (!(act_global_scale > 0.0f) || !std::isfinite(act_global_scale)) return DQ_ERR_INVALID_ARG;
    if (!aligned(workspace_dev, 1024)) return DQ_ERR_ALIGN;
    size_t need = 0;
    dq_prefill_workspace_bytes(w, M, &need);
    if (workspace_bytes < need) return DQ_ERR_WORKSPACE;
    return DQ_OK;
}

// the part of the activation stage that does not depend on how the activations were produced: for a handle that stores
// only LUT3, cast the weights to NVFP4 for this call (Sec. 2.3, same code map as the pack-time view); rows that pad the
// scale layout to the GEMM tile must read as zero
static int prefill_weight_view(const dq_weights *w, uint8_t *ws, const WsLayout &L, cudaStream_t s)
{
    if (has_nvfp4_view(w)) return DQ_OK;
    if (w->N % dq::kSfRowPad != 0 && cudaMemsetAsync(ws + L.w_sf, 0, L.w_sf_bytes, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (dq::launch_autocast(reinterpret_cast<const dq::PackedHeader *>(w->base), w->base + w->layout.lut_off, w->N, w->K,
                            ws + L.w_codes, ws + L.w_sf, s) != cudaSuccess)
        return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_prefill_quantize(const dq_weights *w, const void *A_dev, int64_t M, int64_t lda, float act_global_scale,
                        void *workspace_dev, size_t workspace_bytes, void *stream)
{
    if (!A_dev) return DQ_ERR_INVALID_ARG;
    int st = prefill_checks(w, M, act_global_scale, workspace_dev, workspace_bytes);
    if (st != DQ_OK) return st;
    if (lda < w->K || lda % 8 != 0 || !aligned(A_dev, 16)) return DQ_ERR_ALIGN;
    st = check_arch();
    if (st != DQ_OK) return st;
    uint8_t *ws = reinterpret_cast<uint8_t *>(workspace_dev);
    const WsLayout L = ws_layout(w, M);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (dq::launch_quant_act(A_dev, M, w->K, lda, act_global_scale, ws, ws + L.a_sf, 1, s) != cudaSuccess)
        return DQ_ERR_CUDA;
    return prefill_weight_view(w, ws, L, s);
}

int dq_prefill_rmsnorm_quantize(const dq_weights *w, const void *X_dev, int64_t M, int64_t ldx, const void *gamma_dev,
                                float eps, float act_global_scale, void *workspace_dev, size_t workspace_bytes,
                                void *stream)
{
    if (!X_dev || !gamma_dev) return DQ_ERR_INVALID_ARG;
    if (!(eps >= 0.0f) || !std::isfinite(eps)) return DQ_ERR_INVALID_ARG;
    int st = prefill_checks(w, M, act_global_scale, workspace_dev, workspace_bytes);
    if (st != DQ_OK) return st;
    if (w->K > 131072) return DQ_ERR_SHAPE;
    if (ldx < w->K || ldx % 8 != 0 || !aligned(X_dev, 16) || !aligned(gamma_dev, 16)) return DQ_ERR_ALIGN;
    st = check_arch();
    if (st != DQ_OK) return st;
    uint8_t *ws = reinterpret_cast<uint8_t *>(workspace_dev);
    const WsLayout L = ws_layout(w, M);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (dq::launch_rmsnorm_quant(X_dev, M, w->K, ldx, gamma_dev, eps, act_global_scale, ws, ws + L.a_sf, 1, s) != cudaSuccess)
        return DQ_ERR_CUDA;
    return prefill_weight_view(w, ws, L, s);
}

int dq_prefill_silu_mul_quantize(const dq_weights *w, const void *GU_dev, int64_t M, int64_t ldgu, float act_global_scale,
                                 void *workspace_dev, size_t workspace_bytes, void *stream)
{
    if (!GU_dev) return DQ_ERR_INVALID_ARG;
    int st = prefill_checks(w, M, act_global_scale, workspace_dev, workspace_bytes);
    if (st != DQ_OK) return st;
    if (ldgu < 2 * w->K || ldgu % 8 != 0 || !aligned(GU_dev, 16)) return DQ_ERR_ALIGN;
    st = check_arch();
    if (st != DQ_OK) return st;
    uint8_t *ws = reinterpret_cast<uint8_t *>(workspace_dev);
    const WsLayout L = ws_layout(w, M);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (dq::launch_silu_mul_quant(GU_dev, M, w->K, ldgu, act_global_scale, ws, ws + L.a_sf, 1, s) != cudaSuccess)
        return DQ_ERR_CUDA;
    return prefill_weight_view(w, ws, L, s);
}

static int prefill_gemm(const dq_weights *w, int64_t M, float act_global_scale, void *Y_dev, int64_t ldy,
                        const void *workspace_dev, size_t workspace_bytes, void *stream, bool mma_only)
{
    if (!Y_dev) return DQ_ERR_INVALID_ARG;
    int st = prefill_checks(w, M, act_global_scale, workspace_dev, workspace_bytes);
    if (st != DQ_OK) return st;
    if (ldy < w->N || ldy % 8 != 0 || !aligned(Y_dev, 16)) return DQ_ERR_ALIGN;
    if (mma_only && M <= 128) return DQ_ERR_INVALID_ARG;          // the measurement mode exists in the pair kernel only
    st = check_arch();
    if (st != DQ_OK) return st;
    dq::StatusWord *sw = status_word_ptr();
    if (!sw) return DQ_ERR_CUDA;
    const uint8_t *ws = reinterpret_cast<const uint8_t *>(workspace_dev);
    dq::GemmArgs g;
    const WsLayout L = ws_layout(w, M);
    g.a_codes = ws;
    g.a_sf = ws + L.a_sf;
    g.w_codes = has_nvfp4_view(w) ? w->base + w->layout.nv_codes_off : ws + L.w_codes;
    g.w_sf = has_nvfp4_view(w) ? w->base + w->layout.nv_sf_off : ws + L.w_sf;
    g.hdr = reinterpret_cast<const dq::PackedHeader *>(w->base);
    g.act_scale = act_global_scale;
    g.Y = Y_dev;
    g.ldy = ldy;
    g.M = M;
    g.N = w->N;
    g.K = w->K;
    g.status = sw;
    g.mma_only = mma_only;
    if (dq::launch_gemm_nvfp4(g, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_prefill_gemm(const dq_weights *w, int64_t M, float act_global_scale, void *Y_dev, int64_t ldy,
                    const void *workspace_dev, size_t workspace_bytes, void *stream)
{
    return prefill_gemm(w, M, act_global_scale, Y_dev, ldy, workspace_dev, workspace_bytes, stream, false);
}

int dq_prefill_gemm_silu_mul_quantize(const dq_weights *w_gate_up, int64_t M, float act_global_scale,
                                      const void *workspace_dev, size_t workspace_bytes, const dq_weights *w_down,
                                      float out_global_scale, void *out_workspace_dev, size_t out_workspace_bytes,
                                      void *stream)
{
    int st = prefill_checks(w_gate_up, M, act_global_scale, workspace_dev, workspace_bytes);
    if (st != DQ_OK) return st;
    st = prefill_checks(w_down, M, out_global_scale, out_workspace_dev, out_workspace_bytes);
    if (st != DQ_OK) return st;
    if (w_gate_up->N != 2 * w_down->K) return DQ_ERR_SHAPE;
    {   // the GEMM reads one workspace while its epilogue writes the other
        const uintptr_t a0 = reinterpret_cast<uintptr_t>(workspace_dev), a1 = a0 + workspace_bytes;
        const uintptr_t b0 = reinterpret_cast<uintptr_t>(out_workspace_dev), b1 = b0 + out_workspace_bytes;
        if (a0 < b1 && b0 < a1) return DQ_ERR_INVALID_ARG;
    }
    st = check_arch();
    if (st != DQ_OK) return st;
    dq::StatusWord *sw = status_word_ptr();
    if (!sw) return DQ_ERR_CUDA;
    const uint8_t *ws = reinterpret_cast<const uint8_t *>(workspace_dev);
    uint8_t *ows = reinterpret_cast<uint8_t *>(out_workspace_dev);
    const WsLayout L = ws_layout(w_gate_up, M), LO = ws_layout(w_down, M);
    dq::GemmArgs g;
    g.a_codes = ws;
    g.a_sf = ws + L.a_sf;
    g.w_codes = has_nvfp4_view(w_gate_up) ? w_gate_up->base + w_gate_up->layout.nv_codes_off : ws + L.w_codes;
    g.w_sf = has_nvfp4_view(w_gate_up) ? w_gate_up->base + w_gate_up->layout.nv_sf_off : ws + L.w_sf;
    g.hdr = reinterpret_cast<const dq::PackedHeader *>(w_gate_up->base);
    g.act_scale = act_global_scale;
    g.Y = nullptr;
    g.ldy = w_gate_up->N;
    g.M = M;
    g.N = w_gate_up->N;
    g.K = w_gate_up->K;
    g.status = sw;
    g.gated_codes = ows;
    g.gated_sf = ows + LO.a_sf;
    g.gated_scale = out_global_scale;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (dq::launch_gemm_nvfp4(g, s) != cudaSuccess) return DQ_ERR_CUDA;
    return prefill_weight_view(w_down, ows, LO, s);
}

int dq_bench_gemm_mma_only(const dq_weights *w, int64_t M, void *Y_dev, int64_t ldy, const void *workspace_dev,
                           size_t workspace_bytes, void *stream)
{
    return prefill_gemm(w, M, 1.0f, Y_dev, ldy, workspace_dev, workspace_bytes, stream, true);
}

int dq_bench_stream_read(const void *src_dev, size_t bytes, void *out_dev, void *stream)
{
    if (!src_dev || !out_dev || bytes < 16) return DQ_ERR_INVALID_ARG;
    if (!aligned(src_dev, 16) || !aligned(out_dev, 8)) return DQ_ERR_ALIGN;
    int st = check_arch();
    if (st != DQ_OK) return st;
    if (dq::launch_stream_read(src_dev, bytes, out_dev, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
        return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_prefill_linear(const dq_weights *w, const void *A_dev, int64_t M, int64_t lda, float act_global_scale,
                      void *Y_dev, int64_t ldy, void *workspace_dev, size_t workspace_bytes, void *stream)
{
    if (!A_dev || !Y_dev) return DQ_ERR_INVALID_ARG;
    int st = prefill_checks(w, M, act_global_scale, workspace_dev, workspace_bytes);
    if (st != DQ_OK) return st;
    if (lda < w->K || ldy < w->N || lda % 8 != 0 || ldy % 8 != 0) return DQ_ERR_ALIGN;
    if (!aligned(A_dev, 16) || !aligned(Y_dev, 16)) return DQ_ERR_ALIGN;
    st = dq_prefill_quantize(w, A_dev, M, lda, act_global_scale, workspace_dev, workspace_bytes, stream);
    if (st != DQ_OK) return st;
    return dq_prefill_gemm(w, M, act_global_scale, Y_dev, ldy, workspace_dev, workspace_bytes, stream);
}

static int decode_nvfp4(const dq_weights *w, const void *X_dev, int64_t B, int64_t ldx, void *Y_dev, int64_t ldy,
                        void *stream, bool tensor_cores)
{
    if (!valid_handle(w) || !X_dev || !Y_dev) return DQ_ERR_INVALID_ARG;
    if (!has_nvfp4_view(w) || !on_handle_device(w)) return DQ_ERR_INVALID_ARG;
    if (B < 1 || B > 64) return DQ_ERR_INVALID_ARG;
    if (ldx < w->K || ldy < w->N || ldx % 8 != 0 || ldy % 8 != 0) return DQ_ERR_ALIGN;
    if (!aligned(X_dev, 16) || !aligned(Y_dev, 16)) return DQ_ERR_ALIGN;
    int st = check_arch();
    if (st != DQ_OK) return st;
    dq::GemvNvArgs g;
    g.codes = w->base + w->layout.nv_codes_off;
    g.sf = w->base + w->layout.nv_sf_off;
    g.hdr = reinterpret_cast<const dq::PackedHeader *>(w->base);
    g.status = status_word_ptr();
    if (!g.status) return DQ_ERR_CUDA;
    g.X = X_dev;
    g.ldx = ldx;
    g.B = B;
    g.Y = Y_dev;
    g.ldy = ldy;
    g.N = w->N;
    g.K = w->K;
    const cudaError_t ce = tensor_cores ? dq::launch_gemv_nvfp4_mma(g, reinterpret_cast<cudaStream_t>(stream))
                                        : dq::launch_gemv_nvfp4(g, reinterpret_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_decode_linear_nvfp4(const dq_weights *w, const void *X_dev, int64_t B, int64_t ldx, void *Y_dev, int64_t ldy,
                           void *stream)
{
    return decode_nvfp4(w, X_dev, B, ldx, Y_dev, ldy, stream, true);
}

static int decode_lut(const dq_weights *w, unsigned format, const void *X_dev, int64_t B, int64_t ldx, void *Y_dev,
                      int64_t ldy, void *stream, int P, int G, int S, long long wait_cycles, int drop_first_copy = 0,
                      int kernel = 0)
{
    if (!valid_handle(w) || !X_dev || !Y_dev) return DQ_ERR_INVALID_ARG;
    if (format != DQ_FMT_LUT3 && format != DQ_FMT_LUT2) return DQ_ERR_INVALID_ARG;
    if (!(w->formats & format) || !on_handle_device(w)) return DQ_ERR_INVALID_ARG;
    if (B < 1 || B > 64) return DQ_ERR_INVALID_ARG;
    if (ldx < w->K || ldy < w->N || ldx % 8 != 0 || ldy % 8 != 0) return DQ_ERR_ALIGN;
    if (!aligned(X_dev, 16) || !aligned(Y_dev, 16)) return DQ_ERR_ALIGN;
    int st = check_arch();
    if (st != DQ_OK) return st;
    dq::GemvArgs g;
    g.bits = (format == DQ_FMT_LUT3) ? 3 : 2;
    g.lut = w->base + (format == DQ_FMT_LUT3 ? w->layout.lut_off : w->layout.lut2_off);
    g.status = status_word_ptr();
    if (!g.status) return DQ_ERR_CUDA;
    g.hdr = reinterpret_cast<const dq::PackedHeader *>(w->base);
    g.X = X_dev;
    g.ldx = ldx;
    g.B = B;
    g.Y = Y_dev;
    g.ldy = ldy;
    g.N = w->N;
    g.K = w->K;
    g.force_P = P;
    g.force_G = G;
    g.force_S = S;
    g.wait_cycles = wait_cycles;
    g.drop_first_copy = drop_first_copy;
    g.kernel = kernel;
    const cudaError_t ce = dq::launch_gemv_lut(g, reinterpret_cast<cudaStream_t>(stream));
    if (ce == cudaErrorInvalidValue) return DQ_ERR_INVALID_ARG;
    if (ce != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_decode_linear(const dq_weights *w, const void *X_dev, int64_t B, int64_t ldx, void *Y_dev, int64_t ldy,
                     void *stream)
{
    return decode_lut(w, DQ_FMT_LUT3, X_dev, B, ldx, Y_dev, ldy, stream, 0, 0, 0, 0);
}

int dq_decode_linear_lut2(const dq_weights *w, const void *X_dev, int64_t B, int64_t ldx, void *Y_dev, int64_t ldy,
                          void *stream)
{
    return decode_lut(w, DQ_FMT_LUT2, X_dev, B, ldx, Y_dev, ldy, stream, 0, 0, 0, 0);
}

int dq_test_decode_linear(const dq_weights *w, unsigned format, int variant, int warps_per_group, int groups_per_cta,
                          int ring_stages, long long wait_cycles, const void *X_dev, int64_t B, int64_t ldx, void *Y_dev,
                          int64_t ldy, void *stream)
{
    if (format == DQ_FMT_NVFP4 || format == DQ_FMT_NVFP4_FROM_LUT3)
        return decode_nvfp4(w, X_dev, B, ldx, Y_dev, ldy, stream, variant == 0);
    if (warps_per_group < 0 || groups_per_cta < 0 || ring_stages < 0 || ring_stages > 8 || wait_cycles < 0)
        return DQ_ERR_INVALID_ARG;
    if (variant < 0 || variant > 4) return DQ_ERR_INVALID_ARG;
    return decode_lut(w, format, X_dev, B, ldx, Y_dev, ldy, stream, warps_per_group, groups_per_cta, ring_stages,
                      wait_cycles, variant == 1 ? 1 : 0, variant == 2 ? 1 : variant == 3 ? 2 : variant == 4 ? 3 : 0);
}

int dq_export_canonical(const dq_weights *w, unsigned format, void *codes_dev, void *scales_dev,
                        float *global_scale_dev, void *stream)
{
    if (!valid_handle(w) || !codes_dev || !scales_dev) return DQ_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const dq::PackedHeader *hdr = reinterpret_cast<const dq::PackedHeader *>(w->base);
    if (format == DQ_FMT_NVFP4 || format == DQ_FMT_NVFP4_FROM_LUT3) {
        if (!(w->formats & format)) return DQ_ERR_INVALID_ARG;
        if (dq::launch_export_nvfp4(hdr, w->base + w->layout.nv_codes_off, w->base + w->layout.nv_sf_off, w->N, w->K,
                                    reinterpret_cast<uint8_t *>(codes_dev), reinterpret_cast<uint8_t *>(scales_dev),
                                    global_scale_dev, s) != cudaSuccess)
            return DQ_ERR_CUDA;
        return DQ_OK;
    }
    if (format == DQ_FMT_LUT3 || format == DQ_FMT_LUT2) {
        if (!(w->formats & format)) return DQ_ERR_INVALID_ARG;
        const bool l3 = (format == DQ_FMT_LUT3);
        if (dq::launch_export_lut(l3 ? 3 : 2, hdr, w->base + (l3 ? w->layout.lut_off : w->layout.lut2_off), w->N, w->K,
                                  reinterpret_cast<uint32_t *>(codes_dev), reinterpret_cast<uint8_t *>(scales_dev),
                                  global_scale_dev, s) != cudaSuccess)
            return DQ_ERR_CUDA;
        return DQ_OK;
    }
    return DQ_ERR_INVALID_ARG;
}

int dq_quantize_activations(const void *A_dev, int64_t M, int64_t K, int64_t lda, float act_global_scale,
                            void *codes_dev, void *scales_dev, void *stream)
{
    if (!A_dev || !codes_dev || !scales_dev) return DQ_ERR_INVALID_ARG;
    if (M < 1 || K < 1 || K % 128 != 0) return DQ_ERR_SHAPE;
    if (!(act_global_scale > 0.0f) || !std::isfinite(act_global_scale)) return DQ_ERR_INVALID_ARG;
    if (lda < K || lda % 8 != 0 || !aligned(A_dev, 16) || !aligned(codes_dev, 16) || !aligned(scales_dev, 4))
        return DQ_ERR_ALIGN;
    int st = check_arch();
    if (st != DQ_OK) return st;
    if (dq::launch_quant_act(A_dev, M, K, lda, act_global_scale, reinterpret_cast<uint8_t *>(codes_dev),
                             reinterpret_cast<uint8_t *>(scales_dev), 0,
                             reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
        return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_rmsnorm_quantize_activations(const void *X_dev, int64_t M, int64_t K, int64_t ldx, const void *gamma_dev, float eps,
                                    float act_global_scale, void *codes_dev, void *scales_dev, void *stream)
{
    if (!X_dev || !gamma_dev || !codes_dev || !scales_dev) return DQ_ERR_INVALID_ARG;
    if (M < 1 || K < 1 || K % 128 != 0 || K > 131072) return DQ_ERR_SHAPE;
    if (!(act_global_scale > 0.0f) || !std::isfinite(act_global_scale)) return DQ_ERR_INVALID_ARG;
    if (!(eps >= 0.0f) || !std::isfinite(eps)) return DQ_ERR_INVALID_ARG;
    if (ldx < K || ldx % 8 != 0 || !aligned(X_dev, 16) || !aligned(gamma_dev, 16) || !aligned(codes_dev, 16) ||
        !aligned(scales_dev, 4))
        return DQ_ERR_ALIGN;
    int st = check_arch();
    if (st != DQ_OK) return st;
    if (dq::launch_rmsnorm_quant(X_dev, M, K, ldx, gamma_dev, eps, act_global_scale, reinterpret_cast<uint8_t *>(codes_dev),
                                 reinterpret_cast<uint8_t *>(scales_dev), 0, reinterpret_cast<cudaStream_t>(stream)) !=
        cudaSuccess)
        return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_silu_mul_quantize_activations(const void *GU_dev, int64_t M, int64_t F, int64_t ldgu, float act_global_scale,
                                     void *codes_dev, void *scales_dev, void *stream)
{
    if (!GU_dev || !codes_dev || !scales_dev) return DQ_ERR_INVALID_ARG;
    if (M < 1 || F < 1 || F % 128 != 0) return DQ_ERR_SHAPE;
    if (!(act_global_scale > 0.0f) || !std::isfinite(act_global_scale)) return DQ_ERR_INVALID_ARG;
    if (ldgu < 2 * F || ldgu % 8 != 0 || !aligned(GU_dev, 16) || !aligned(codes_dev, 16) || !aligned(scales_dev, 4))
        return DQ_ERR_ALIGN;
    int st = check_arch();
    if (st != DQ_OK) return st;
    if (dq::launch_silu_mul_quant(GU_dev, M, F, ldgu, act_global_scale, reinterpret_cast<uint8_t *>(codes_dev),
                                  reinterpret_cast<uint8_t *>(scales_dev), 0, reinterpret_cast<cudaStream_t>(stream)) !=
        cudaSuccess)
        return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_test_silu(const void *g_dev, int64_t n, float *out_dev, void *stream)
{
    if (!g_dev || !out_dev || n < 1) return DQ_ERR_INVALID_ARG;
    int st = check_arch();
    if (st != DQ_OK) return st;
    if (dq::launch_silu_probe(g_dev, n, out_dev, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_get_status(void *stream, int *status_host, int *detail_host)
{
    if (!status_host) return DQ_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    dq::StatusWord *sw = status_word_ptr();
    if (!sw) return DQ_ERR_CUDA;
    int h[2] = {0, 0};                                     // status and detail: the first two words
    if (cudaMemcpyAsync(h, sw, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaMemsetAsync(sw, 0, sizeof(h), s) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return DQ_ERR_CUDA;
    *status_host = h[0];
    if (detail_host) *detail_host = h[1];
    return DQ_OK;
}

int dq_bench_gemm_clocks(void *stream, unsigned long long *sm_cycles_host, unsigned long long *ns_host)
{
    if (!sm_cycles_host || !ns_host) return DQ_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    dq::StatusWord *sw = status_word_ptr();
    if (!sw) return DQ_ERR_CUDA;
    dq::StatusWord h;
    if (cudaMemcpyAsync(&h, sw, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return DQ_ERR_CUDA;
    *sm_cycles_host = h.gemm_cycles;
    *ns_host = h.gemm_ns;
    return DQ_OK;
}

}  // extern "C"
