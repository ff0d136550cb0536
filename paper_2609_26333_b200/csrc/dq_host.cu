// Host-buffer entry points: the prefill and decode linears on activations and outputs that live in
// (pinned) host memory, with the copies in both directions inside the call.  The paper has no
// counterpart; these exist so that the end-to-end cost of the path can be measured and used through
// the C ABI.  The prefill version cuts M into row chunks and runs three streams (copy in, compute, copy
// out) so that the host-to-device copy of chunk c+1 and the device-to-host copy of chunk c-1 overlap the
// quantiser and GEMM of chunk c; PCIe in the output direction is the bound for realistic shapes.
#include <cuda_runtime.h>

#include "dq_common.cuh"

namespace {

constexpr int kMaxChunks = 64;
constexpr int kMaxDevices = 64;

struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t start = nullptr, a_ready[kMaxChunks], y_ready[kMaxChunks], out_done = nullptr;
};
HostPipe g_pipe[kMaxDevices];

int pipe_for_current_device(HostPipe **out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DQ_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return DQ_ERR_INVALID_ARG;
    HostPipe &p = g_pipe[dev];
    if (!p.ready) {
        if (cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking) != cudaSuccess) return DQ_ERR_CUDA;
        if (cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking) != cudaSuccess) return DQ_ERR_CUDA;
        if (cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) != cudaSuccess) return DQ_ERR_CUDA;
        if (cudaEventCreateWithFlags(&p.out_done, cudaEventDisableTiming) != cudaSuccess) return DQ_ERR_CUDA;
        for (int i = 0; i < kMaxChunks; ++i) {
            if (cudaEventCreateWithFlags(&p.a_ready[i], cudaEventDisableTiming) != cudaSuccess) return DQ_ERR_CUDA;
            if (cudaEventCreateWithFlags(&p.y_ready[i], cudaEventDisableTiming) != cudaSuccess) return DQ_ERR_CUDA;
        }
        p.ready = true;
    }
    *out = &p;
    return DQ_OK;
}

inline size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int64_t chunk_rows(int64_t M)
{
    int64_t rows = 1024;                                    // whole GEMM row tiles; at most kMaxChunks chunks
    while ((M + rows - 1) / rows > kMaxChunks) rows *= 2;
    return rows;
}

}  // namespace

extern "C" {

int dq_prefill_host_staging_bytes(const dq_weights *w, int64_t M, size_t *bytes_host)
{
    if (!bytes_host || M < 1) return DQ_ERR_INVALID_ARG;
    int64_t N = 0, K = 0;
    int st = dq_weights_shape(w, &N, &K, nullptr);
    if (st != DQ_OK) return st;
    size_t ws = 0;
    st = dq_prefill_workspace_bytes(w, M < chunk_rows(M) ? M : chunk_rows(M), &ws);
    if (st != DQ_OK) return st;
    *bytes_host = up((size_t)M * K * 2, 1024) + up((size_t)M * N * 2, 1024) + up(ws, 1024);
    return DQ_OK;
}

int dq_prefill_linear_host(const dq_weights *w, const void *A_host, int64_t M, int64_t lda, float act_global_scale,
                           void *Y_host, int64_t ldy, void *staging_dev, size_t staging_bytes, void *stream)
{
    if (!A_host || !Y_host || !staging_dev || M < 1) return DQ_ERR_INVALID_ARG;
    int64_t N = 0, K = 0;
    int st = dq_weights_shape(w, &N, &K, nullptr);
    if (st != DQ_OK) return st;
    if (lda < K || ldy < N) return DQ_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(staging_dev) % 1024 != 0) return DQ_ERR_ALIGN;
    size_t need = 0;
    st = dq_prefill_host_staging_bytes(w, M, &need);
    if (st != DQ_OK) return st;
    if (staging_bytes < need) return DQ_ERR_WORKSPACE;
    HostPipe *p = nullptr;
    st = pipe_for_current_device(&p);
    if (st != DQ_OK) return st;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint8_t *base = reinterpret_cast<uint8_t *>(staging_dev);
    uint8_t *A_dev = base;
    uint8_t *Y_dev = A_dev + up((size_t)M * K * 2, 1024);
    uint8_t *ws = Y_dev + up((size_t)M * N * 2, 1024);
    const size_t ws_bytes = staging_bytes - (size_t)(ws - base);
    const int64_t rows = chunk_rows(M);
    const int chunks = (int)((M + rows - 1) / rows);

    // the side streams start after everything already queued on the caller's stream
    if (cudaEventRecord(p->start, s) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamWaitEvent(p->s_in, p->start, 0) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamWaitEvent(p->s_out, p->start, 0) != cudaSuccess) return DQ_ERR_CUDA;
    for (int c = 0; c < chunks; ++c) {
        const int64_t r0 = c * rows, mc = (M - r0 < rows) ? (M - r0) : rows;
        if (cudaMemcpy2DAsync(A_dev + (size_t)r0 * K * 2, (size_t)K * 2,
                              reinterpret_cast<const uint8_t *>(A_host) + (size_t)r0 * lda * 2, (size_t)lda * 2,
                              (size_t)K * 2, (size_t)mc, cudaMemcpyHostToDevice, p->s_in) != cudaSuccess)
            return DQ_ERR_CUDA;
        if (cudaEventRecord(p->a_ready[c], p->s_in) != cudaSuccess) return DQ_ERR_CUDA;
    }
    for (int c = 0; c < chunks; ++c) {
        const int64_t r0 = c * rows, mc = (M - r0 < rows) ? (M - r0) : rows;
        if (cudaStreamWaitEvent(s, p->a_ready[c], 0) != cudaSuccess) return DQ_ERR_CUDA;
        st = dq_prefill_linear(w, A_dev + (size_t)r0 * K * 2, mc, K, act_global_scale, Y_dev + (size_t)r0 * N * 2, N, ws,
                               ws_bytes, s);
        if (st != DQ_OK) return st;
        if (cudaEventRecord(p->y_ready[c], s) != cudaSuccess) return DQ_ERR_CUDA;
        if (cudaStreamWaitEvent(p->s_out, p->y_ready[c], 0) != cudaSuccess) return DQ_ERR_CUDA;
        if (cudaMemcpy2DAsync(reinterpret_cast<uint8_t *>(Y_host) + (size_t)r0 * ldy * 2, (size_t)ldy * 2,
                              Y_dev + (size_t)r0 * N * 2, (size_t)N * 2, (size_t)N * 2, (size_t)mc,
                              cudaMemcpyDeviceToHost, p->s_out) != cudaSuccess)
            return DQ_ERR_CUDA;
    }
    // the caller's stream is done when the last output chunk has landed
    if (cudaEventRecord(p->out_done, p->s_out) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamWaitEvent(s, p->out_done, 0) != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int dq_decode_linear_host(const dq_weights *w, const void *X_host, int64_t B, int64_t ldx, void *Y_host, int64_t ldy,
                          void *staging_dev, size_t staging_bytes, void *stream)
{
    if (!X_host || !Y_host || !staging_dev || B < 1 || B > 64) return DQ_ERR_INVALID_ARG;
    int64_t N = 0, K = 0;
    int st = dq_weights_shape(w, &N, &K, nullptr);
    if (st != DQ_OK) return st;
    if (ldx < K || ldy < N) return DQ_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(staging_dev) % 1024 != 0) return DQ_ERR_ALIGN;
    const size_t x_bytes = up((size_t)B * K * 2, 1024);
    if (staging_bytes < x_bytes + (size_t)B * N * 2) return DQ_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint8_t *X_dev = reinterpret_cast<uint8_t *>(staging_dev);
    uint8_t *Y_dev = X_dev + x_bytes;
    if (cudaMemcpy2DAsync(X_dev, (size_t)K * 2, X_host, (size_t)ldx * 2, (size_t)K * 2, (size_t)B, cudaMemcpyHostToDevice,
                          s) != cudaSuccess)
        return DQ_ERR_CUDA;
    st = dq_decode_linear(w, X_dev, B, K, Y_dev, N, s);
    if (st != DQ_OK) return st;
    if (cudaMemcpy2DAsync(Y_host, (size_t)ldy * 2, Y_dev, (size_t)N * 2, (size_t)N * 2, (size_t)B, cudaMemcpyDeviceToHost,
                          s) != cudaSuccess)
        return DQ_ERR_CUDA;
    return DQ_OK;
}

}  // extern "C"
