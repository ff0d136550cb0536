// dq_prefill_linear_static: the prefill linear for callers that cannot hand the library
// scratch memory.
//
// Who needs this.  dq_prefill_linear wants a workspace for the quantised activations, and
// normally the caller carves it out of memory it allocated.  Some callers have no way to do
// that at the point of the call: a serving engine that has already given every free byte of
// HBM to its KV-cache pool (a cudaMalloc there fails, or succeeds only by fragmenting what
// the pool counted on), a plug-in that runs inside someone else's process and may not touch
// its allocator, or a latency-critical thread for which the device-wide synchronisation
// hidden inside cudaMalloc / cudaFree is unacceptable.  For them the scratch below is part of
// the library image itself: it is reserved when the library is loaded onto a GPU and is
// never allocated or freed at run time.
#include "dq_common.cuh"

namespace {

// Usable scratch: 8 MiB (enough for e.g. 2048 tokens x 4096 features or 1024 x 12288).
// 1 KiB more is reserved so the start can be rounded up to the 1024-byte alignment the
// prefill path asks of its workspace.  Every GPU that loads the library holds this until the
// process exits.
constexpr size_t kStaticScratchUsable = 8u << 20;
static __device__ __align__(256) unsigned char g_prefill_scratch[kStaticScratchUsable + 1024];

constexpr int kMaxDevices = 64;
unsigned char *g_scratch_ptr[kMaxDevices] = {};     // device address of the array, per device

// In host code `g_prefill_scratch` is only a handle for the symbol, not an address a kernel
// can use; the device address has to be asked for, once per device, with that device current.
int scratch_for_current_device(unsigned char **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DQ_ERR_CUDA;
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_prefill_scratch) != cudaSuccess || p == nullptr) return DQ_ERR_CUDA;
        g_scratch_ptr[dev] = reinterpret_cast<unsigned char *>(p);
    }
    uintptr_t a = reinterpret_cast<uintptr_t>(g_scratch_ptr[dev]);
    a = (a + 1023) & ~static_cast<uintptr_t>(1023);
    *out = reinterpret_cast<unsigned char *>(a);
    return DQ_OK;
}

}  // namespace

extern "C" int dq_prefill_linear_static(const dq_weights *w, const void *A_dev, int64_t M, int64_t lda,
                                        float act_global_scale, void *Y_dev, int64_t ldy, void *stream)
{
    size_t need = 0;
    int st = dq_prefill_workspace_bytes(w, M, &need);
    if (st != DQ_OK) return st;
    if (need > kStaticScratchUsable) return DQ_ERR_WORKSPACE;      // M * K too large for the built-in scratch
    int64_t N = 0, K = 0;
    st = dq_weights_shape(w, &N, &K, nullptr);
    if (st != DQ_OK) return st;
    // Everything dq_prefill_linear would reject is rejected here, before any work is put on the stream.
    if (!dq::handle_on_current_device(w)) return DQ_ERR_INVALID_ARG;
    if (!A_dev || !Y_dev || !(act_global_scale > 0.0f) || !(act_global_scale <= 3.0e38f)) return DQ_ERR_INVALID_ARG;
    if (lda < K || ldy < N || lda % 8 != 0 || ldy % 8 != 0 || reinterpret_cast<uintptr_t>(A_dev) % 16 != 0 ||
        reinterpret_cast<uintptr_t>(Y_dev) % 16 != 0)
        return DQ_ERR_ALIGN;
    unsigned char *scratch = nullptr;
    st = scratch_for_current_device(&scratch);
    if (st != DQ_OK) return st;
    // The array keeps whatever the previous call left.  Codes and scales of the M live rows are
    // rewritten by this call; the only bytes read without being rewritten are the scale rows that
    // pad M up to a multiple of 128.  They can only influence output rows >= M, which are never
    // stored, but they are cleared anyway so that no stale NaN pattern enters the tensor cores.
    if (M % 128 != 0) {
        const size_t sf_off = dq::align_up((size_t)M * K / 2, 1024);
        const size_t group_bytes = (size_t)(K / 64) * 512;
        const size_t last_group = (size_t)(M / 128) * group_bytes;
        if (cudaMemsetAsync(scratch + sf_off + last_group, 0, group_bytes, reinterpret_cast<cudaStream_t>(stream)) !=
            cudaSuccess)
            return DQ_ERR_CUDA;
    }
    return dq_prefill_linear(w, A_dev, M, lda, act_global_scale, Y_dev, ldy, scratch, kStaticScratchUsable, stream);
}
