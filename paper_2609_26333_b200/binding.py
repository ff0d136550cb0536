"""ctypes binding of include/dq.h.  Argument marshalling only: torch supplies
device memory and streams, every computation happens inside libdq.so."""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libdq.so"

FMT_NVFP4 = 1
FMT_LUT3 = 2
FMT_NVFP4_FROM_LUT3 = 4
FMT_LUT2 = 8
DT_BF16 = 0
DT_FP32 = 1

# every symbol include/dq.h declares
SYMBOLS = ("dq_version", "dq_status_string", "dq_packed_bytes", "dq_pack_weights", "dq_free_weights",
           "dq_prefill_workspace_bytes", "dq_prefill_linear", "dq_prefill_quantize", "dq_prefill_gemm",
           "dq_prefill_linear_static",
           "dq_decode_linear", "dq_decode_linear_nvfp4", "dq_decode_linear_lut2", "dq_test_decode_linear",
           "dq_bench_gemm_mma_only", "dq_bench_stream_read", "dq_bench_gemm_clocks",
           "dq_prefill_rmsnorm_quantize", "dq_prefill_silu_mul_quantize", "dq_prefill_gemm_silu_mul_quantize",
           "dq_rmsnorm_quantize_activations",
           "dq_silu_mul_quantize_activations", "dq_test_silu", "dq_export_canonical", "dq_import_canonical",
           "dq_import_canonical_lut2",
           "dq_quantize_activations", "dq_get_status", "dq_weights_shape",
           "dq_prefill_host_staging_bytes", "dq_prefill_linear_host", "dq_decode_linear_host")


class DQError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib = None


def lib() -> C.CDLL:
    """Loads libdq.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                              "(nvcc, sm_100a) first; there is no CPU fallback")
        L = C.CDLL(str(_LIB_PATH))
        i64, vp, sz = C.c_int64, C.c_void_p, C.c_size_t
        L.dq_version.restype = C.c_int
        L.dq_version.argtypes = []
        L.dq_status_string.restype = C.c_char_p
        L.dq_status_string.argtypes = [C.c_int]
        L.dq_packed_bytes.restype = C.c_int
        L.dq_packed_bytes.argtypes = [i64, i64, C.c_uint, C.POINTER(sz)]
        L.dq_pack_weights.restype = C.c_int
        L.dq_pack_weights.argtypes = [vp, C.c_int, i64, i64, i64, C.c_uint, C.POINTER(C.c_uint16), vp, sz, vp,
                                      C.POINTER(vp)]
        L.dq_free_weights.restype = C.c_int
        L.dq_free_weights.argtypes = [vp]
        L.dq_prefill_workspace_bytes.restype = C.c_int
        L.dq_prefill_workspace_bytes.argtypes = [vp, i64, C.POINTER(sz)]
        L.dq_prefill_linear.restype = C.c_int
        L.dq_prefill_linear.argtypes = [vp, vp, i64, i64, C.c_float, vp, i64, vp, sz, vp]
        L.dq_prefill_quantize.restype = C.c_int
        L.dq_prefill_quantize.argtypes = [vp, vp, i64, i64, C.c_float, vp, sz, vp]
        L.dq_prefill_gemm.restype = C.c_int
        L.dq_prefill_gemm.argtypes = [vp, i64, C.c_float, vp, i64, vp, sz, vp]
        L.dq_prefill_linear_static.restype = C.c_int
        L.dq_prefill_linear_static.argtypes = [vp, vp, i64, i64, C.c_float, vp, i64, vp]
        L.dq_decode_linear.restype = C.c_int
        L.dq_decode_linear.argtypes = [vp, vp, i64, i64, vp, i64, vp]
        L.dq_prefill_host_staging_bytes.restype = C.c_int
        L.dq_prefill_host_staging_bytes.argtypes = [vp, i64, C.POINTER(C.c_size_t)]
        L.dq_prefill_linear_host.restype = C.c_int
        L.dq_prefill_linear_host.argtypes = [vp, vp, i64, i64, C.c_float, vp, i64, vp, C.c_size_t, vp]
        L.dq_decode_linear_host.restype = C.c_int
        L.dq_decode_linear_host.argtypes = [vp, vp, i64, i64, vp, i64, vp, C.c_size_t, vp]
        L.dq_decode_linear_nvfp4.restype = C.c_int
        L.dq_decode_linear_nvfp4.argtypes = [vp, vp, i64, i64, vp, i64, vp]
        L.dq_decode_linear_lut2.restype = C.c_int
        L.dq_decode_linear_lut2.argtypes = [vp, vp, i64, i64, vp, i64, vp]
        L.dq_test_decode_linear.restype = C.c_int
        L.dq_test_decode_linear.argtypes = [vp, C.c_uint, C.c_int, C.c_int, C.c_int, C.c_int, C.c_longlong, vp, i64, i64,
                                            vp, i64, vp]
        L.dq_prefill_rmsnorm_quantize.restype = C.c_int
        L.dq_prefill_rmsnorm_quantize.argtypes = [vp, vp, i64, i64, vp, C.c_float, C.c_float, vp, sz, vp]
        L.dq_prefill_silu_mul_quantize.restype = C.c_int
        L.dq_prefill_silu_mul_quantize.argtypes = [vp, vp, i64, i64, C.c_float, vp, sz, vp]
        L.dq_bench_gemm_clocks.restype = C.c_int
        L.dq_bench_gemm_clocks.argtypes = [vp, C.POINTER(C.c_ulonglong), C.POINTER(C.c_ulonglong)]
        L.dq_test_silu.restype = C.c_int
        L.dq_test_silu.argtypes = [vp, i64, vp, vp]
        L.dq_prefill_gemm_silu_mul_quantize.restype = C.c_int
        L.dq_prefill_gemm_silu_mul_quantize.argtypes = [vp, i64, C.c_float, vp, sz, vp, C.c_float, vp, sz, vp]
        L.dq_rmsnorm_quantize_activations.restype = C.c_int
        L.dq_rmsnorm_quantize_activations.argtypes = [vp, i64, i64, i64, vp, C.c_float, C.c_float, vp, vp, vp]
        L.dq_silu_mul_quantize_activations.restype = C.c_int
        L.dq_silu_mul_quantize_activations.argtypes = [vp, i64, i64, i64, C.c_float, vp, vp, vp]
        L.dq_bench_gemm_mma_only.restype = C.c_int
        L.dq_bench_gemm_mma_only.argtypes = [vp, i64, vp, i64, vp, sz, vp]
        L.dq_bench_stream_read.restype = C.c_int
        L.dq_bench_stream_read.argtypes = [vp, sz, vp, vp]
        L.dq_import_canonical.restype = C.c_int
        L.dq_import_canonical.argtypes = [C.c_int64, C.c_int64, C.c_uint, vp, vp, vp, vp, C.c_float,
                                          C.POINTER(C.c_uint16), vp, C.c_size_t, vp, C.POINTER(vp)]
        L.dq_import_canonical_lut2.restype = C.c_int
        L.dq_import_canonical_lut2.argtypes = [C.c_int64, C.c_int64, vp, vp, C.c_float, vp, C.c_size_t, vp, C.POINTER(vp)]
        L.dq_export_canonical.restype = C.c_int
        L.dq_export_canonical.argtypes = [vp, C.c_uint, vp, vp, vp, vp]
        L.dq_quantize_activations.restype = C.c_int
        L.dq_quantize_activations.argtypes = [vp, i64, i64, i64, C.c_float, vp, vp, vp]
        L.dq_get_status.restype = C.c_int
        L.dq_get_status.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.dq_weights_shape.restype = C.c_int
        L.dq_weights_shape.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(C.c_uint)]
        _lib = L
    return _lib


def version() -> int:
    return int(lib().dq_version())


def status_string(code: int) -> str:
    return lib().dq_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise DQError(code, where)


def _stream_ptr(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def packed_bytes(N: int, K: int, formats: int) -> int:
    out = C.c_size_t(0)
    _check(lib().dq_packed_bytes(N, K, formats, C.byref(out)), "dq_packed_bytes")
    return int(out.value)


class DQWeights:
    """Handle returned by :func:`pack_weights`; keeps the packed device buffer alive."""

    def __init__(self, handle: int, packed: torch.Tensor, N: int, K: int, formats: int):
        self.handle = handle
        self.packed = packed
        self.N, self.K, self.formats = N, K, formats

    def free(self):
        if self.handle:
            lib().dq_free_weights(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def pack_weights(W: torch.Tensor, formats: int = FMT_NVFP4 | FMT_LUT3, codebook_f16=None, stream=None) -> DQWeights:
    """dq_pack_weights on a CUDA tensor W (N x K, bf16 or fp32, rows contiguous)."""
    assert W.is_cuda and W.dim() == 2 and W.stride(1) == 1
    if W.dtype == torch.bfloat16:
        dt = DT_BF16
    elif W.dtype == torch.float32:
        dt = DT_FP32
    else:
        raise TypeError("W must be bf16 or fp32")
    N, K = W.shape
    nbytes = packed_bytes(N, K, formats)
    packed = torch.empty(nbytes + 1024, dtype=torch.uint8, device=W.device)
    off = (-packed.data_ptr()) % 1024
    view = packed[off:off + nbytes]
    cb = None
    if codebook_f16 is not None:
        cb = (C.c_uint16 * 8)(*[int(v) for v in codebook_f16])
    out = C.c_void_p(0)
    _check(lib().dq_pack_weights(W.data_ptr(), dt, N, K, W.stride(0), formats, cb, view.data_ptr(), nbytes,
                                 _stream_ptr(stream), C.byref(out)), "dq_pack_weights")
    if formats & FMT_NVFP4_FROM_LUT3:
        formats |= FMT_LUT3
    return DQWeights(out.value, packed, N, K, formats)


def import_canonical(N: int, K: int, formats: int, global_scale: float, nvfp4=None, lut3=None, codebook_f16=None,
                     stream=None) -> DQWeights:
    """dq_import_canonical: handle from canonical (codes, scales) pairs of CUDA tensors."""
    dev = (nvfp4 or lut3)[0].device
    nbytes = packed_bytes(N, K, formats)
    packed = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
    off = (-packed.data_ptr()) % 1024
    view = packed[off:off + nbytes]
    cb = None
    if codebook_f16 is not None:
        cb = (C.c_uint16 * 8)(*[int(v) for v in codebook_f16])
    ptr = lambda pair, i: pair[i].data_ptr() if pair is not None else None
    if nvfp4 is not None:
        assert nvfp4[0].is_contiguous() and nvfp4[1].is_contiguous() and nvfp4[0].shape == (N, K // 2)
    if lut3 is not None:
        assert lut3[0].is_contiguous() and lut3[1].is_contiguous() and lut3[0].shape == (N, 3, K // 32)
    out = C.c_void_p(0)
    _check(lib().dq_import_canonical(N, K, formats, ptr(nvfp4, 0), ptr(nvfp4, 1), ptr(lut3, 0), ptr(lut3, 1),
                                     float(global_scale), cb, view.data_ptr(), nbytes, _stream_ptr(stream),
                                     C.byref(out)), "dq_import_canonical")
    if formats & FMT_NVFP4_FROM_LUT3:
        formats |= FMT_LUT3
    return DQWeights(out.value, packed, N, K, formats)


def import_canonical_lut2(N: int, K: int, global_scale: float, planes: torch.Tensor, scales: torch.Tensor,
                          stream=None) -> DQWeights:
    """dq_import_canonical_lut2: a LUT2 handle from canonical bit-planes (N, 2, K/32) and scales (N, K/16)."""
    assert planes.is_cuda and planes.is_contiguous() and tuple(planes.shape) == (N, 2, K // 32)
    assert scales.is_cuda and scales.is_contiguous() and tuple(scales.shape) == (N, K // 16)
    nbytes = packed_bytes(N, K, FMT_LUT2)
    packed = torch.empty(nbytes + 1024, dtype=torch.uint8, device=planes.device)
    off = (-packed.data_ptr()) % 1024
    view = packed[off:off + nbytes]
    out = C.c_void_p(0)
    _check(lib().dq_import_canonical_lut2(N, K, planes.data_ptr(), scales.data_ptr(), float(global_scale),
                                          view.data_ptr(), nbytes, _stream_ptr(stream), C.byref(out)),
           "dq_import_canonical_lut2")
    return DQWeights(out.value, packed, N, K, FMT_LUT2)


def prefill_workspace_bytes(w: DQWeights, M: int) -> int:
    out = C.c_size_t(0)
    _check(lib().dq_prefill_workspace_bytes(w.handle, M, C.byref(out)), "dq_prefill_workspace_bytes")
    return int(out.value)


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    buf = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + nbytes]


def prefill_linear(w: DQWeights, A: torch.Tensor, act_global_scale: float, out: torch.Tensor = None,
                   workspace: torch.Tensor = None, stream=None) -> torch.Tensor:
    """dq_prefill_linear: Y = NVFP4(A) @ NVFP4(W)^T, bf16 out."""
    assert A.is_cuda and A.dtype == torch.bfloat16 and A.dim() == 2 and A.stride(1) == 1 and A.shape[1] == w.K
    M = A.shape[0]
    if out is None:
        out = torch.empty(M, w.N, dtype=torch.bfloat16, device=A.device)
    if workspace is None:
        workspace = alloc_workspace(prefill_workspace_bytes(w, M), A.device)
    _check(lib().dq_prefill_linear(w.handle, A.data_ptr(), M, A.stride(0), float(act_global_scale), out.data_ptr(),
                                   out.stride(0), workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)),
           "dq_prefill_linear")
    return out


def prefill_linear_static(w: DQWeights, A: torch.Tensor, act_global_scale: float, out: torch.Tensor = None,
                          stream=None) -> torch.Tensor:
    """dq_prefill_linear_static: the prefill linear on the library's built-in 8 MiB scratch.

    For callers that cannot allocate device memory at the call site (all HBM owned by a pool,
    foreign allocator, no tolerance for cudaMalloc's synchronisation).  Calls that overlap on
    the GPU race on the shared scratch."""
    assert A.is_cuda and A.dtype == torch.bfloat16 and A.dim() == 2 and A.stride(1) == 1 and A.shape[1] == w.K
    M = A.shape[0]
    if out is None:
        out = torch.empty(M, w.N, dtype=torch.bfloat16, device=A.device)
    _check(lib().dq_prefill_linear_static(w.handle, A.data_ptr(), M, A.stride(0), float(act_global_scale),
                                          out.data_ptr(), out.stride(0), _stream_ptr(stream)),
           "dq_prefill_linear_static")
    return out


def prefill_quantize(w: DQWeights, A: torch.Tensor, act_global_scale: float, workspace: torch.Tensor, stream=None):
    """dq_prefill_quantize: stage 1 of the prefill linear (activations -> NVFP4 in the workspace)."""
    _check(lib().dq_prefill_quantize(w.handle, A.data_ptr(), A.shape[0], A.stride(0), float(act_global_scale),
                                     workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)),
           "dq_prefill_quantize")


def prefill_rmsnorm_quantize(w: DQWeights, X: torch.Tensor, gamma: torch.Tensor, eps: float, act_global_scale: float,
                             workspace: torch.Tensor, stream=None):
    """dq_prefill_rmsnorm_quantize: RMSNorm fused with stage 1 of the prefill linear."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.stride(1) == 1 and X.shape[1] == w.K
    assert gamma.is_cuda and gamma.dtype == torch.bfloat16 and gamma.is_contiguous() and gamma.numel() == w.K
    _check(lib().dq_prefill_rmsnorm_quantize(w.handle, X.data_ptr(), X.shape[0], X.stride(0), gamma.data_ptr(), float(eps),
                                             float(act_global_scale), workspace.data_ptr(), workspace.numel(),
                                             _stream_ptr(stream)), "dq_prefill_rmsnorm_quantize")


def prefill_silu_mul_quantize(w: DQWeights, GU: torch.Tensor, act_global_scale: float, workspace: torch.Tensor, stream=None):
    """dq_prefill_silu_mul_quantize: SiLU(gate) * up fused with stage 1 of the prefill linear (GU = [gate | up])."""
    assert GU.is_cuda and GU.dtype == torch.bfloat16 and GU.stride(1) == 1 and GU.shape[1] == 2 * w.K
    _check(lib().dq_prefill_silu_mul_quantize(w.handle, GU.data_ptr(), GU.shape[0], GU.stride(0), float(act_global_scale),
                                              workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)),
           "dq_prefill_silu_mul_quantize")


def gate_up_row_order(F: int) -> torch.Tensor:
    """Row order dq_prefill_gemm_silu_mul_quantize expects of a fused gate/up matrix: entry r of the result is the row
    of [gate; up] (gate rows 0..F-1, up rows F..2F-1) that goes to row r, i.e. row 256 t + 128 h + 64 p + j holds
    gate (p = 0) or up (p = 1) of feature 128 t + 64 h + j.  Index arithmetic only."""
    assert F % 128 == 0
    r = torch.arange(2 * F)
    t, h, p, j = r // 256, (r // 128) % 2, (r // 64) % 2, r % 64
    return p * F + 128 * t + 64 * h + j


def prefill_gemm_silu_mul_quantize(w_gate_up: DQWeights, M: int, act_global_scale: float, workspace: torch.Tensor,
                                   w_down: DQWeights, out_global_scale: float, out_workspace: torch.Tensor, stream=None):
    """dq_prefill_gemm_silu_mul_quantize: the gate/up GEMM with SiLU(gate) * up and the down projection's activation
    quantiser in its epilogue; follow with prefill_gemm(w_down, M, out_global_scale, Y, out_workspace)."""
    _check(lib().dq_prefill_gemm_silu_mul_quantize(w_gate_up.handle, M, float(act_global_scale), workspace.data_ptr(),
                                                   workspace.numel(), w_down.handle, float(out_global_scale),
                                                   out_workspace.data_ptr(), out_workspace.numel(), _stream_ptr(stream)),
           "dq_prefill_gemm_silu_mul_quantize")


def test_silu(g: torch.Tensor, stream=None) -> torch.Tensor:
    """dq_test_silu: the device SiLU of the gated quantisers, value by value (fp32)."""
    assert g.is_cuda and g.dtype == torch.bfloat16 and g.is_contiguous()
    out = torch.empty(g.numel(), dtype=torch.float32, device=g.device)
    _check(lib().dq_test_silu(g.data_ptr(), g.numel(), out.data_ptr(), _stream_ptr(stream)), "dq_test_silu")
    return out


def rmsnorm_quantize_activations(X: torch.Tensor, gamma: torch.Tensor, eps: float, act_global_scale: float, stream=None):
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=X.device)
    scales = torch.empty(M, K // 16, dtype=torch.uint8, device=X.device)
    _check(lib().dq_rmsnorm_quantize_activations(X.data_ptr(), M, K, X.stride(0), gamma.data_ptr(), float(eps),
                                                 float(act_global_scale), codes.data_ptr(), scales.data_ptr(),
                                                 _stream_ptr(stream)), "dq_rmsnorm_quantize_activations")
    return codes, scales


def silu_mul_quantize_activations(GU: torch.Tensor, act_global_scale: float, stream=None):
    assert GU.is_cuda and GU.dtype == torch.bfloat16 and GU.dim() == 2 and GU.stride(1) == 1 and GU.shape[1] % 2 == 0
    M, F = GU.shape[0], GU.shape[1] // 2
    codes = torch.empty(M, F // 2, dtype=torch.uint8, device=GU.device)
    scales = torch.empty(M, F // 16, dtype=torch.uint8, device=GU.device)
    _check(lib().dq_silu_mul_quantize_activations(GU.data_ptr(), M, F, GU.stride(0), float(act_global_scale),
                                                  codes.data_ptr(), scales.data_ptr(), _stream_ptr(stream)),
           "dq_silu_mul_quantize_activations")
    return codes, scales


def prefill_gemm(w: DQWeights, M: int, act_global_scale: float, out: torch.Tensor, workspace: torch.Tensor,
                 stream=None):
    """dq_prefill_gemm: stage 2 of the prefill linear (block-scaled FP4 GEMM)."""
    _check(lib().dq_prefill_gemm(w.handle, M, float(act_global_scale), out.data_ptr(), out.stride(0),
                                 workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)), "dq_prefill_gemm")


def decode_linear(w: DQWeights, X: torch.Tensor, out: torch.Tensor = None, stream=None) -> torch.Tensor:
    """dq_decode_linear: Y = X @ LUT3(W)^T, bf16 out, batch 1..64."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    B = X.shape[0]
    if out is None:
        out = torch.empty(B, w.N, dtype=torch.bfloat16, device=X.device)
    _check(lib().dq_decode_linear(w.handle, X.data_ptr(), B, X.stride(0), out.data_ptr(), out.stride(0),
                                  _stream_ptr(stream)), "dq_decode_linear")
    return out


def decode_linear_nvfp4(w: DQWeights, X: torch.Tensor, out: torch.Tensor = None, stream=None) -> torch.Tensor:
    """dq_decode_linear_nvfp4: Y = X @ NVFP4(W)^T (weight-only NVFP4A16), bf16 out, batch 1..64."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    B = X.shape[0]
    if out is None:
        out = torch.empty(B, w.N, dtype=torch.bfloat16, device=X.device)
    _check(lib().dq_decode_linear_nvfp4(w.handle, X.data_ptr(), B, X.stride(0), out.data_ptr(), out.stride(0),
                                        _stream_ptr(stream)), "dq_decode_linear_nvfp4")
    return out


def decode_linear_lut2(w: DQWeights, X: torch.Tensor, out: torch.Tensor = None, stream=None) -> torch.Tensor:
    """dq_decode_linear_lut2: Y = X @ LUT2(W)^T, bf16 out, batch 1..64."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    B = X.shape[0]
    if out is None:
        out = torch.empty(B, w.N, dtype=torch.bfloat16, device=X.device)
    _check(lib().dq_decode_linear_lut2(w.handle, X.data_ptr(), B, X.stride(0), out.data_ptr(), out.stride(0),
                                       _stream_ptr(stream)), "dq_decode_linear_lut2")
    return out


def test_decode_linear(w: DQWeights, fmt: int, X: torch.Tensor, out: torch.Tensor = None, variant: int = 0,
                       warps_per_group: int = 0, groups_per_cta: int = 0, ring_stages: int = 0, wait_cycles: int = 0,
                       stream=None) -> torch.Tensor:
    """dq_test_decode_linear: a decode call with forced launch parameters (test hook)."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1 and X.shape[1] == w.K
    B = X.shape[0]
    if out is None:
        out = torch.empty(B, w.N, dtype=torch.bfloat16, device=X.device)
    _check(lib().dq_test_decode_linear(w.handle, fmt, variant, warps_per_group, groups_per_cta, ring_stages,
                                       int(wait_cycles), X.data_ptr(), B, X.stride(0), out.data_ptr(), out.stride(0),
                                       _stream_ptr(stream)), "dq_test_decode_linear")
    return out


test_decode_linear.__test__ = False      # not a pytest test
test_silu.__test__ = False


def bench_gemm_clocks(stream=None):
    """dq_bench_gemm_clocks: (SM clock cycles, nanoseconds) the last CTA-pair GEMM launch took on its first CTA's SM."""
    cyc, ns = C.c_ulonglong(0), C.c_ulonglong(0)
    _check(lib().dq_bench_gemm_clocks(_stream_ptr(stream), C.byref(cyc), C.byref(ns)), "dq_bench_gemm_clocks")
    return int(cyc.value), int(ns.value)


def bench_gemm_mma_only(w: DQWeights, M: int, out: torch.Tensor, workspace: torch.Tensor, stream=None):
    """dq_bench_gemm_mma_only: the GEMM kernel's MMA issue sequence alone (measurement hook; `out` is not written)."""
    _check(lib().dq_bench_gemm_mma_only(w.handle, M, out.data_ptr(), out.stride(0), workspace.data_ptr(),
                                        workspace.numel(), _stream_ptr(stream)), "dq_bench_gemm_mma_only")


def bench_stream_read(src: torch.Tensor, scratch: torch.Tensor, stream=None):
    """dq_bench_stream_read: read `src` once with 128-bit loads (measurement hook); scratch: >= 8 bytes on the device."""
    _check(lib().dq_bench_stream_read(src.data_ptr(), src.numel() * src.element_size(), scratch.data_ptr(),
                                      _stream_ptr(stream)), "dq_bench_stream_read")


def prefill_host_staging_bytes(w: DQWeights, M: int) -> int:
    out = C.c_size_t(0)
    _check(lib().dq_prefill_host_staging_bytes(w.handle, M, C.byref(out)), "dq_prefill_host_staging_bytes")
    return int(out.value)


def prefill_linear_host(w: DQWeights, A_host: torch.Tensor, act_global_scale: float, Y_host: torch.Tensor,
                        staging: torch.Tensor, stream=None) -> torch.Tensor:
    """dq_prefill_linear_host: A_host / Y_host are (pinned) CPU tensors, staging a CUDA byte buffer."""
    assert not A_host.is_cuda and not Y_host.is_cuda and staging.is_cuda
    assert A_host.dtype == torch.bfloat16 and Y_host.dtype == torch.bfloat16 and A_host.stride(1) == 1
    M = A_host.shape[0]
    _check(lib().dq_prefill_linear_host(w.handle, A_host.data_ptr(), M, A_host.stride(0), float(act_global_scale),
                                        Y_host.data_ptr(), Y_host.stride(0), staging.data_ptr(), staging.numel(),
                                        _stream_ptr(stream)), "dq_prefill_linear_host")
    return Y_host


def decode_linear_host(w: DQWeights, X_host: torch.Tensor, Y_host: torch.Tensor, staging: torch.Tensor, stream=None):
    """dq_decode_linear_host: X_host / Y_host are (pinned) CPU tensors, staging a CUDA byte buffer."""
    assert not X_host.is_cuda and not Y_host.is_cuda and staging.is_cuda
    _check(lib().dq_decode_linear_host(w.handle, X_host.data_ptr(), X_host.shape[0], X_host.stride(0),
                                       Y_host.data_ptr(), Y_host.stride(0), staging.data_ptr(), staging.numel(),
                                       _stream_ptr(stream)), "dq_decode_linear_host")
    return Y_host


def export_canonical(w: DQWeights, fmt: int, stream=None):
    """Returns (codes, scales, s) in the canonical layouts of include/dq.h (CUDA tensors)."""
    dev = w.packed.device
    if fmt in (FMT_NVFP4, FMT_NVFP4_FROM_LUT3):
        codes = torch.empty(w.N, w.K // 2, dtype=torch.uint8, device=dev)
    else:
        codes = torch.empty(w.N, 3 if fmt == FMT_LUT3 else 2, w.K // 32, dtype=torch.int32, device=dev)
    scales = torch.empty(w.N, w.K // 16, dtype=torch.uint8, device=dev)
    s = torch.empty(1, dtype=torch.float32, device=dev)
    _check(lib().dq_export_canonical(w.handle, fmt, codes.data_ptr(), scales.data_ptr(), s.data_ptr(),
                                     _stream_ptr(stream)), "dq_export_canonical")
    return codes, scales, s


def quantize_activations(A: torch.Tensor, act_global_scale: float, stream=None):
    assert A.is_cuda and A.dtype == torch.bfloat16 and A.dim() == 2 and A.stride(1) == 1
    M, K = A.shape
    codes = torch.empty(M, K // 2, dtype=torch.uint8, device=A.device)
    scales = torch.empty(M, K // 16, dtype=torch.uint8, device=A.device)
    _check(lib().dq_quantize_activations(A.data_ptr(), M, K, A.stride(0), float(act_global_scale), codes.data_ptr(),
                                         scales.data_ptr(), _stream_ptr(stream)), "dq_quantize_activations")
    return codes, scales


def get_status(stream=None):
    st, det = C.c_int(0), C.c_int(0)
    _check(lib().dq_get_status(_stream_ptr(stream), C.byref(st), C.byref(det)), "dq_get_status")
    return int(st.value), int(det.value)
