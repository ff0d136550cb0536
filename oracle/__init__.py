"""CPU oracle for the format-disaggregated quantized linear layer.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
bench's CPU-baseline / reference legs.  The product path never imports it and
it imports nothing from the CUDA package.

The arithmetic lives in ``dq_oracle.c`` (plain C, scalar loops); this file only
marshals numpy arrays into it.  Every function names the passage of the paper
it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "dq_oracle.c"
_LIB = _HERE / "libdq_oracle.so"

BLOCK = 16                      # App. A.3: groups of 16 along the contraction dim
E2M1_MAGNITUDES = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)   # App. A.3 "NVFP4"


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (no FMA contraction, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-o", str(_LIB), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        c = ctypes
        f32p, u8p, u16p, u32p, f64p = (c.POINTER(c.c_float), c.POINTER(c.c_uint8), c.POINTER(c.c_uint16),
                                       c.POINTER(c.c_uint32), c.POINTER(c.c_double))
        i64 = c.c_int64
        L.dqo_e2m1_decode.restype = c.c_float
        L.dqo_e2m1_decode.argtypes = [c.c_uint8]
        L.dqo_e2m1_encode.restype = c.c_uint8
        L.dqo_e2m1_encode.argtypes = [c.c_float]
        L.dqo_e4m3_decode.restype = c.c_float
        L.dqo_e4m3_decode.argtypes = [c.c_uint8]
        L.dqo_e4m3_encode.restype = c.c_uint8
        L.dqo_e4m3_encode.argtypes = [c.c_float]
        L.dqo_f16_decode.restype = c.c_float
        L.dqo_f16_decode.argtypes = [c.c_uint16]
        L.dqo_f16_encode.restype = c.c_uint16
        L.dqo_f16_encode.argtypes = [c.c_float]
        L.dqo_bf16_decode.restype = c.c_float
        L.dqo_bf16_decode.argtypes = [c.c_uint16]
        L.dqo_bf16_encode.restype = c.c_uint16
        L.dqo_bf16_encode.argtypes = [c.c_float]
        L.dqo_lut3_default_codebook.restype = None
        L.dqo_lut3_default_codebook.argtypes = [u16p]
        L.dqo_absmax.restype = c.c_float
        L.dqo_absmax.argtypes = [f32p, i64, i64, i64]
        L.dqo_global_scale.restype = c.c_float
        L.dqo_global_scale.argtypes = [c.c_float]
        L.dqo_quant_nvfp4.restype = None
        L.dqo_quant_nvfp4.argtypes = [f32p, i64, i64, i64, c.c_float, u8p, u8p]
        L.dqo_quant_lut3.restype = None
        L.dqo_quant_lut3.argtypes = [f32p, i64, i64, i64, c.c_float, u16p, u32p, u8p]
        L.dqo_lut2_default_codebook.restype = None
        L.dqo_lut2_default_codebook.argtypes = [u16p]
        L.dqo_quant_lut2.restype = None
        L.dqo_quant_lut2.argtypes = [f32p, i64, i64, i64, c.c_float, u16p, u32p, u8p]
        L.dqo_dequant_lut2.restype = None
        L.dqo_dequant_lut2.argtypes = [u32p, u8p, i64, i64, c.c_float, u16p, f64p]
        L.dqo_rmsnorm_bf16.restype = None
        L.dqo_rmsnorm_bf16.argtypes = [f32p, i64, i64, i64, f32p, c.c_float, f32p]
        L.dqo_silu_f32.restype = c.c_float
        L.dqo_silu_f32.argtypes = [c.c_float]
        L.dqo_silu_mul_bf16.restype = None
        L.dqo_silu_mul_bf16.argtypes = [f32p, i64, i64, i64, f32p]
        L.dqo_autocast_lut3_to_nvfp4.restype = None
        L.dqo_autocast_lut3_to_nvfp4.argtypes = [u32p, u8p, i64, i64, u16p, u8p, u8p]
        L.dqo_dequant_nvfp4.restype = None
        L.dqo_dequant_nvfp4.argtypes = [u8p, u8p, i64, i64, c.c_float, f64p]
        L.dqo_dequant_lut3.restype = None
        L.dqo_dequant_lut3.argtypes = [u32p, u8p, i64, i64, c.c_float, u16p, f64p]
        L.dqo_matmul_nt.restype = None
        L.dqo_matmul_nt.argtypes = [f64p, i64, i64, f64p, i64, f64p, f64p]
        L.dqo_num_threads.restype = c.c_int
        L.dqo_num_threads.argtypes = []
        _lib = L
    return _lib


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def _f32_2d(x) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert x.ndim == 2
    return x


# ---------------------------------------------------------------- codecs

def e2m1_decode(code: int) -> float:
    """E2M1 code (sign<<3 | magnitude index) -> value (App. A.3 "NVFP4")."""
    return float(lib().dqo_e2m1_decode(code))


def e2m1_encode(y: float) -> int:
    return int(lib().dqo_e2m1_encode(np.float32(y)))


def e4m3_decode(b: int) -> float:
    """E4M3 byte -> value (the FP8 block-scale type of App. A.3)."""
    return float(lib().dqo_e4m3_decode(b))


def e4m3_encode(t: float) -> int:
    return int(lib().dqo_e4m3_encode(np.float32(t)))


def f16_decode(h: int) -> float:
    return float(lib().dqo_f16_decode(h))


def f16_encode(x: float) -> int:
    return int(lib().dqo_f16_encode(np.float32(x)))


def bf16_decode(b: int) -> float:
    return float(lib().dqo_bf16_decode(b))


def bf16_encode(x: float) -> int:
    return int(lib().dqo_bf16_encode(np.float32(x)))


def lut3_default_codebook() -> np.ndarray:
    """The LUT3A16 grid of App. A.3 rounded to fp16, as uint16 bit patterns."""
    cb = np.zeros(8, dtype=np.uint16)
    lib().dqo_lut3_default_codebook(_p(cb, ctypes.c_uint16))
    return cb


def lut2_default_codebook() -> np.ndarray:
    """The LUT2A16 grid of App. A.3 rounded to fp16, as uint16 bit patterns."""
    cb = np.zeros(4, dtype=np.uint16)
    lib().dqo_lut2_default_codebook(_p(cb, ctypes.c_uint16))
    return cb


def codebook_values(codebook_f16: np.ndarray) -> np.ndarray:
    return np.array([f16_decode(int(h)) for h in codebook_f16], dtype=np.float64)


# ---------------------------------------------------------------- scales

def absmax(x) -> float:
    x = _f32_2d(x)
    return float(lib().dqo_absmax(_p(x, ctypes.c_float), x.shape[0], x.shape[1], x.shape[1]))


def global_scale(amax: float) -> float:
    """s = max|W| / (6*448) (App. A.3 two-level scaling); 1 for an all-zero tensor."""
    return float(lib().dqo_global_scale(np.float32(amax)))


# ------------------------------------------------------------ quantisers

def quant_nvfp4(x, s: float):
    """RTN NVFP4 of a (rows, K) fp32 matrix with tensor scale ``s``.

    Returns (codes uint8[rows, K/2], scales uint8[rows, K/16])."""
    x = _f32_2d(x)
    rows, K = x.shape
    assert K % BLOCK == 0
    codes = np.zeros((rows, K // 2), dtype=np.uint8)
    scales = np.zeros((rows, K // BLOCK), dtype=np.uint8)
    lib().dqo_quant_nvfp4(_p(x, ctypes.c_float), rows, K, K, np.float32(s),
                          _p(codes, ctypes.c_uint8), _p(scales, ctypes.c_uint8))
    return codes, scales


def quant_lut3(x, s: float, codebook_f16=None):
    """RTN LUT3 of a (rows, K) fp32 matrix.

    Returns (planes uint32[rows, 3, K/32], scales uint8[rows, K/16] signed E4M3)."""
    x = _f32_2d(x)
    rows, K = x.shape
    assert K % 32 == 0
    cb = lut3_default_codebook() if codebook_f16 is None else np.ascontiguousarray(codebook_f16, dtype=np.uint16)
    planes = np.zeros((rows, 3, K // 32), dtype=np.uint32)
    scales = np.zeros((rows, K // BLOCK), dtype=np.uint8)
    lib().dqo_quant_lut3(_p(x, ctypes.c_float), rows, K, K, np.float32(s), _p(cb, ctypes.c_uint16),
                         _p(planes, ctypes.c_uint32), _p(scales, ctypes.c_uint8))
    return planes, scales


def quant_lut2(x, s: float, codebook_f16=None):
    """RTN LUT2 of a (rows, K) fp32 matrix (App. A.3 "LUT formats", 4 levels).

    Returns (planes uint32[rows, 2, K/32], scales uint8[rows, K/16] signed E4M3)."""
    x = _f32_2d(x)
    rows, K = x.shape
    assert K % 32 == 0
    cb = lut2_default_codebook() if codebook_f16 is None else np.ascontiguousarray(codebook_f16, dtype=np.uint16)
    planes = np.zeros((rows, 2, K // 32), dtype=np.uint32)
    scales = np.zeros((rows, K // BLOCK), dtype=np.uint8)
    lib().dqo_quant_lut2(_p(x, ctypes.c_float), rows, K, K, np.float32(s), _p(cb, ctypes.c_uint16),
                         _p(planes, ctypes.c_uint32), _p(scales, ctypes.c_uint8))
    return planes, scales


def rmsnorm_bf16(x, gamma, eps: float) -> np.ndarray:
    """RMSNorm of a (rows, K) fp32 matrix (bf16 values) with weight gamma, result rounded to bf16 (App. C.1 fused
    activation processing; fp32 arithmetic as fixed in dq_oracle.c).  Returns fp32 holding bf16 values."""
    x = _f32_2d(x)
    rows, K = x.shape
    assert K % BLOCK == 0
    g = np.ascontiguousarray(gamma, dtype=np.float32)
    assert g.shape == (K,)
    h = np.zeros((rows, K), dtype=np.float32)
    lib().dqo_rmsnorm_bf16(_p(x, ctypes.c_float), rows, K, K, _p(g, ctypes.c_float), np.float32(eps), _p(h, ctypes.c_float))
    return h


def silu_f32(g: float) -> float:
    return float(lib().dqo_silu_f32(np.float32(g)))


def silu_mul_bf16(gate_up) -> np.ndarray:
    """bf16( SiLU(gate) * up ) for a (rows, 2F) fp32 matrix [gate | up] (App. C.1 fused activation processing)."""
    gu = _f32_2d(gate_up)
    rows, F2 = gu.shape
    assert F2 % 2 == 0
    F = F2 // 2
    h = np.zeros((rows, F), dtype=np.float32)
    lib().dqo_silu_mul_bf16(_p(gu, ctypes.c_float), rows, F, F2, _p(h, ctypes.c_float))
    return h


def rmsnorm_quant_nvfp4(x, gamma, eps: float, act_scale: float):
    """Fused RMSNorm + NVFP4 activation quantiser: the quantiser applied to the bf16-rounded norm output."""
    return quant_nvfp4(rmsnorm_bf16(x, gamma, eps), act_scale)


def silu_mul_quant_nvfp4(gate_up, act_scale: float):
    """Fused SiLU(gate)*up + NVFP4 activation quantiser."""
    return quant_nvfp4(silu_mul_bf16(gate_up), act_scale)


def autocast_lut3_to_nvfp4(planes, lut_scales, codebook_f16=None):
    """NVFP4 view of LUT3 weights (Sec. 2.3 autocast). Returns (codes, scales)."""
    planes = np.ascontiguousarray(planes, dtype=np.uint32)
    lut_scales = np.ascontiguousarray(lut_scales, dtype=np.uint8)
    rows, _, W = planes.shape
    K = W * 32
    cb = lut3_default_codebook() if codebook_f16 is None else np.ascontiguousarray(codebook_f16, dtype=np.uint16)
    codes = np.zeros((rows, K // 2), dtype=np.uint8)
    scales = np.zeros((rows, K // BLOCK), dtype=np.uint8)
    lib().dqo_autocast_lut3_to_nvfp4(_p(planes, ctypes.c_uint32), _p(lut_scales, ctypes.c_uint8), rows, K,
                                     _p(cb, ctypes.c_uint16), _p(codes, ctypes.c_uint8), _p(scales, ctypes.c_uint8))
    return codes, scales


# ------------------------------------------------------------ dequantise

def dequant_nvfp4(codes, scales, s: float) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.zeros((rows, K), dtype=np.float64)
    lib().dqo_dequant_nvfp4(_p(codes, ctypes.c_uint8), _p(scales, ctypes.c_uint8), rows, K, np.float32(s),
                            _p(out, ctypes.c_double))
    return out


def dequant_lut3(planes, scales, s: float, codebook_f16=None) -> np.ndarray:
    planes = np.ascontiguousarray(planes, dtype=np.uint32)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rows, K = planes.shape[0], planes.shape[2] * 32
    cb = lut3_default_codebook() if codebook_f16 is None else np.ascontiguousarray(codebook_f16, dtype=np.uint16)
    out = np.zeros((rows, K), dtype=np.float64)
    lib().dqo_dequant_lut3(_p(planes, ctypes.c_uint32), _p(scales, ctypes.c_uint8), rows, K, np.float32(s),
                           _p(cb, ctypes.c_uint16), _p(out, ctypes.c_double))
    return out


def dequant_lut2(planes, scales, s: float, codebook_f16=None) -> np.ndarray:
    planes = np.ascontiguousarray(planes, dtype=np.uint32)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rows, K = planes.shape[0], planes.shape[2] * 32
    cb = lut2_default_codebook() if codebook_f16 is None else np.ascontiguousarray(codebook_f16, dtype=np.uint16)
    out = np.zeros((rows, K), dtype=np.float64)
    lib().dqo_dequant_lut2(_p(planes, ctypes.c_uint32), _p(scales, ctypes.c_uint8), rows, K, np.float32(s),
                           _p(cb, ctypes.c_uint16), _p(out, ctypes.c_double))
    return out


def unpack_lut2_indices(planes) -> np.ndarray:
    """Bit-planes (rows, 2, K/32) -> indices (rows, K), LSB-first (App. C.2 storage)."""
    planes = np.asarray(planes, dtype=np.uint32)
    rows, _, W = planes.shape
    bits = (planes[:, :, :, None] >> np.arange(32, dtype=np.uint32)) & 1      # rows,2,W,32
    idx = bits[:, 0] | (bits[:, 1] << 1)
    return idx.reshape(rows, W * 32).astype(np.uint8)


def unpack_lut3_indices(planes) -> np.ndarray:
    """Bit-planes (rows, 3, K/32) -> indices (rows, K), LSB-first (App. C.2 storage)."""
    planes = np.asarray(planes, dtype=np.uint32)
    rows, _, W = planes.shape
    bits = (planes[:, :, :, None] >> np.arange(32, dtype=np.uint32)) & 1      # rows,3,W,32
    idx = bits[:, 0] | (bits[:, 1] << 1) | (bits[:, 2] << 2)
    return idx.reshape(rows, W * 32).astype(np.uint8)


# -------------------------------------------------------------- products

def matmul_nt(A, W, with_abs: bool = True):
    """Y = A W^T and Sabs = |A| |W|^T in fp64, plain triple loop (the definition)."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    W = np.ascontiguousarray(W, dtype=np.float64)
    M, K = A.shape
    N = W.shape[0]
    assert W.shape[1] == K
    Y = np.zeros((M, N), dtype=np.float64)
    S = np.zeros((M, N), dtype=np.float64) if with_abs else None
    lib().dqo_matmul_nt(_p(A, ctypes.c_double), M, K, _p(W, ctypes.c_double), N, _p(Y, ctypes.c_double),
                        _p(S, ctypes.c_double) if with_abs else None)
    return (Y, S) if with_abs else Y


def matmul_nt_lib(A, W):
    """Same products through the library fp64 matmul (numpy); used where the
    triple loop would take minutes.  tests pin it to ``matmul_nt``."""
    A = np.asarray(A, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    return A @ W.T, np.abs(A) @ np.abs(W).T


def num_threads() -> int:
    return int(lib().dqo_num_threads())


# ------------------------------------------------- whole-layer reference

def pack_weights(W_f32, codebook_f16=None):
    """What the packer must produce for a (fused) weight matrix (App. A.3).

    Returns a dict with the tensor scale and both encodings in canonical layout."""
    W_f32 = _f32_2d(W_f32)
    s = global_scale(absmax(W_f32))
    nv_codes, nv_scales = quant_nvfp4(W_f32, s)
    planes, lut_scales = quant_lut3(W_f32, s, codebook_f16)
    return {"s": s, "nvfp4_codes": nv_codes, "nvfp4_scales": nv_scales,
            "lut3_planes": planes, "lut3_scales": lut_scales}


def prefill_linear(A_f32, act_scale: float, nv_codes, nv_scales, s_w: float, rows=None, lib_matmul=True):
    """Prefill: NVFP4-quantised activations times NVFP4 weights, fp64 (Sec. 2.3)."""
    A_f32 = _f32_2d(A_f32)
    if rows is not None:
        A_f32 = A_f32[rows]
    a_codes, a_scales = quant_nvfp4(A_f32, act_scale)
    Ah = dequant_nvfp4(a_codes, a_scales, act_scale)
    Wh = dequant_nvfp4(nv_codes, nv_scales, s_w)
    return matmul_nt_lib(Ah, Wh) if lib_matmul else matmul_nt(Ah, Wh)


def decode_linear_nvfp4(X_f32, nv_codes, nv_scales, s_w: float, lib_matmul=True):
    """Decode on the NVFP4 view (weight-only NVFP4A16, Sec. 2.3 / Table 1): raw bf16 activations
    times NVFP4-dequantised weights, fp64."""
    X = np.asarray(X_f32, dtype=np.float64)
    Wh = dequant_nvfp4(nv_codes, nv_scales, s_w)
    return matmul_nt_lib(X, Wh) if lib_matmul else matmul_nt(X, Wh)


def decode_linear_lut2(X_f32, planes, lut_scales, s_w: float, codebook_f16=None, lib_matmul=True):
    """Decode: raw bf16 activations times LUT2-dequantised weights, fp64 (App. C.2, Table 1 LUT2 rows)."""
    X = np.asarray(X_f32, dtype=np.float64)
    Wh = dequant_lut2(planes, lut_scales, s_w, codebook_f16)
    return matmul_nt_lib(X, Wh) if lib_matmul else matmul_nt(X, Wh)


def decode_linear(X_f32, planes, lut_scales, s_w: float, codebook_f16=None, lib_matmul=True):
    """Decode: raw bf16 activations times LUT3-dequantised weights, fp64 (App. C.2)."""
    X = np.asarray(X_f32, dtype=np.float64)
    Wh = dequant_lut3(planes, lut_scales, s_w, codebook_f16)
    return matmul_nt_lib(X, Wh) if lib_matmul else matmul_nt(X, Wh)
