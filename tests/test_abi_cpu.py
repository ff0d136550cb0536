"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every
symbol include/dq.h declares, and validates arguments before touching a device."""
import ctypes as C
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def dq():
    import __graft_entry__ as g
    g.build()
    import paper_2609_26333_b200 as dq
    return dq


def test_library_exports_every_declared_symbol(dq):
    header = (ROOT / "include" / "dq.h").read_text()
    declared = set(re.findall(r"\b(dq_[a-z0-9_]+)\s*\(", header))
    declared -= {"dq_status", "dq_format", "dq_dtype"}
    assert {"dq_pack_weights", "dq_prefill_linear", "dq_decode_linear"} <= declared
    from paper_2609_26333_b200 import binding
    assert declared == set(binding.SYMBOLS)
    L = dq.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert dq.version() >= 100
    assert dq.status_string(0) == "ok" and "shape" in dq.status_string(2)


def test_library_exports_nothing_the_header_does_not_declare(dq):
    """Every dynamic symbol named dq_* of libdq.so is declared in include/dq.h (no hidden switches)."""
    import subprocess
    header = (ROOT / "include" / "dq.h").read_text()
    declared = set(re.findall(r"\b(dq_[a-z0-9_]+)\s*\(", header))
    from paper_2609_26333_b200 import binding
    out = subprocess.run(["nm", "-D", "--defined-only", str(binding._LIB_PATH)], capture_output=True, text=True, check=True).stdout
    exported = {line.split()[-1] for line in out.splitlines() if line.split() and line.split()[-1].startswith("dq_")}
    assert exported, "nm listed no dq_* symbol"
    assert exported <= declared, sorted(exported - declared)


def test_packed_bytes_follows_storage_cost(dq):
    N, K = 6144, 4096
    nv = dq.packed_bytes(N, K, dq.FMT_NVFP4) - 1024
    lut = dq.packed_bytes(N, K, dq.FMT_LUT3) - 1024
    lut2 = dq.packed_bytes(N, K, dq.FMT_LUT2) - 1024
    assert nv == N * K // 2 + N * K // 16           # 4.5 bit per weight
    assert lut == 3 * N * K // 8 + N * K // 16      # 3.5 bit per weight
    assert lut2 == 2 * N * K // 8 + N * K // 16     # 2.5 bit per weight
    assert dq.packed_bytes(N, K, dq.FMT_NVFP4 | dq.FMT_LUT3) == 1024 + nv + lut
    assert dq.packed_bytes(N, K, dq.FMT_NVFP4_FROM_LUT3) == 1024 + nv + lut
    assert dq.packed_bytes(N, K, dq.FMT_LUT3 | dq.FMT_LUT2) == 1024 + lut + lut2


def test_argument_validation_needs_no_device(dq):
    L = dq.lib()
    out = C.c_size_t(0)
    assert L.dq_packed_bytes(512, 200, 3, C.byref(out)) == 2          # K % 128
    assert L.dq_packed_bytes(500, 256, 3, C.byref(out)) == 2          # N % 16
    assert L.dq_packed_bytes(512, 256, 0, C.byref(out)) == 1          # no format
    assert L.dq_packed_bytes(512, 256, 1 | 4, C.byref(out)) == 1      # two NVFP4 views
    assert L.dq_packed_bytes(512, 256, 3, None) == 1
    assert L.dq_packed_bytes(512, 32768 + 128, 1, C.byref(out)) == 0  # NVFP4 alone has no K limit
    assert L.dq_packed_bytes(512, 32768 + 128, 2, C.byref(out)) == 2  # LUT decode keeps a row of K in shared memory
    assert L.dq_packed_bytes(512, 32768 + 128, 8, C.byref(out)) == 2
    assert L.dq_packed_bytes(512, 256, 16, C.byref(out)) == 1         # unknown format bit
    h = C.c_void_p(0)
    assert L.dq_pack_weights(None, 0, 512, 256, 256, 3, None, None, 0, None, C.byref(h)) == 1
    assert L.dq_pack_weights(4096, 7, 512, 256, 256, 3, None, 4096, 1 << 20, None, C.byref(h)) == 1   # dtype
    assert L.dq_pack_weights(4096, 0, 512, 256, 250, 3, None, 4096, 1 << 20, None, C.byref(h)) == 3   # ldw
    assert L.dq_pack_weights(4100, 0, 512, 256, 256, 3, None, 4096, 1 << 20, None, C.byref(h)) == 3   # W alignment
    assert L.dq_pack_weights(4096, 0, 512, 256, 256, 3, None, 4096 + 16, 1 << 20, None, C.byref(h)) == 3
    bad_cb = (C.c_uint16 * 8)(0, 1, 2, 3, 4, 5, 6, 7)
    assert L.dq_pack_weights(4096, 0, 512, 256, 256, 3, bad_cb, 4096, 1 << 20, None, C.byref(h)) == 1
    assert L.dq_free_weights(None) == 1
    assert L.dq_prefill_linear(None, 4096, 1, 256, 1.0, 4096, 512, 4096, 0, None) == 1
    assert L.dq_decode_linear(None, 4096, 1, 256, 4096, 512, None) == 1
    assert L.dq_decode_linear_lut2(None, 4096, 1, 256, 4096, 512, None) == 1
    assert L.dq_test_decode_linear(None, 2, 0, 0, 0, 0, 0, 4096, 1, 256, 4096, 512, None) == 1
    assert L.dq_quantize_activations(4096, 4, 200, 200, 1.0, 4096, 4096, None) == 2
    assert L.dq_quantize_activations(4096, 4, 256, 256, 0.0, 4096, 4096, None) == 1
    assert L.dq_quantize_activations(4096, 4, 256, 256, float("nan"), 4096, 4096, None) == 1


def test_binding_fails_loudly_without_library(dq, tmp_path, monkeypatch):
    from paper_2609_26333_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "missing.so")
    with pytest.raises(ImportError):
        binding.lib()


def test_gate_up_row_order_is_the_documented_interleave(dq):
    """Row 256 t + 128 h + 64 p + j of the interleaved gate/up matrix is gate (p = 0) or up (p = 1) of feature
    128 t + 64 h + j: a permutation of the 2F rows of [gate; up] in which every 256-row tile holds both halves of the
    same 128 features, each 128-column half of a tile gate and up of the same 64."""
    import torch
    F = 384
    order = dq.gate_up_row_order(F)
    assert sorted(order.tolist()) == list(range(2 * F))
    for r in (0, 63, 64, 127, 128, 191, 192, 255, 256, 700):
        t, h, p, j = r // 256, (r // 128) % 2, (r // 64) % 2, r % 64
        assert int(order[r]) == p * F + 128 * t + 64 * h + j
    for tile in range(2 * F // 256):
        rows = order[256 * tile: 256 * (tile + 1)]
        feats = rows % F
        assert sorted(set(feats.tolist())) == list(range(128 * tile, 128 * (tile + 1)))
        for half in range(2):
            g, u = rows[128 * half: 128 * half + 64], rows[128 * half + 64: 128 * half + 128]
            assert torch.all(g < F) and torch.all(u >= F) and torch.equal(g, u - F)
    with pytest.raises(AssertionError):
        dq.gate_up_row_order(200)


def test_gated_gemm_entry_point_rejects_bad_arguments_without_a_device(dq):
    L = dq.lib()
    assert L.dq_prefill_gemm_silu_mul_quantize(None, 1, C.c_float(1.0), None, 0, None, C.c_float(1.0), None, 0, None) == 1
    cyc, ns = C.c_ulonglong(0), C.c_ulonglong(0)
    assert L.dq_bench_gemm_clocks(None, None, C.byref(ns)) == 1
    assert L.dq_test_silu(None, 0, None, None) == 1
