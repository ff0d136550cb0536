"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times
(dq_prefill_quantize + dq_prefill_gemm + dq_decode_linear on one packed layer).
Codes and scales are compared in full; GEMM / GEMV outputs on sampled rows the oracle
computes one by one (all columns of random rows plus the first and last row of tile bands)."""
import numpy as np
import pytest
import torch

import dq_inputs
from parity_utils import check_outputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def dq():
    import __graft_entry__ as g
    g.build()
    import paper_2609_26333_b200 as dq
    assert torch.cuda.is_available()
    return dq


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _run_config(dq, oracle, name, full_rows, layer=0):
    cfg = name if isinstance(name, dq_inputs.LayerConfig) else dq_inputs.CONFIGS[name]
    name = cfg.name
    W = dq_inputs.make_weight(cfg, layer)
    A = dq_inputs.make_activations(cfg, cfg.M, layer=layer)
    X = dq_inputs.make_activations(cfg, max(cfg.decode_batches), salt=2, layer=layer)
    sa = dq_inputs.static_act_scale(A)
    w = dq.pack_weights(W.to(DEV))
    ws = dq.alloc_workspace(dq.prefill_workspace_bytes(w, cfg.M), DEV)
    Y = torch.empty(cfg.M, cfg.N, dtype=torch.bfloat16, device=DEV)
    Ad = A.to(DEV)
    dq.prefill_quantize(w, Ad, sa, ws)
    dq.prefill_gemm(w, cfg.M, sa, Y, ws)
    Yd = {b: dq.decode_linear(w, X[:b].to(DEV)) for b in cfg.decode_batches}
    torch.cuda.synchronize()
    st, det = dq.get_status()
    assert st == 0, (st, det)

    ref = oracle.pack_weights(dq_inputs.bf16_to_f32_numpy(W))
    codes, scales, s = dq.export_canonical(w, dq.FMT_NVFP4)
    planes, lsc, _ = dq.export_canonical(w, dq.FMT_LUT3)
    assert np.float32(s.cpu().numpy()[0]) == np.float32(ref["s"])
    assert np.array_equal(codes.cpu().numpy(), ref["nvfp4_codes"])
    assert np.array_equal(scales.cpu().numpy(), ref["nvfp4_scales"])
    assert np.array_equal(planes.cpu().numpy().view(np.uint32), ref["lut3_planes"])
    assert np.array_equal(lsc.cpu().numpy(), ref["lut3_scales"])

    if full_rows:
        rows = np.arange(cfg.M)
    else:
        rng = np.random.default_rng(123)
        edges = [0, 127, 128, 255, 256, 511, cfg.M // 2 - 1, cfg.M // 2, cfg.M - 257, cfg.M - 256, cfg.M - 1]
        rows = np.unique(np.concatenate([rng.choice(cfg.M, 48, replace=False), np.array(edges)]))
    Yr, S = oracle.prefill_linear(dq_inputs.bf16_to_f32_numpy(A), sa, ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"],
                                  rows=rows)
    check_outputs(_f64(Y[torch.from_numpy(rows).to(DEV)]), Yr, S, f"{name} prefill")
    for b, y in Yd.items():
        Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(X[:b]), ref["lut3_planes"], ref["lut3_scales"], ref["s"])
        check_outputs(_f64(y), Yr, S, f"{name} decode batch {b}")


def test_c2_fused_qkv_full(dq, oracle):
    _run_config(dq, oracle, "c2_qkv8b", full_rows=True)


def test_c3_gate_up_sampled(dq, oracle):
    _run_config(dq, oracle, "c3_gate_up27b", full_rows=False)


def test_c3_down_sampled(dq, oracle):
    _run_config(dq, oracle, "c3_down27b", full_rows=False)


def test_c5_outlier_sampled(dq, oracle):
    """70B-class layer with heavy-tailed activations and x50 outlier channels under a static
    activation scale: block scales saturate and underflow on both sides in the same way."""
    _run_config(dq, oracle, "c5_outlier70b", full_rows=False)


@pytest.mark.parametrize("which", [0, 1, 2, 3])
def test_c4_stack_layer_shapes(dq, oracle, which):
    """The matrices of one layer of the 27B-class stack (fused q/k/v, o, fused gate/up, down) at
    4096 prefill tokens and decode batches 1..64; the other 63 layers repeat these shapes."""
    _run_config(dq, oracle, dq_inputs.c4_fused_layer(layer=3)[which], full_rows=False, layer=3)
