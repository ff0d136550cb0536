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


def test_c3_gated_ffn_sampled(dq, oracle):
    """The gated FFN of the bench line (`gated_ffn`: M = 8192, gate/up 34816 x 5120 with interleaved rows, down
    5120 x 17408).  Codes and scales the gated epilogue writes: bit for bit the two-call path's, in full; against the
    oracle (quantised operands, fp64 product, bf16, SiLU*up, NVFP4) on sampled rows, where the GEMM's summation order may
    move one code in ten thousand; the down projection on those rows against the oracle's product."""
    from test_gpu_fused import _workspace_codes_scales
    up_cfg = dq_inputs.LayerConfig("c3_up27b", N=17408, K=5120, M=8192, cfg_id=3, matrix_id=2)
    gate_cfg, down_cfg = dq_inputs.CONFIGS["c3_gate_up27b"], dq_inputs.CONFIGS["c3_down27b"]
    M, F, H = gate_cfg.M, gate_cfg.N, gate_cfg.K
    Wgu = torch.cat([dq_inputs.make_weight(gate_cfg), dq_inputs.make_weight(up_cfg)], 0)         # [gate; up], one tensor
    Wd = dq_inputs.make_weight(down_cfg)
    A = dq_inputs.make_activations(gate_cfg, M)
    sa1 = dq_inputs.static_act_scale(A)
    order = dq.gate_up_row_order(F)
    w_gu = dq.pack_weights(Wgu[order].contiguous().to(DEV), formats=dq.FMT_NVFP4)
    w_d = dq.pack_weights(Wd.to(DEV), formats=dq.FMT_NVFP4)
    ws = dq.alloc_workspace(dq.prefill_workspace_bytes(w_gu, M), DEV)
    ows = dq.alloc_workspace(dq.prefill_workspace_bytes(w_d, M), DEV)
    ows2 = dq.alloc_workspace(dq.prefill_workspace_bytes(w_d, M), DEV)
    dq.prefill_quantize(w_gu, A.to(DEV), sa1, ws)
    # the static scale of the down projection's input: from a calibration pass of the two-call path
    GU_il = torch.empty(M, 2 * F, dtype=torch.bfloat16, device=DEV)
    dq.prefill_gemm(w_gu, M, sa1, GU_il, ws)
    GU = torch.empty_like(GU_il)
    GU[:, order.to(DEV)] = GU_il
    del GU_il
    h_abs = (torch.nn.functional.silu(GU[:, :F].float()) * GU[:, F:].float()).abs().max()
    sa2 = float(h_abs) / 2688.0
    dq.prefill_gemm_silu_mul_quantize(w_gu, M, sa1, ws, w_d, sa2, ows)
    dq.prefill_silu_mul_quantize(w_d, GU, sa2, ows2)
    Y = torch.empty(M, H, dtype=torch.bfloat16, device=DEV)
    dq.prefill_gemm(w_d, M, sa2, Y, ows)
    torch.cuda.synchronize()
    st, det = dq.get_status()
    assert st == 0, (st, det)
    del GU
    codes, scales = _workspace_codes_scales(ows, M, F)
    c2, s2 = _workspace_codes_scales(ows2, M, F)
    assert np.array_equal(codes, c2) and np.array_equal(scales, s2)
    # the oracle on sampled rows
    rng = np.random.default_rng(321)
    rows = np.unique(np.concatenate([rng.choice(M, 24, replace=False), np.array([0, 127, 128, 255, 256, M - 129, M - 128, M - 1])]))
    ref_gu = oracle.pack_weights(dq_inputs.bf16_to_f32_numpy(Wgu))
    Yr, _ = oracle.prefill_linear(dq_inputs.bf16_to_f32_numpy(A), sa1, ref_gu["nvfp4_codes"], ref_gu["nvfp4_scales"], ref_gu["s"],
                                  rows=rows)
    h_ref = oracle.silu_mul_bf16(dq_inputs.bf16_to_f32_numpy(torch.from_numpy(Yr).to(torch.bfloat16)))
    rc, rs = oracle.quant_nvfp4(h_ref, sa2)
    code_diff = np.count_nonzero(((codes[rows] ^ rc) & 0x0F) != 0) + np.count_nonzero(((codes[rows] ^ rc) & 0xF0) != 0)
    scale_diff = np.count_nonzero(scales[rows] != rs)
    assert code_diff <= 1e-4 * rows.size * F, f"{code_diff} of {rows.size * F} codes differ from the oracle's"
    assert scale_diff <= 1e-4 * rows.size * F / 16, f"{scale_diff} block scales differ from the oracle's"
    ref_d = oracle.pack_weights(dq_inputs.bf16_to_f32_numpy(Wd))
    Yd, _ = oracle.prefill_linear(h_ref, sa2, ref_d["nvfp4_codes"], ref_d["nvfp4_scales"], ref_d["s"])
    Yg = _f64(Y[torch.from_numpy(rows).to(DEV)])
    assert np.linalg.norm(Yg - Yd) <= 2.5e-3 * np.linalg.norm(Yd)
