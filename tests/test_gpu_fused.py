"""GPU parity of the fused activation stages (RMSNorm / SiLU(gate)*up in front of the NVFP4 quantiser, App. C.1):
codes and scales bit for bit against the oracle, and the prefill linear built on them against the oracle's fp64
product, through the C ABI."""
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
    assert torch.cuda.is_available() and torch.cuda.get_device_capability(0) == (10, 0)
    return dq


def _np(t):
    return t.detach().cpu().numpy()


def _status_ok(dq):
    torch.cuda.synchronize()
    st, det = dq.get_status()
    assert st == 0, f"device status {dq.status_string(st)} detail {det}"


def _gamma(K, seed):
    return (dq_inputs.gaussian_bf16(1, K, 0.3, seed)[0].float() + 1.0).to(torch.bfloat16)


@pytest.mark.parametrize("M,K,kind", [(64, 256, "gauss"), (300, 640, "gauss"), (129, 5120, "gauss"), (33, 17408, "student"),
                                        (5, 33024, "gauss")])   # one block per thread, two per thread, the two-pass kernel
def test_rmsnorm_quantiser_bit_exact(dq, oracle, M, K, kind):
    X = dq_inputs.gaussian_bf16(M, K, 1.0, 400 + M) if kind == "gauss" else dq_inputs.student_t_outlier_bf16(M, K, 401)
    X[0] = 0                                              # a zero row: eps keeps it finite
    X[1] = X[1] * 300.0                                   # rows of very different magnitude normalise alike
    gamma = _gamma(K, 402)
    eps = 1e-6
    Xf, gf = dq_inputs.bf16_to_f32_numpy(X), dq_inputs.bf16_to_f32_numpy(gamma[None])[0]
    h = oracle.rmsnorm_bf16(Xf, gf, eps)
    sa = float(np.abs(h).max()) / 2688.0
    big = torch.zeros(M, K + 64, dtype=torch.bfloat16, device=DEV)      # strided rows
    big[:, :K] = X.to(DEV)
    codes, scales = dq.rmsnorm_quantize_activations(big[:, :K], gamma.to(DEV), eps, sa)
    _status_ok(dq)
    rc, rs = oracle.quant_nvfp4(h, sa)
    assert np.array_equal(_np(scales), rs)
    assert np.array_equal(_np(codes), rc)


@pytest.mark.parametrize("M,F", [(64, 256), (300, 640), (130, 17408)])
def test_silu_mul_quantiser_bit_exact(dq, oracle, M, F):
    GU = dq_inputs.gaussian_bf16(M, 2 * F, 2.0, 410 + M)
    GU[0, :16] = 0
    GU[1, :32] = torch.tensor([-200.0, -100.0, -90.0, -88.0, -87.0, -50.0, -20.0, -1e-3, 1e-3, 20.0, 50.0, 87.0, 88.0, 90.0, 100.0, 3e4] * 2)
    h = oracle.silu_mul_bf16(dq_inputs.bf16_to_f32_numpy(GU))
    sa = float(np.abs(h).max()) / 2688.0
    codes, scales = dq.silu_mul_quantize_activations(GU.to(DEV), sa)
    _status_ok(dq)
    rc, rs = oracle.quant_nvfp4(h, sa)
    assert np.array_equal(_np(scales), rs)
    assert np.array_equal(_np(codes), rc)


def test_prefill_linear_on_fused_stages(dq, oracle):
    """RMSNorm -> gate/up projection -> SiLU*up -> down projection, the activation stages fused: each GEMM output
    against the oracle's product of the oracle's quantised operands; same bits as quantising the bf16 intermediate."""
    M, H, F = 320, 512, 1024
    Wgu = dq_inputs.gaussian_bf16(2 * F, H, 0.02, 420)
    Wd = dq_inputs.gaussian_bf16(H, F, 0.02, 421)
    X = dq_inputs.gaussian_bf16(M, H, 1.0, 422)
    gamma = _gamma(H, 423)
    eps = 1e-5
    w_gu = dq.pack_weights(Wgu.to(DEV), formats=dq.FMT_NVFP4)
    w_d = dq.pack_weights(Wd.to(DEV), formats=dq.FMT_NVFP4)
    ref_gu = oracle.pack_weights(dq_inputs.bf16_to_f32_numpy(Wgu))
    ref_d = oracle.pack_weights(dq_inputs.bf16_to_f32_numpy(Wd))
    # stage 1: fused norm + quant, then the gate/up GEMM
    h = oracle.rmsnorm_bf16(dq_inputs.bf16_to_f32_numpy(X), dq_inputs.bf16_to_f32_numpy(gamma[None])[0], eps)
    sa1 = float(np.abs(h).max()) / 2688.0
    ws = dq.alloc_workspace(max(dq.prefill_workspace_bytes(w_gu, M), dq.prefill_workspace_bytes(w_d, M)), DEV)
    GU = torch.empty(M, 2 * F, dtype=torch.bfloat16, device=DEV)
    dq.prefill_rmsnorm_quantize(w_gu, X.to(DEV), gamma.to(DEV), eps, sa1, ws)
    dq.prefill_gemm(w_gu, M, sa1, GU, ws)
    _status_ok(dq)
    Yr, S = oracle.prefill_linear(h, sa1, ref_gu["nvfp4_codes"], ref_gu["nvfp4_scales"], ref_gu["s"])
    check_outputs(GU.float().cpu().numpy().astype(np.float64), Yr, S, "gate/up projection on fused norm + quant")
    # the unfused route gives the same bits
    H_dev = torch.from_numpy(h).to(torch.bfloat16).to(DEV)
    assert torch.equal(dq.prefill_linear(w_gu, H_dev, sa1), GU)
    # stage 2: fused SiLU*up + quant on the GPU's own gate/up output, then the down GEMM
    a2 = oracle.silu_mul_bf16(dq_inputs.bf16_to_f32_numpy(GU.cpu()))
    sa2 = float(np.abs(a2).max()) / 2688.0
    Y = torch.empty(M, H, dtype=torch.bfloat16, device=DEV)
    dq.prefill_silu_mul_quantize(w_d, GU, sa2, ws)
    dq.prefill_gemm(w_d, M, sa2, Y, ws)
    _status_ok(dq)
    Yr, S = oracle.prefill_linear(a2, sa2, ref_d["nvfp4_codes"], ref_d["nvfp4_scales"], ref_d["s"])
    check_outputs(Y.float().cpu().numpy().astype(np.float64), Yr, S, "down projection on fused SiLU*up + quant")
    A2_dev = torch.from_numpy(a2).to(torch.bfloat16).to(DEV)
    assert torch.equal(dq.prefill_linear(w_d, A2_dev, sa2), Y)
    # a row stride below 2 K is rejected before anything is launched
    rc = dq.lib().dq_prefill_silu_mul_quantize(w_d.handle, GU.data_ptr(), M, F, float(sa2), ws.data_ptr(), ws.numel(), None)
    assert rc == 3
