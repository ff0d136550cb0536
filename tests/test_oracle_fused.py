"""Pins for the oracle's fused activation-processing operators (CPU only): RMSNorm and SiLU(gate)*up in front of
the NVFP4 activation quantiser (App. C.1: the prefill stack fuses activation processing with the quantiser).

The operators are defined as "processing step rounded to bf16, then the quantiser"; the processing steps are pinned
against their textbook definitions evaluated in fp64 with numpy and torch."""
import numpy as np
import torch

import dq_inputs


def _bf16(a64):
    return torch.from_numpy(np.asarray(a64, dtype=np.float64)).to(torch.float32).to(torch.bfloat16).float().numpy()


def test_rmsnorm_matches_the_definition_in_fp64(oracle):
    rows, K = 64, 1280                     # 80 blocks: two full groups of 32 and a partial one
    x = dq_inputs.bf16_to_f32_numpy(dq_inputs.gaussian_bf16(rows, K, 1.0, 300))
    x[3] *= 40.0
    x[4] *= 1e-3
    gamma = dq_inputs.bf16_to_f32_numpy(dq_inputs.gaussian_bf16(1, K, 0.3, 301))[0] + 1.0
    eps = 1e-6
    h = oracle.rmsnorm_bf16(x, gamma, eps)
    x64 = x.astype(np.float64)
    ref = x64 / np.sqrt((x64 ** 2).mean(axis=1, keepdims=True) + eps) * gamma.astype(np.float64)
    # the values are bf16 and sit within one bf16 rounding of the exact result ...
    assert np.array_equal(h, _bf16(h))
    assert np.all(np.abs(h - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)
    # ... and almost all of them ARE the correctly rounded result (fp32 arithmetic differs only at rounding boundaries)
    assert (h == _bf16(ref)).mean() > 0.995
    # torch's own rms_norm on the same data agrees to bf16 precision
    tref = torch.nn.functional.rms_norm(torch.from_numpy(x64), (K,), torch.from_numpy(gamma.astype(np.float64)), eps).numpy()
    assert np.allclose(tref, ref, rtol=1e-12)
    # unit rows: x = c * ones -> h = sign(c) * gamma exactly when eps is negligible
    ones = np.full((2, K), 3.0, dtype=np.float32)
    ones[1] = -0.5
    hu = oracle.rmsnorm_bf16(ones, gamma, 0.0)
    assert np.array_equal(hu[0], _bf16(gamma)) and np.array_equal(hu[1], _bf16(-gamma))
    # a zero row stays zero (eps keeps the scale finite)
    assert not oracle.rmsnorm_bf16(np.zeros((1, K), dtype=np.float32), gamma, eps).any()


def test_silu_matches_the_definition_within_a_few_fp32_ulps(oracle):
    g = np.concatenate([np.linspace(-30, 30, 20001), np.array([0.0, 1e-8, -1e-8, 80.0, -80.0, 200.0, -200.0, 1e4, -1e4])])
    g32 = g.astype(np.float32)
    got = np.array([oracle.silu_f32(v) for v in g32], dtype=np.float64)
    g64 = g32.astype(np.float64)
    with np.errstate(over="ignore"):
        ref = g64 / (1.0 + np.exp(-g64))
    ulp = np.spacing(np.abs(ref).astype(np.float32)).astype(np.float64)
    # beyond |g| = 87 the exponent is clamped at 126: the result is |g| * 2^-126 at most instead of an underflow to 0
    assert np.all(np.abs(got - ref) <= 4 * ulp + np.abs(g64) * 2.0 ** -125)
    assert oracle.silu_f32(0.0) == 0.0
    assert oracle.silu_f32(100.0) == 100.0 and abs(oracle.silu_f32(-100.0)) < 1e-35 and oracle.silu_f32(-100.0) <= 0.0
    tr = torch.nn.functional.silu(torch.from_numpy(g64)).numpy()
    assert np.allclose(tr, ref, rtol=1e-12, atol=1e-300)      # the fp64 formula used here is the textbook SiLU


def test_silu_mul_and_fused_quantisers_are_the_two_steps_composed(oracle):
    rows, F = 32, 512
    gu = dq_inputs.bf16_to_f32_numpy(dq_inputs.gaussian_bf16(rows, 2 * F, 2.0, 302))
    h = oracle.silu_mul_bf16(gu)
    g64, u64 = gu[:, :F].astype(np.float64), gu[:, F:].astype(np.float64)
    ref = g64 / (1.0 + np.exp(-g64)) * u64
    assert np.array_equal(h, _bf16(h))
    assert np.all(np.abs(h - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)
    assert (h == _bf16(ref)).mean() > 0.995
    sa = float(np.abs(h).max()) / 2688.0
    c, s = oracle.silu_mul_quant_nvfp4(gu, sa)
    c2, s2 = oracle.quant_nvfp4(h, sa)
    assert np.array_equal(c, c2) and np.array_equal(s, s2)
    x = dq_inputs.bf16_to_f32_numpy(dq_inputs.gaussian_bf16(rows, F, 1.0, 303))
    gamma = np.ones(F, dtype=np.float32)
    hn = oracle.rmsnorm_bf16(x, gamma, 1e-6)
    sn = float(np.abs(hn).max()) / 2688.0
    c, s = oracle.rmsnorm_quant_nvfp4(x, gamma, 1e-6, sn)
    c2, s2 = oracle.quant_nvfp4(hn, sn)
    assert np.array_equal(c, c2) and np.array_equal(s, s2)
    # the quantised norm output dequantises back to the norm output within NVFP4's error
    back = oracle.dequant_nvfp4(c, s, sn)
    assert np.linalg.norm(back - hn) / np.linalg.norm(hn) < 0.12
