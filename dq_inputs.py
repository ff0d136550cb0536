"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side
tests / bench.  Holds none of the method's arithmetic: it only draws tensors.

The paper measures on Qwen3 / Gemma3 / Qwen3.8-27B checkpoints; none of them is
available offline, so layers of the same shapes with Gaussian weights and
Gaussian (or heavy-tailed) activations stand in for them.  All tensors are drawn
in fp32 on the CPU from a seeded ``torch.Generator`` and rounded to bf16; both
sides receive the same bytes.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch


@dataclass(frozen=True)
class LayerConfig:
    name: str
    N: int                     # out features (rows of W)
    K: int                     # in features (contraction)
    M: int                     # prefill tokens
    decode_batches: tuple = (1,)
    act: str = "gauss"         # "gauss" | "student_t_outlier"
    cfg_id: int = 0
    matrix_id: int = 0
    w_std: float = 0.02


CONFIGS = {
    # "Tiny DQ linear": full brute-force parity
    "c1_tiny": LayerConfig("c1_tiny", N=512, K=256, M=64, decode_batches=(1,), cfg_id=0),
    # 8B-class fused QKV
    "c2_qkv8b": LayerConfig("c2_qkv8b", N=6144, K=4096, M=2048, decode_batches=(1, 8), cfg_id=2),
    # 27B-class FFN
    "c3_gate_up27b": LayerConfig("c3_gate_up27b", N=17408, K=5120, M=8192, decode_batches=(1, 4, 16, 40), cfg_id=3,
                                 matrix_id=0),
    "c3_down27b": LayerConfig("c3_down27b", N=5120, K=17408, M=8192, decode_batches=(1, 4, 16), cfg_id=3,
                              matrix_id=1),
    # 70B-class outlier stress
    "c5_outlier70b": LayerConfig("c5_outlier70b", N=28672, K=8192, M=16384, decode_batches=(1,),
                                 act="student_t_outlier", cfg_id=5),
}

# 27B-class full linear stack (hidden 5120, FFN 17408, 64 q heads / 8 kv heads of dim 128)
C4_LAYERS = 64
C4_MATRICES = (("q", 8192, 5120), ("k", 1024, 5120), ("v", 1024, 5120), ("o", 5120, 8192),
               ("gate", 17408, 5120), ("up", 17408, 5120), ("down", 5120, 17408))
C4_PREFILL_M = 4096
C4_DECODE_BATCHES = (1, 2, 4, 8, 16, 32, 64)


def c4_fused_layer(layer: int = 0):
    """The four matrices one layer of the 27B-class stack serves: q/k/v and gate/up are stored
    fused (each fused tensor has one global scale), o and down on their own."""
    shapes = (("qkv", 8192 + 1024 + 1024, 5120), ("o", 5120, 8192), ("gate_up", 2 * 17408, 5120),
              ("down", 5120, 17408))
    return [LayerConfig(f"c4_l{layer}_{nm}", N=n, K=k, M=C4_PREFILL_M, decode_batches=C4_DECODE_BATCHES, cfg_id=4,
                        matrix_id=i) for i, (nm, n, k) in enumerate(shapes)]


def seed_of(cfg: LayerConfig, layer: int = 0) -> int:
    if cfg.cfg_id == 0:
        return 0
    return 1000 * cfg.cfg_id + 10 * layer + cfg.matrix_id


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def gaussian_bf16(rows: int, cols: int, std: float, seed: int) -> torch.Tensor:
    x = torch.randn(rows, cols, generator=_gen(seed), dtype=torch.float32) * std
    return x.to(torch.bfloat16)


def student_t_outlier_bf16(rows: int, cols: int, seed: int, nu: int = 3, frac: float = 0.01,
                           gain: float = 50.0) -> torch.Tensor:
    """Student-t(nu) entries; a seeded 1 % of the K channels (columns) scaled x50."""
    g = _gen(seed)
    z = torch.randn(rows, cols, generator=g, dtype=torch.float32)
    chi = torch.zeros(rows, cols, dtype=torch.float32)
    for _ in range(nu):
        chi += torch.randn(rows, cols, generator=g, dtype=torch.float32) ** 2
    x = z / torch.sqrt(chi / nu)
    n_out = max(1, int(round(frac * cols)))
    perm = torch.randperm(cols, generator=g)[:n_out]
    x[:, perm] *= gain
    return x.to(torch.bfloat16)


def make_weight(cfg: LayerConfig, layer: int = 0) -> torch.Tensor:
    return gaussian_bf16(cfg.N, cfg.K, cfg.w_std, seed_of(cfg, layer))


def make_activations(cfg: LayerConfig, rows: int, salt: int = 1, layer: int = 0) -> torch.Tensor:
    seed = seed_of(cfg, layer) + 100003 * salt
    if cfg.act == "gauss":
        return gaussian_bf16(rows, cfg.K, 1.0, seed)
    if cfg.act == "student_t_outlier":
        return student_t_outlier_bf16(rows, cfg.K, seed)
    raise ValueError(cfg.act)


def static_act_scale(A: torch.Tensor) -> float:
    """Stand-in for the running-maximum observer: the scale a calibration pass
    over this very tensor would have frozen, max|A| / (6*448) in fp32."""
    amax = A.abs().max().to(torch.float32)
    if float(amax) == 0.0:
        return 1.0
    return float((amax / torch.tensor(2688.0, dtype=torch.float32)).item())


def bf16_to_f32_numpy(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float32).contiguous().numpy()


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)
