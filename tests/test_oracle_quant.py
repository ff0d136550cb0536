"""Pins for the oracle's quantisers, packers, autocast and dequantisers (CPU only).

The oracle is compared with invariants that follow from the paper's two-level
scaling, with an independently written fp64 brute-force RTN, with tensors that
are exactly representable, and with the optimality statement for the LUT grid.
"""
from pathlib import Path

import numpy as np
import pytest

import dq_inputs

GOLD = Path(__file__).resolve().parent / "golden"
E2M1 = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
E2M1_SIGNED = np.concatenate([E2M1, -E2M1])            # index = code


def _consts():
    out = {}
    for l in (GOLD / "format_constants.txt").read_text().splitlines():
        l = l.split("#")[0].strip()
        if l:
            k, v = l.split()
            out[k] = float(v)
    return out


def _e4m3_table(oracle):
    return np.array([oracle.e4m3_decode(b) for b in range(256)], dtype=np.float64)


def _unpack_nvfp4(codes):
    lo = codes & 0xF
    hi = codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


def _weights(N=96, K=256, seed=5, std=0.02):
    return dq_inputs.bf16_to_f32_numpy(dq_inputs.gaussian_bf16(N, K, std, seed))


# --------------------------------------------------------------- global scale

def test_global_scale_formula(oracle):
    c = _consts()
    W = _weights()
    amax = float(np.abs(W).max())
    assert oracle.absmax(W) == amax
    s = oracle.global_scale(amax)
    assert s == np.float32(amax) / np.float32(c["global_scale_divisor"])
    assert c["global_scale_divisor"] == 6 * c["e4m3_max"]
    assert oracle.global_scale(0.0) == 1.0


# --------------------------------------------------------------------- NVFP4

def test_nvfp4_block_scale_and_absmax_invariants(oracle):
    W = _weights(128, 512)
    s = oracle.global_scale(oracle.absmax(W))
    codes, scales = oracle.quant_nvfp4(W, s)
    tab = _e4m3_table(oracle)
    d = tab[scales]
    assert scales.max() <= 0x7E and d.max() <= 448.0
    assert np.all(scales < 0x80)                                 # unsigned for NVFP4
    # the block that holds the tensor maximum gets the largest E4M3 value
    r, k = np.unravel_index(np.argmax(np.abs(W)), W.shape)
    assert scales[r, k // 16] == 0x7E
    # E4M3's relative rounding error is at most 2^-4, so every block extreme lands
    # in [6/1.0625, 6/0.9375] after normalisation and is coded as magnitude 6
    a_b = np.abs(W).reshape(128, -1, 16).max(axis=2).astype(np.float64)
    normal = scales >= 0x08
    ratio = a_b[normal] / (float(s) * d[normal])
    assert ratio.min() >= 6 / 1.0625 - 1e-6 and ratio.max() <= 6 / 0.9375 + 1e-6
    mags = (_unpack_nvfp4(codes) & 7).reshape(128, -1, 16)
    assert np.all(mags.max(axis=2)[normal] == 7)


def test_nvfp4_is_rtn_against_fp64_brute_force(oracle):
    W = _weights(256, 512, seed=6)
    s = oracle.global_scale(oracle.absmax(W))
    codes, scales = oracle.quant_nvfp4(W, s)
    tab = _e4m3_table(oracle)
    d = np.repeat(tab[scales], 16, axis=1)
    y = W.astype(np.float64) / (float(s) * d)
    # nearest signed E2M1 value; saturate beyond 6
    dist = np.abs(np.abs(y)[..., None] - E2M1[None, None, :])
    ideal_mag = dist.argmin(axis=2)
    got = _unpack_nvfp4(codes)
    mism = (got & 7) != ideal_mag
    # the fp32 reciprocal-multiply recipe may differ from exact division only at a rounding
    # threshold (bf16 inputs sit on such thresholds often: x = 1.75/6 of the block extreme etc.)
    assert mism.mean() < 2e-3
    thresholds = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    near = np.abs(np.abs(y)[mism][:, None] - thresholds[None, :]).min(axis=1)
    assert np.all(near < 1e-5)
    nz = (got & 7) != 0
    assert np.array_equal((got >> 3)[nz] == 1, (W < 0)[nz])
    # elementwise error bound: half the local level gap, plus saturation slack above 6
    xhat = oracle.dequant_nvfp4(codes, scales, s)
    err = np.abs(xhat - W) / (float(s) * d)
    assert err.max() <= 1.0 + 0.41


def test_nvfp4_exact_round_trip_of_representable_tensor(oracle):
    rng = np.random.default_rng(7)
    N, K = 32, 256
    s = 2.0 ** -12
    sc = rng.integers(0x20, 0x7F, size=(N, K // 16)).astype(np.uint8)
    sc[0, 0] = 0x7E                                            # a block with d = 448 ...
    code = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    code[code == 8] = 0                                        # no negative zero
    code.reshape(N, -1, 16)[:, :, 0] = 7                      # ... every block holds its extreme +-6
    code[1::2].reshape(-1, K // 16, 16)[:, :, 0] = 15
    tab = _e4m3_table(oracle)
    W = (s * np.repeat(tab[sc], 16, axis=1) * E2M1_SIGNED[code]).astype(np.float32)
    assert oracle.global_scale(oracle.absmax(W)) == s
    codes, scales = oracle.quant_nvfp4(W, s)
    assert np.array_equal(scales, sc)
    assert np.array_equal(_unpack_nvfp4(codes), code)
    assert np.array_equal(oracle.dequant_nvfp4(codes, scales, s), W.astype(np.float64))


def test_nvfp4_nibble_order_and_zero_blocks(oracle):
    s = 2.0 ** -10
    W = np.zeros((2, 32), dtype=np.float32)
    W[0, :16] = s * 448 * np.array([6, -0.5, 1, -1.5, 2, 3, -4, 0, 0, 0, 0, 0, 0, 0, 0, 0.5])
    codes, scales = oracle.quant_nvfp4(W, s)
    assert scales[0, 0] == 0x7E and scales[0, 1] == 0 and np.all(scales[1] == 0)
    assert codes[0, 0] == (0x7 | (0x9 << 4))       # element 0 low nibble, element 1 high nibble
    assert codes[0, 1] == (0x2 | (0xB << 4))
    assert np.all(codes[0, 8:] == 0) and np.all(codes[1] == 0)
    # block scale underflow: extreme far below s*2^-10 gives a zero scale and zero codes
    W2 = np.full((1, 16), 1e-9, dtype=np.float32)
    c2, s2 = oracle.quant_nvfp4(W2, 1.0)
    assert np.all(s2 == 0) and np.all(c2 == 0)


def test_storage_cost_matches_paper(oracle):
    c = _consts()
    N, K = 64, 512
    W = _weights(N, K)
    p = oracle.pack_weights(W)
    nv_bits = 8 * (p["nvfp4_codes"].nbytes + p["nvfp4_scales"].nbytes) / (N * K)
    lut_bits = 8 * (p["lut3_planes"].nbytes + p["lut3_scales"].nbytes) / (N * K)
    assert nv_bits == c["bits_per_weight_nvfp4"]
    assert lut_bits == c["bits_per_weight_lut3"]
    assert p["lut3_planes"].shape == (N, 3, K // int(c["plane_word_bits"]))
    assert p["lut3_planes"].dtype == np.uint32


# ---------------------------------------------------------------------- LUT3

def test_lut3_block_extreme_is_plus_six(oracle):
    W = _weights(128, 512, seed=8)
    s = oracle.global_scale(oracle.absmax(W))
    planes, scales = oracle.quant_lut3(W, s)
    idx = oracle.unpack_lut3_indices(planes)
    tab = _e4m3_table(oracle)
    blk = W.reshape(128, -1, 16)
    # position of the maximum-magnitude element; when +max and -max both occur (bf16 data
    # makes that common) the positive one is the extreme
    amax_b = np.abs(blk).max(axis=2, keepdims=True)
    pos = np.where((blk == amax_b).any(axis=2), (blk == amax_b).argmax(axis=2), (blk == -amax_b).argmax(axis=2))
    m = np.take_along_axis(blk, pos[..., None], axis=2)[..., 0]
    assert np.array_equal(np.abs(m), amax_b[..., 0])
    assert ((blk == amax_b).any(axis=2) & (blk == -amax_b).any(axis=2)).sum() > 0     # the tie case is exercised
    normal = (scales & 0x7F) >= 0x08
    # the scale carries the sign of the maximum-magnitude element ...
    assert np.array_equal((scales >= 0x80)[normal], (m < 0)[normal])
    # ... so that element is always the +6 level (index 7)
    top = np.take_along_axis(idx.reshape(128, -1, 16), pos[..., None], axis=2)[..., 0]
    assert np.all(top[normal] == 7)
    # about half of the block scales are negative on symmetric data
    assert 0.45 < (scales >= 0x80).mean() < 0.55
    # the block holding the tensor maximum has |d| = 448
    r, k = np.unravel_index(np.argmax(np.abs(W)), W.shape)
    assert (scales[r, k // 16] & 0x7F) == 0x7E
    assert np.abs(tab[scales]).max() <= 448


def test_lut3_is_nearest_level_against_fp64_brute_force(oracle):
    W = _weights(256, 512, seed=9)
    s = oracle.global_scale(oracle.absmax(W))
    planes, scales = oracle.quant_lut3(W, s)
    idx = oracle.unpack_lut3_indices(planes)
    G = oracle.codebook_values(oracle.lut3_default_codebook())
    tab = _e4m3_table(oracle)
    d = np.repeat(tab[scales], 16, axis=1)
    y = W.astype(np.float64) / (float(s) * d)
    ideal = np.abs(y[..., None] - G[None, None, :]).argmin(axis=2)
    mism = idx != ideal
    assert mism.mean() < 1e-4
    T = (G[1:] + G[:-1]) / 2
    near = np.abs(y[mism][:, None] - T[None, :]).min(axis=1)
    assert np.all(near < 1e-5)
    xhat = oracle.dequant_lut3(planes, scales, s)
    # inside the grid the error is at most half the widest gap; outside it the normalised value
    # lies in [-6.4, 6.4] (E4M3 rounding of the block scale), so the worst case is the distance
    # from -6.4 to the lowest level
    gap = np.diff(G).max() / 2
    assert (np.abs(xhat - W) / np.abs(float(s) * d)).max() <= max(gap, 6.4 + G[0]) + 1e-6


def test_lut3_grid_is_lloyd_stationary_on_gaussian_data(oracle):
    # App. A.3: the grid minimises the expected squared error over N(0,1) samples under the
    # two-level scaling with 0 and +6 fixed; at such a minimum every free level equals
    # the mean of the normalised values assigned to it.
    rng = np.random.default_rng(10)
    X = rng.normal(0, 1, size=(4096, 1024)).astype(np.float32)
    s = oracle.global_scale(oracle.absmax(X))
    planes, scales = oracle.quant_lut3(X, s)
    idx = oracle.unpack_lut3_indices(planes)
    tab = _e4m3_table(oracle)
    d = np.repeat(tab[scales], 16, axis=1)
    y = X.astype(np.float64) / (float(s) * d)
    grids = {}
    for l in (GOLD / "lut_grids.txt").read_text().splitlines():
        if l and not l.startswith("#"):
            grids[l.split(":")[0]] = [float(v) for v in l.split(":")[1].split()]
    paper = grids["LUT3A16"]
    for j in (0, 1, 2, 4, 5, 6):                       # 0 and +6 are constrained, not free
        cell_mean = y[idx == j].mean()
        assert abs(cell_mean - paper[j]) < 0.02, (j, cell_mean, paper[j])
    # level usage and error level of this scheme on Gaussian data (independent numpy estimate: design notes)
    freq = np.bincount(idx.ravel(), minlength=8) / idx.size
    ref_freq = np.array([.077, .130, .170, .175, .154, .124, .084, .087])
    assert np.abs(freq - ref_freq).max() < 0.01
    xhat = oracle.dequant_lut3(planes, scales, s)
    rel_mse = ((xhat - X) ** 2).sum() / (X.astype(np.float64) ** 2).sum()
    assert abs(rel_mse - 2.23e-2) / 2.23e-2 < 0.05
    c4, s4 = oracle.quant_nvfp4(X, s)
    rel_mse4 = ((oracle.dequant_nvfp4(c4, s4, s) - X) ** 2).sum() / (X.astype(np.float64) ** 2).sum()
    assert abs(rel_mse4 - 9.04e-3) / 9.04e-3 < 0.05
    assert rel_mse4 < rel_mse                           # 4.5 bit beats 3.5 bit


def test_lut3_exact_round_trip_and_bit_planes(oracle):
    rng = np.random.default_rng(11)
    N, K = 16, 256
    s = 2.0 ** -11
    G = oracle.codebook_values(oracle.lut3_default_codebook())
    tab = _e4m3_table(oracle)
    sc = rng.integers(0x20, 0x7F, size=(N, K // 16)).astype(np.uint8)
    sc[rng.random(sc.shape) < 0.5] |= 0x80
    sc[0, 0] = 0x7E
    idx = np.tile(np.arange(K) % 8, (N, 1)).astype(np.uint8)     # every block of 16 holds level 7 twice
    W = (s * np.repeat(tab[sc], 16, axis=1) * G[idx]).astype(np.float32)
    assert np.array_equal(W.astype(np.float64), s * np.repeat(tab[sc], 16, axis=1) * G[idx])   # exact in fp32
    planes, scales = oracle.quant_lut3(W, s)
    assert np.array_equal(scales, sc)
    assert np.array_equal(oracle.unpack_lut3_indices(planes), idx)
    # idx = k mod 8 gives constant plane words (LSB-first bit order, plane p = bit p)
    assert np.all(planes[:, 0, :] == 0xAAAAAAAA)
    assert np.all(planes[:, 1, :] == 0xCCCCCCCC)
    assert np.all(planes[:, 2, :] == 0xF0F0F0F0)
    assert np.array_equal(oracle.dequant_lut3(planes, scales, s), W.astype(np.float64))
    # random indices survive pack / unpack
    idx2 = rng.integers(0, 8, size=(N, K)).astype(np.uint8)
    idx2.reshape(N, -1, 16)[:, :, 5] = 7
    W2 = (s * np.repeat(tab[sc], 16, axis=1) * G[idx2]).astype(np.float32)
    p2, s2 = oracle.quant_lut3(W2, s)
    assert np.array_equal(oracle.unpack_lut3_indices(p2), idx2) and np.array_equal(s2, sc)


def test_lut3_sign_tie_zero_block_and_custom_codebook(oracle):
    s = 2.0 ** -10
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, 0], W[0, 3] = -0.5, 0.5                  # equal magnitudes, both signs: positive wins
    W[0, 16], W[0, 19] = -0.25, -0.25             # only negatives: negative scale
    W[0, 32:48] = 0.0                             # all-zero block
    planes, scales = oracle.quant_lut3(W, s)
    idx = oracle.unpack_lut3_indices(planes)
    assert scales[0, 0] < 0x80 and idx[0, 3] == 7 and idx[0, 0] == 0
    assert scales[0, 1] >= 0x80 and idx[0, 16] == 7 and idx[0, 19] == 7
    assert scales[0, 2] == 0 and np.all(idx[0, 32:48] == 3)      # index of the 0.0 level
    assert np.all(oracle.dequant_lut3(planes, scales, s)[0, 32:48] == 0)
    # halfway between two levels goes to the lower one
    G = oracle.codebook_values(oracle.lut3_default_codebook())
    d = 1.0                                        # E4M3 0x38
    mid = (G[4] + G[5]) / 2
    W3 = np.zeros((1, 32), dtype=np.float32)
    W3[0, 0] = 6.0 * s * d
    W3[0, 1] = np.float32(mid * s * d)
    p3, s3 = oracle.quant_lut3(W3, s)
    assert s3[0, 0] == 0x38 and oracle.unpack_lut3_indices(p3)[0, 1] == 4
    # a different codebook is honoured
    cb = np.array([oracle.f16_encode(v) for v in (-5, -3, -1, 0, 1, 2, 4, 6)], dtype=np.uint16)
    W4 = np.zeros((1, 32), dtype=np.float32)
    W4[0, :8] = s * np.array([6, -5, -3, -1, 0, 1, 2, 4])
    p4, s4 = oracle.quant_lut3(W4, s, cb)
    assert list(oracle.unpack_lut3_indices(p4)[0, :8]) == [7, 0, 1, 2, 3, 4, 5, 6]


# ------------------------------------------------------------------ autocast

def test_autocast_level_map_and_equivalence_with_rtn(oracle):
    grids = {}
    for l in (GOLD / "lut_grids.txt").read_text().splitlines():
        if l and not l.startswith("#"):
            grids[l.split(":")[0]] = [float(v) for v in l.split(":")[1].split()]
    # nearest E2M1 value of each printed LUT3 level (App. A.3 grids)
    want = [-4.0, -3.0, -1.5, 0.0, 1.0, 3.0, 4.0, 6.0]
    for lvl, w in zip(grids["LUT3A16"], want):
        assert E2M1_SIGNED[np.abs(E2M1_SIGNED - lvl).argmin()] == w
    W = _weights(64, 512, seed=12)
    s = oracle.global_scale(oracle.absmax(W))
    planes, lsc = oracle.quant_lut3(W, s)
    codes, sc = oracle.autocast_lut3_to_nvfp4(planes, lsc)
    idx = oracle.unpack_lut3_indices(planes)
    got = E2M1_SIGNED[_unpack_nvfp4(codes)]
    sign = np.where(np.repeat(lsc, 16, axis=1) >= 0x80, -1.0, 1.0)
    assert np.array_equal(got, np.array(want)[idx] * sign + 0.0)
    assert np.array_equal(sc, lsc & 0x7F)
    # same as RTN-NVFP4 of the dequantised LUT3 tensor with the tensor scale held at s
    What = oracle.dequant_lut3(planes, lsc, s).astype(np.float32)
    c2, s2 = oracle.quant_nvfp4(What, s)
    normal = (lsc & 0x7F) >= 0x08
    assert np.array_equal(s2[normal], sc[normal])
    m = np.repeat(normal, 16, axis=1)
    # by value: a zero level under a negative block scale dequantises to -0.0, whose RTN code
    # keeps the sign bit, while the autocast writes the canonical +0
    assert np.array_equal(E2M1_SIGNED[_unpack_nvfp4(c2)][m], E2M1_SIGNED[_unpack_nvfp4(codes)][m])
    assert not np.any(_unpack_nvfp4(codes) == 8)
