"""Pins for the oracle's number formats (CPU only).

Each check compares the oracle with something other than itself: values the
paper prints (tests/golden), an independent library conversion (torch's
float8 / float16 / bfloat16 casts), or a brute-force nearest-value search.
"""
from pathlib import Path

import numpy as np
import pytest
import torch

GOLD = Path(__file__).resolve().parent / "golden"


def _golden_e2m1():
    return [float(l) for l in (GOLD / "e2m1_values.txt").read_text().splitlines() if l and not l.startswith("#")]


def _golden_grids():
    out = {}
    for l in (GOLD / "lut_grids.txt").read_text().splitlines():
        if l and not l.startswith("#"):
            name, vals = l.split(":")
            out[name.strip()] = [float(v) for v in vals.split()]
    return out


def test_e2m1_value_set_is_the_papers(oracle):
    mags = _golden_e2m1()
    assert mags == [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    for code in range(16):
        v = oracle.e2m1_decode(code)
        assert abs(v) == mags[code & 7]
        assert (np.signbit(v)) == bool(code & 8)
    assert tuple(mags) == oracle.E2M1_MAGNITUDES


def test_e2m1_round_trip_of_representable_values(oracle):
    for code in range(16):
        assert oracle.e2m1_encode(oracle.e2m1_decode(code)) == code


def test_e2m1_encode_is_nearest_with_even_ties(oracle):
    mags = np.array(_golden_e2m1())
    rng = np.random.default_rng(1)
    ys = np.concatenate([rng.uniform(-7, 7, 20000), rng.normal(0, 2, 20000),
                         [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0,
                          6.0, 6.5, 100.0, -100.0, 1e-30, -1e-30]]).astype(np.float32)
    for y in ys:
        code = oracle.e2m1_encode(float(y))
        a = abs(float(y))
        dist = np.abs(mags - a)
        best = np.flatnonzero(dist == dist.min())
        if len(best) == 2:                       # tie: the code with an even mantissa bit
            want = [b for b in best if b % 2 == 0][0]
        else:
            want = best[0]
        assert (code & 7) == want, (y, code)
        assert bool(code & 8) == bool(np.signbit(y))
    # the documented tie table
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for y, v in ties.items():
        assert oracle.e2m1_decode(oracle.e2m1_encode(y)) == v
    assert oracle.e2m1_encode(float("nan")) == 0x7
    assert oracle.e2m1_encode(-0.0) == 0x8


def test_e4m3_decode_matches_torch_float8(oracle):
    allb = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    ref = allb.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    for b in range(256):
        v = oracle.e4m3_decode(b)
        if np.isnan(ref[b]):
            assert np.isnan(v)
        else:
            assert v == ref[b] and np.signbit(v) == np.signbit(ref[b])
    assert oracle.e4m3_decode(0x7E) == 448.0          # the 448 in s = max|W|/(6*448)


def test_e4m3_round_trip_all_finite_bytes(oracle):
    for b in range(256):
        if (b & 0x7F) == 0x7F:
            continue
        assert oracle.e4m3_encode(oracle.e4m3_decode(b)) == b


def test_e4m3_encode_matches_torch_in_range_and_saturates(oracle):
    rng = np.random.default_rng(2)
    t = np.concatenate([rng.uniform(-448, 448, 50000), rng.normal(0, 1, 50000), rng.normal(0, 0.01, 50000),
                        rng.uniform(-2 ** -6, 2 ** -6, 50000)]).astype(np.float32)
    ref = torch.from_numpy(t).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    enc = np.array([oracle.e4m3_encode(float(v)) for v in t], dtype=np.uint8)
    assert np.array_equal(enc, ref)
    # saturation instead of NaN above the largest finite value
    for v in (448.0, 449.0, 463.9, 464.0, 480.0, 1e9, float("inf")):
        assert oracle.e4m3_encode(v) == 0x7E
        assert oracle.e4m3_encode(-v) == 0xFE
    # smallest subnormal is 2^-9; half of it ties to zero (even)
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00
    assert oracle.e4m3_encode(np.nextafter(np.float32(2.0 ** -10), np.float32(1))) == 0x01
    assert oracle.e4m3_encode(1.5 * 2.0 ** -9) == 0x02     # tie to even


def test_e4m3_encode_brute_force_nearest(oracle):
    vals = np.array([oracle.e4m3_decode(b) for b in range(0x7F)], dtype=np.float64)   # positive finite
    rng = np.random.default_rng(3)
    ts = np.exp(rng.uniform(np.log(2.0 ** -11), np.log(448.0), 20000)).astype(np.float32)
    for t in ts:
        b = oracle.e4m3_encode(float(t))
        d = np.abs(vals - float(t))
        best = np.flatnonzero(d == d.min())
        want = best[0] if len(best) == 1 else [x for x in best if x % 2 == 0][0]
        assert b == want, (t, b, want)
    # monotone
    grid = np.linspace(0, 460, 5000, dtype=np.float32)
    codes = [oracle.e4m3_encode(float(g)) for g in grid]
    assert all(c1 <= c2 for c1, c2 in zip(codes, codes[1:]))


def test_f16_and_bf16_codecs_match_torch(oracle):
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.normal(0, 1, 20000), rng.normal(0, 1e-3, 5000), rng.uniform(-7e4, 7e4, 5000),
                        rng.normal(0, 1e-6, 5000)]).astype(np.float32)
    h_ref = torch.from_numpy(x).to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    b_ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for i in range(0, len(x), 7):
        assert oracle.f16_encode(float(x[i])) == h_ref[i]
        assert oracle.bf16_encode(float(x[i])) == b_ref[i]
    hs = rng.integers(0, 1 << 16, 4000).astype(np.uint16)
    hv = torch.from_numpy(hs.view(np.int16)).view(torch.float16).to(torch.float32).numpy()
    bv = torch.from_numpy(hs.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    for i, h in enumerate(hs):
        a, b = oracle.f16_decode(int(h)), oracle.bf16_decode(int(h))
        assert (np.isnan(a) and np.isnan(hv[i])) or a == hv[i]
        assert (np.isnan(b) and np.isnan(bv[i])) or b == bv[i]


def test_lut3_codebook_is_paper_grid_rounded_to_fp16(oracle):
    grid = _golden_grids()["LUT3A16"]
    cb = oracle.lut3_default_codebook()
    ref = torch.tensor(grid, dtype=torch.float32).to(torch.float16)
    assert np.array_equal(cb, ref.view(torch.int16).numpy().view(np.uint16))
    vals = oracle.codebook_values(cb)
    assert np.all(np.diff(vals) > 0)
    assert vals[3] == 0.0 and vals[7] == 6.0
    assert np.max(np.abs(vals - np.array(grid))) < 2e-3      # fp16 rounding of 4-decimal values
    # the values the format section of the design notes lists
    assert list(vals) == [-4.703125, -2.869140625, -1.369140625, 0.0, 1.220703125, 2.529296875, 4.046875, 6.0]
