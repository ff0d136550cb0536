"""Pins for the oracle's products (CPU only): exact integer arithmetic, one-hot
reductions, an independently written loop, and the library matmul."""
import numpy as np

import dq_inputs

E2M1 = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
E2M1_SIGNED = np.concatenate([E2M1, -E2M1])


def _unpack_nvfp4(codes):
    return np.stack([codes & 0xF, codes >> 4], axis=-1).reshape(codes.shape[0], -1)


def test_prefill_product_is_exact_integer_arithmetic(oracle):
    # 2*E2M1 values and 2^9*E4M3 values are integers, so with power-of-two tensor scales
    # sum_k (dA eA)(dW eW) is an exact integer the fp64 oracle must reproduce to the last bit.
    rng = np.random.default_rng(20)
    M, N, K = 8, 12, 128
    sa, sw = 2.0 ** -8, 2.0 ** -14
    A = (rng.normal(0, 1, (M, K))).astype(np.float32)
    W = (rng.normal(0, 0.02, (N, K))).astype(np.float32)
    ac, asc = oracle.quant_nvfp4(A, sa)
    wc, wsc = oracle.quant_nvfp4(W, sw)
    Y, S = oracle.matmul_nt(oracle.dequant_nvfp4(ac, asc, sa), oracle.dequant_nvfp4(wc, wsc, sw))
    tab512 = np.array([0 if (b & 0x7F) == 0x7F else int(round(oracle.e4m3_decode(b) * 512)) for b in range(256)],
                      dtype=np.int64)
    eA = (2 * E2M1_SIGNED[_unpack_nvfp4(ac)]).astype(np.int64)
    eW = (2 * E2M1_SIGNED[_unpack_nvfp4(wc)]).astype(np.int64)
    dA = np.repeat(tab512[asc], 16, axis=1)
    dW = np.repeat(tab512[wsc], 16, axis=1)
    Yi = (eA * dA) @ (eW * dW).T                       # int64, exact
    Si = np.abs(eA * dA) @ np.abs(eW * dW).T
    unit = sa * sw / (4.0 * 512 * 512)                 # power of two
    assert np.array_equal(Y, Yi.astype(np.float64) * unit)
    assert np.array_equal(S, Si.astype(np.float64) * unit)
    assert np.abs(Yi).max() < 2 ** 52


def test_decode_product_one_hot_reads_a_dequantised_column(oracle):
    rng = np.random.default_rng(21)
    N, K = 24, 128
    W = rng.normal(0, 0.02, (N, K)).astype(np.float32)
    s = oracle.global_scale(oracle.absmax(W))
    planes, sc = oracle.quant_lut3(W, s)
    What = oracle.dequant_lut3(planes, sc, s)
    for k in (0, 17, 127):
        x = np.zeros((1, K), dtype=np.float32)
        x[0, k] = 1.0
        Y, S = oracle.decode_linear(x, planes, sc, s, lib_matmul=False)
        assert np.array_equal(Y[0], What[:, k])
        assert np.array_equal(S[0], np.abs(What[:, k]))
    # value of one dequantised weight, assembled by hand: s * d * level
    G = oracle.codebook_values(oracle.lut3_default_codebook())
    idx = oracle.unpack_lut3_indices(planes)
    assert What[3, 40] == float(np.float32(s)) * oracle.e4m3_decode(int(sc[3, 40 // 16])) * G[idx[3, 40]]


def test_tiny_config_against_independent_loop_and_library_matmul(oracle):
    cfg = dq_inputs.CONFIGS["c1_tiny"]
    W = dq_inputs.bf16_to_f32_numpy(dq_inputs.make_weight(cfg))
    A_t = dq_inputs.make_activations(cfg, cfg.M)
    A = dq_inputs.bf16_to_f32_numpy(A_t)
    sa = dq_inputs.static_act_scale(A_t)
    p = oracle.pack_weights(W)
    Y, S = oracle.prefill_linear(A, sa, p["nvfp4_codes"], p["nvfp4_scales"], p["s"], lib_matmul=False)
    Yl, Sl = oracle.prefill_linear(A, sa, p["nvfp4_codes"], p["nvfp4_scales"], p["s"], lib_matmul=True)
    assert np.abs(Y - Yl).max() <= 1e-12 * S.max()
    assert np.abs(S - Sl).max() <= 1e-12 * S.max()
    # second, independently written evaluation: decode everything with numpy tables, sum per 16-block
    ac, asc = oracle.quant_nvfp4(A, sa)
    tab = np.array([oracle.e4m3_decode(b) for b in range(256)], dtype=np.float64)
    eA = E2M1_SIGNED[_unpack_nvfp4(ac)].reshape(cfg.M, -1, 16)
    eW = E2M1_SIGNED[_unpack_nvfp4(p["nvfp4_codes"])].reshape(cfg.N, -1, 16)
    blk = np.einsum("mbk,nbk->mnb", eA, eW)                        # per-block integer-valued dot products
    Y2 = np.einsum("mnb,mb,nb->mn", blk, tab[asc], tab[p["nvfp4_scales"]]) * float(np.float32(sa)) * float(np.float32(p["s"]))
    assert np.abs(Y - Y2).max() <= 1e-12 * S.max()
    # decode path on the same layer
    x_t = dq_inputs.make_activations(cfg, 1, salt=2)
    x = dq_inputs.bf16_to_f32_numpy(x_t)
    Yd, Sd = oracle.decode_linear(x, p["lut3_planes"], p["lut3_scales"], p["s"], lib_matmul=False)
    G = oracle.codebook_values(oracle.lut3_default_codebook())
    idx = oracle.unpack_lut3_indices(p["lut3_planes"])
    Wd = float(np.float32(p["s"])) * np.repeat(tab[p["lut3_scales"]], 16, axis=1) * G[idx]
    assert np.abs(Yd[0] - Wd @ x[0].astype(np.float64)).max() <= 1e-12 * Sd.max()
    # quantisation error of the whole layer is of the expected size (3.5-bit weights, exact activations)
    Yfull = W.astype(np.float64) @ x[0].astype(np.float64)
    rel = np.linalg.norm(Yd[0] - Yfull) / np.linalg.norm(Yfull)
    assert 0.05 < rel < 0.3


def test_nvfp4_decode_is_activations_times_dequantised_weights(oracle):
    """Weight-only decode on the NVFP4 view (Sec. 2.3): a one-hot activation picks one dequantised
    column, an all-ones activation gives row sums of s * d * e2m1 evaluated here from the printed value set,
    and the triple-loop and library products agree."""
    rng = np.random.default_rng(11)
    N, K = 48, 128
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    ref = oracle.pack_weights(W)
    codes, scales, s = ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"]
    e2m1 = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)          # App. A.3 "NVFP4"
    lo, hi = codes & 0xF, codes >> 4
    nib = np.stack([lo, hi], axis=-1).reshape(N, K)
    vals = np.where(nib & 8, -1.0, 1.0) * e2m1[nib & 7]
    sc = scales.astype(np.uint32)
    e, m = (sc >> 3) & 15, sc & 7
    d = np.where(e > 0, (1.0 + m / 8.0) * 2.0 ** (e.astype(np.float64) - 7), m / 8.0 * 2.0 ** -6)
    What = np.float64(np.float32(s)) * np.repeat(d, 16, axis=1) * vals
    X = np.zeros((3, K)); X[0, 5] = 1.0; X[1, 127] = -2.0; X[2, :] = 1.0
    Y, S = oracle.decode_linear_nvfp4(X, codes, scales, s, lib_matmul=False)
    assert np.array_equal(Y[0], What[:, 5]) and np.array_equal(Y[1], -2.0 * What[:, 127])
    assert np.allclose(Y[2], What.sum(axis=1), rtol=1e-13, atol=1e-15)
    assert np.allclose(S[2], np.abs(What).sum(axis=1), rtol=1e-13)
    Y2, _ = oracle.decode_linear_nvfp4(X, codes, scales, s, lib_matmul=True)
    assert np.allclose(Y, Y2, rtol=1e-13, atol=1e-15)
