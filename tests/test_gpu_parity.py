"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Codes and scales bit for bit; GEMM / GEMV outputs
within relative Frobenius error 2e-3 and, per element, one bf16 ulp plus
1e-4 * sum_k |a*w| (see parity_utils)."""
import numpy as np
import pytest
import torch

import dq_inputs
from parity_utils import check_outputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dq():
    import __graft_entry__ as g
    g.build()
    import paper_2609_26333_b200 as dq
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    assert torch.cuda.get_device_capability(0) == (10, 0), "this library targets sm_100a only"
    return dq


DEV = "cuda:0"


def _np(t):
    return t.detach().cpu().numpy()


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _status_ok(dq):
    torch.cuda.synchronize()
    st, det = dq.get_status()
    assert st == 0, f"device status {dq.status_string(st)} detail {det}"


_ref_cache = {}


def _layer(oracle, N, K, seed, std=0.02, dtype=torch.bfloat16):
    key = (N, K, seed, std, dtype)
    if key not in _ref_cache:
        if dtype == torch.bfloat16:
            W = dq_inputs.gaussian_bf16(N, K, std, seed)
            Wf = dq_inputs.bf16_to_f32_numpy(W)
        else:
            g = torch.Generator().manual_seed(seed)
            W = torch.randn(N, K, generator=g, dtype=torch.float32) * std
            Wf = W.numpy()
        _ref_cache[key] = (W, oracle.pack_weights(Wf))
    return _ref_cache[key]


# shapes: tiny config; ragged multi-tile (N not a multiple of the tile, K with a 128 tail); several tiles
PACK_SHAPES = [(512, 256, 0), (144, 384, 31), (784, 1152, 32)]


@pytest.mark.parametrize("N,K,seed", PACK_SHAPES)
def test_pack_bit_exact(dq, oracle, N, K, seed):
    W, ref = _layer(oracle, N, K, seed)
    w = dq.pack_weights(W.to(DEV))
    codes, scales, s = dq.export_canonical(w, dq.FMT_NVFP4)
    planes, lsc, s2 = dq.export_canonical(w, dq.FMT_LUT3)
    _status_ok(dq)
    assert np.float32(_np(s)[0]) == np.float32(ref["s"]) and _np(s2)[0] == _np(s)[0]
    assert np.array_equal(_np(scales), ref["nvfp4_scales"])
    assert np.array_equal(_np(codes), ref["nvfp4_codes"])
    assert np.array_equal(_np(lsc), ref["lut3_scales"])
    assert np.array_equal(_np(planes).view(np.uint32), ref["lut3_planes"])


def test_pack_fp32_master_and_strided_rows(dq, oracle):
    N, K = 160, 256
    W, ref = _layer(oracle, N, K, 33, dtype=torch.float32)
    big = torch.zeros(N, K + 64, dtype=torch.float32, device=DEV)
    big[:, :K] = W.to(DEV)
    w = dq.pack_weights(big[:, :K])
    codes, scales, s = dq.export_canonical(w, dq.FMT_NVFP4)
    planes, lsc, _ = dq.export_canonical(w, dq.FMT_LUT3)
    _status_ok(dq)
    assert np.array_equal(_np(codes), ref["nvfp4_codes"]) and np.array_equal(_np(scales), ref["nvfp4_scales"])
    assert np.array_equal(_np(planes).view(np.uint32), ref["lut3_planes"]) and np.array_equal(_np(lsc), ref["lut3_scales"])


def test_pack_degenerate_tensors(dq, oracle):
    N, K = 32, 128
    # all zero: s = 1, zero scales, zero codes, LUT index of the 0.0 level
    Z = torch.zeros(N, K, dtype=torch.bfloat16)
    ref = oracle.pack_weights(dq_inputs.bf16_to_f32_numpy(Z))
    w = dq.pack_weights(Z.to(DEV))
    codes, scales, s = dq.export_canonical(w, dq.FMT_NVFP4)
    planes, lsc, _ = dq.export_canonical(w, dq.FMT_LUT3)
    assert _np(s)[0] == 1.0 and not _np(codes).any() and not _np(scales).any() and not _np(lsc).any()
    assert np.array_equal(_np(planes).view(np.uint32), ref["lut3_planes"])
    # sign ties, zero blocks, a single huge outlier (block-scale underflow elsewhere)
    X = dq_inputs.gaussian_bf16(N, K, 0.02, 34)
    X[0, :16] = 0
    X[1, 0], X[1, 5] = 0.5, -0.5
    X[2, 3], X[2, 9] = -0.75, 0.75
    X[3, 7] = 3.0e4
    ref = oracle.pack_weights(dq_inputs.bf16_to_f32_numpy(X))
    w = dq.pack_weights(X.to(DEV))
    codes, scales, s = dq.export_canonical(w, dq.FMT_NVFP4)
    planes, lsc, _ = dq.export_canonical(w, dq.FMT_LUT3)
    _status_ok(dq)
    assert np.float32(_np(s)[0]) == np.float32(ref["s"])
    assert np.array_equal(_np(codes), ref["nvfp4_codes"]) and np.array_equal(_np(scales), ref["nvfp4_scales"])
    assert np.array_equal(_np(planes).view(np.uint32), ref["lut3_planes"]) and np.array_equal(_np(lsc), ref["lut3_scales"])


def test_autocast_view_bit_exact(dq, oracle):
    N, K = 272, 512
    W, ref = _layer(oracle, N, K, 35)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4_FROM_LUT3)
    codes, scales, s = dq.export_canonical(w, dq.FMT_NVFP4_FROM_LUT3)
    planes, lsc, _ = dq.export_canonical(w, dq.FMT_LUT3)
    _status_ok(dq)
    ac, asc = oracle.autocast_lut3_to_nvfp4(ref["lut3_planes"], ref["lut3_scales"])
    assert np.array_equal(_np(planes).view(np.uint32), ref["lut3_planes"])
    assert np.array_equal(_np(codes), ac) and np.array_equal(_np(scales), asc)


def test_import_canonical_round_trip_and_use(dq, oracle):
    """Oracle-made codes go in through dq_import_canonical, come back unchanged through the export,
    and drive both kernels to the same results as a handle packed from the master weights."""
    M, N, K = 160, 272, 640
    W, ref = _layer(oracle, N, K, 36)
    nv = (torch.from_numpy(ref["nvfp4_codes"]).to(DEV), torch.from_numpy(ref["nvfp4_scales"]).to(DEV))
    lut = (torch.from_numpy(ref["lut3_planes"].view(np.int32)).to(DEV), torch.from_numpy(ref["lut3_scales"]).to(DEV))
    w_imp = dq.import_canonical(N, K, dq.FMT_NVFP4 | dq.FMT_LUT3, float(ref["s"]), nvfp4=nv, lut3=lut)
    w_pack = dq.pack_weights(W.to(DEV))
    for fmt, want in ((dq.FMT_NVFP4, (ref["nvfp4_codes"], ref["nvfp4_scales"])),
                      (dq.FMT_LUT3, (ref["lut3_planes"], ref["lut3_scales"]))):
        codes, scales, s = dq.export_canonical(w_imp, fmt)
        assert np.array_equal(_np(codes).view(want[0].dtype), want[0]) and np.array_equal(_np(scales), want[1])
        assert np.float32(_np(s)[0]) == np.float32(ref["s"])
    A = dq_inputs.gaussian_bf16(M, K, 1.0, 37).to(DEV)
    sa = dq_inputs.static_act_scale(A.cpu())
    assert torch.equal(dq.prefill_linear(w_imp, A, sa), dq.prefill_linear(w_pack, A, sa))
    assert torch.equal(dq.decode_linear(w_imp, A[:3]), dq.decode_linear(w_pack, A[:3]))
    # the LUT3-derived view from imported planes equals the oracle's autocast
    w_view = dq.import_canonical(N, K, dq.FMT_NVFP4_FROM_LUT3, float(ref["s"]), lut3=lut)
    codes, scales, _ = dq.export_canonical(w_view, dq.FMT_NVFP4_FROM_LUT3)
    ac, asc = oracle.autocast_lut3_to_nvfp4(ref["lut3_planes"], ref["lut3_scales"])
    assert np.array_equal(_np(codes), ac) and np.array_equal(_np(scales), asc)
    with pytest.raises(dq.DQError):
        dq.import_canonical(N, K, dq.FMT_NVFP4, float(ref["s"]), lut3=lut)      # missing NVFP4 buffers
    _status_ok(dq)


def test_custom_codebook(dq, oracle):
    N, K = 64, 256
    W, _ = _layer(oracle, N, K, 36)
    cb = np.array([oracle.f16_encode(v) for v in (-5, -3, -1.5, 0, 1, 2.25, 4, 6)], dtype=np.uint16)
    Wf = dq_inputs.bf16_to_f32_numpy(W)
    ref = oracle.pack_weights(Wf, cb)
    w = dq.pack_weights(W.to(DEV), codebook_f16=cb)
    planes, lsc, _ = dq.export_canonical(w, dq.FMT_LUT3)
    assert np.array_equal(_np(planes).view(np.uint32), ref["lut3_planes"]) and np.array_equal(_np(lsc), ref["lut3_scales"])
    X = dq_inputs.gaussian_bf16(2, K, 1.0, 37)
    Y = dq.decode_linear(w, X.to(DEV))
    _status_ok(dq)
    Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(X), ref["lut3_planes"], ref["lut3_scales"], ref["s"], cb)
    check_outputs(_f64(Y), Yr, S, "custom codebook decode")


@pytest.mark.parametrize("M,K,kind", [(64, 256, "gauss"), (300, 640, "gauss"), (257, 1024, "student")])
def test_activation_quantiser_bit_exact(dq, oracle, M, K, kind):
    if kind == "gauss":
        A = dq_inputs.gaussian_bf16(M, K, 1.0, 40 + M)
    else:
        A = dq_inputs.student_t_outlier_bf16(M, K, 41)
    sa = dq_inputs.static_act_scale(A)
    codes, scales = dq.quantize_activations(A.to(DEV), sa)
    _status_ok(dq)
    rc, rs = oracle.quant_nvfp4(dq_inputs.bf16_to_f32_numpy(A), sa)
    assert np.array_equal(_np(scales), rs)
    assert np.array_equal(_np(codes), rc)
    # a static scale that is too small saturates instead of misbehaving
    codes2, scales2 = dq.quantize_activations(A.to(DEV), sa / 64)
    rc2, rs2 = oracle.quant_nvfp4(dq_inputs.bf16_to_f32_numpy(A), sa / 64)
    assert np.array_equal(_np(scales2), rs2) and np.array_equal(_np(codes2), rc2)
    assert (rs2 == 0x7E).any()


PREFILL_SHAPES = [
    # M, N, K, seed : tiny config (M below one tile); ragged tiles with a K tail; several tiles per CTA
    (64, 512, 256, 0),
    (300, 784, 640, 51),
    (1, 256, 128, 52),
    (129, 272, 1152, 53),
    (640, 1536, 2048, 54),
]


@pytest.mark.parametrize("M,N,K,seed", PREFILL_SHAPES)
def test_prefill_parity(dq, oracle, M, N, K, seed):
    W, ref = _layer(oracle, N, K, seed)
    A = dq_inputs.gaussian_bf16(M, K, 1.0, seed + 7)
    sa = dq_inputs.static_act_scale(A)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4)
    Y = dq.prefill_linear(w, A.to(DEV), sa)
    _status_ok(dq)
    Yr, S = oracle.prefill_linear(dq_inputs.bf16_to_f32_numpy(A), sa, ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"])
    check_outputs(_f64(Y), Yr, S, f"prefill {M}x{N}x{K}")
    # repeated call on the same handle and workspace gives the same bits
    Y2 = dq.prefill_linear(w, A.to(DEV), sa)
    assert torch.equal(Y, Y2)


def test_prefill_strided_output_and_autocast_weights(dq, oracle):
    M, N, K = 200, 528, 384
    W, ref = _layer(oracle, N, K, 55)
    A = dq_inputs.gaussian_bf16(M, K, 1.0, 56)
    sa = dq_inputs.static_act_scale(A)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4_FROM_LUT3)
    out = torch.full((M, N + 16), 7.0, dtype=torch.bfloat16, device=DEV)
    dq.prefill_linear(w, A.to(DEV), sa, out=out[:, :N])
    _status_ok(dq)
    assert torch.all(out[:, N:] == 7.0)
    ac, asc = oracle.autocast_lut3_to_nvfp4(ref["lut3_planes"], ref["lut3_scales"])
    Yr, S = oracle.prefill_linear(dq_inputs.bf16_to_f32_numpy(A), sa, ac, asc, ref["s"])
    check_outputs(_f64(out[:, :N]), Yr, S, "prefill on autocast weights")


def test_prefill_on_lut3_only_handle_casts_at_call_time(dq, oracle):
    """One stored 3.5-bit matrix serves both phases: the prefill call casts LUT3 to NVFP4 into
    its workspace.  Same result, bit for bit, as the pack-time view; parity against the oracle's
    autocast codes; N is not a multiple of the GEMM tile so the scale padding path runs."""
    M, N, K = 300, 784, 1152
    W, ref = _layer(oracle, N, K, 32)
    Wd = W.to(DEV)
    w_lut = dq.pack_weights(Wd, formats=dq.FMT_LUT3)
    w_view = dq.pack_weights(Wd, formats=dq.FMT_NVFP4_FROM_LUT3)
    assert dq.packed_bytes(N, K, dq.FMT_LUT3) < dq.packed_bytes(N, K, dq.FMT_NVFP4_FROM_LUT3)
    assert dq.prefill_workspace_bytes(w_lut, M) > dq.prefill_workspace_bytes(w_view, M)
    A = dq_inputs.gaussian_bf16(M, K, 1.0, 55)
    sa = dq_inputs.static_act_scale(A)
    ws = dq.alloc_workspace(dq.prefill_workspace_bytes(w_lut, M), DEV)
    ws.fill_(0xFF)                                   # stale workspace contents must not matter
    Y1 = dq.prefill_linear(w_lut, A.to(DEV), sa, workspace=ws)
    Y1b = dq.prefill_linear(w_lut, A.to(DEV), sa, workspace=ws)
    Y2 = dq.prefill_linear(w_view, A.to(DEV), sa)
    _status_ok(dq)
    assert torch.equal(Y1, Y2) and torch.equal(Y1, Y1b)
    ac = oracle.autocast_lut3_to_nvfp4(ref["lut3_planes"], ref["lut3_scales"])
    Yr, S = oracle.prefill_linear(dq_inputs.bf16_to_f32_numpy(A), sa, ac[0], ac[1], ref["s"])
    check_outputs(_f64(Y1), Yr, S, "prefill on a LUT3-only handle")
    y = dq.decode_linear(w_lut, A[:2].to(DEV))       # and the same handle still decodes
    Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(A[:2]), ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    check_outputs(_f64(y), Yr, S, "decode on the same handle")


def test_prefill_outlier_activations(dq, oracle):
    M, N, K = 256, 512, 1024
    W, ref = _layer(oracle, N, K, 57)
    A = dq_inputs.student_t_outlier_bf16(M, K, 58)
    sa = dq_inputs.static_act_scale(A)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4)
    Y = dq.prefill_linear(w, A.to(DEV), sa)
    _status_ok(dq)
    Yr, S = oracle.prefill_linear(dq_inputs.bf16_to_f32_numpy(A), sa, ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"])
    check_outputs(_f64(Y), Yr, S, "prefill with heavy-tailed activations")


DECODE_SHAPES = [(512, 256, 0), (144, 384, 61), (784, 1152, 62), (2048, 4096, 63)]


@pytest.mark.parametrize("N,K,seed", DECODE_SHAPES)
@pytest.mark.parametrize("B", [1, 2, 3, 8, 17, 64])
def test_decode_parity(dq, oracle, N, K, seed, B):
    W, ref = _layer(oracle, N, K, seed)
    X = dq_inputs.gaussian_bf16(B, K, 1.0, seed + 100 + B)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    Y = dq.decode_linear(w, X.to(DEV))
    _status_ok(dq)
    Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(X), ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    check_outputs(_f64(Y), Yr, S, f"decode {B}x{N}x{K}")


@pytest.mark.parametrize("N,K,seed", [(512, 256, 0), (144, 384, 31), (784, 1152, 32), (272, 17408, 33)])
@pytest.mark.parametrize("B", [1, 2, 3, 8, 17, 64])
def test_decode_nvfp4_parity(dq, oracle, N, K, seed, B):
    """Weight-only decode on the NVFP4 view; also from the LUT3-derived view of the same matrix."""
    W, ref = _layer(oracle, N, K, seed)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4)
    X = dq_inputs.gaussian_bf16(B, K, 1.0, 1000 + seed + B)
    Y = dq.decode_linear_nvfp4(w, X.to(DEV))
    _status_ok(dq)
    Yr, S = oracle.decode_linear_nvfp4(dq_inputs.bf16_to_f32_numpy(X), ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"])
    check_outputs(_f64(Y), Yr, S, f"nvfp4 decode {B}x{N}x{K}")
    if B == 2 and K <= 1152:
        w2 = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4_FROM_LUT3)
        ac, asc = oracle.autocast_lut3_to_nvfp4(ref["lut3_planes"], ref["lut3_scales"])
        Yr, S = oracle.decode_linear_nvfp4(dq_inputs.bf16_to_f32_numpy(X), ac, asc, ref["s"])
        check_outputs(_f64(dq.decode_linear_nvfp4(w2, X.to(DEV))), Yr, S, "nvfp4 decode on the LUT3-derived view")
        w3 = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
        with pytest.raises(dq.DQError):
            dq.decode_linear_nvfp4(w3, X.to(DEV))


def test_decode_nvfp4_kernels_agree_and_handle_wide_range_activations(dq, oracle):
    """The tensor-core kernel (default) and the CUDA-core kernel both meet the oracle; activations spanning
    many binades (the tensor-core kernel rescales them to fp16) and strided, guarded outputs."""
    N, K, B = 400, 2048, 5
    W, ref = _layer(oracle, N, K, 90)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4)
    g = torch.Generator().manual_seed(91)
    X = (torch.randn(B, K, generator=g) * torch.exp2(torch.randint(-20, 12, (B, K), generator=g).float())).to(torch.bfloat16)
    Yr, S = oracle.decode_linear_nvfp4(dq_inputs.bf16_to_f32_numpy(X), ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"])
    for variant in (0, 1):
        out = torch.full((B, N + 8), -3.0, dtype=torch.bfloat16, device=DEV)
        dq.test_decode_linear(w, dq.FMT_NVFP4, X.to(DEV), out=out[:, :N], variant=variant)
        _status_ok(dq)
        assert torch.all(out[:, N:] == -3.0)
        check_outputs(_f64(out[:, :N]), Yr, S, f"nvfp4 decode kernel variant {variant}, wide-range activations")


@pytest.mark.parametrize("N,K,seed", DECODE_SHAPES + [(272, 17408, 33), (48, 32768, 34)])
@pytest.mark.parametrize("B", [1, 3, 8, 11])
def test_decode_lut3_long_rows_and_forced_work_splits(dq, oracle, N, K, seed, B):
    """Default launch on long rows, then the same call with other splits of the work: one warp per tile, many
    warps per tile (several slices or a single atom each), shallow and deep copy rings."""
    W, ref = _layer(oracle, N, K, seed)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    X = dq_inputs.gaussian_bf16(B, K, 1.0, 2000 + seed + B)
    Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(X), ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    out = torch.full((B, N + 8), -3.0, dtype=torch.bfloat16, device=DEV)
    dq.decode_linear(w, X.to(DEV), out=out[:, :N])
    _status_ok(dq)
    assert torch.all(out[:, N:] == -3.0)
    check_outputs(_f64(out[:, :N]), Yr, S, f"lut3 decode {B}x{N}x{K}")
    if B in (1, 3):
        slices = (K + 1023) // 1024
        for P, G, S_ in ((1, 1, 2), (1, 7, 3), (min(slices, 3), 2, 8), (min(slices, 16), 1, 4), (min(slices, 32), 1, 2)):
            if 4096 + P * G * (512 + 1152 + S_ * 3584) + (slices * 2048 + 16) > 227 * 1024:
                continue                                     # does not fit shared memory even with one column per pass
            got = dq.test_decode_linear(w, dq.FMT_LUT3, X.to(DEV), warps_per_group=P, groups_per_cta=G, ring_stages=S_)
            _status_ok(dq)
            check_outputs(_f64(got), Yr, S, f"lut3 decode {B}x{N}x{K}, split P={P} G={G} S={S_}")


def test_decode_wait_budget_runs_out_cleanly(dq, oracle):
    """A device-side wait that gives up: one bulk copy is never requested (test hook), the wait for it runs out
    after a millisecond, the kernel returns normally, the status word says DQ_ERR_TIMEOUT, and the next call is right."""
    N, K = 4096, 4096
    W, ref = _layer(oracle, N, K, 99)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    X = dq_inputs.gaussian_bf16(2, K, 1.0, 100).to(DEV)
    torch.cuda.synchronize()
    assert dq.get_status()[0] == 0
    dq.test_decode_linear(w, dq.FMT_LUT3, X, variant=1, wait_cycles=2_000_000)
    torch.cuda.synchronize()
    st, det = dq.get_status()
    assert st == 7 and (det & 0xFF000) == 0x36000, (st, hex(det))      # DQ_ERR_TIMEOUT from the LUT decode kernel
    assert dq.get_status()[0] == 0                                     # the read cleared it
    Y = dq.decode_linear(w, X)
    _status_ok(dq)
    Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(X.cpu()), ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    check_outputs(_f64(Y), Yr, S, "decode after a timed-out call")


def _sparse_patterns(K, seed):
    """Activation rows on which a sum of K products is dominated by a handful of them: 1, 2, 3, 8 and 32 non-zeros
    with random bf16 values and with +-1, two columns of one 16-block that cancel, two columns far apart."""
    g = torch.Generator().manual_seed(seed)
    rows = []
    for nnz in (1, 2, 3, 8, 32):
        for signs_only in (False, True):
            x = torch.zeros(K)
            pos = torch.randperm(K, generator=g)[:nnz]
            if signs_only:
                x[pos] = torch.randint(0, 2, (nnz,), generator=g).float() * 2 - 1
            else:
                x[pos] = torch.randn(nnz, generator=g) * torch.exp2(torch.randint(-3, 4, (nnz,), generator=g).float())
            rows.append(x)
    for blk, i, j in ((0, 0, 1), (K // 32, 3, 12), (K // 16 - 1, 15, 14)):      # +1 / -1 inside one block
        x = torch.zeros(K)
        x[16 * blk + i], x[16 * blk + j] = 1.0, -1.0
        rows.append(x)
    x = torch.zeros(K)
    x[5], x[700] = 1.0, 1.0
    rows.append(x)
    x = torch.zeros(K)
    x[K - 1], x[K // 2] = 3.0, -3.0
    rows.append(x)
    while len(rows) % 8:
        rows.append(rows[len(rows) % 5])
    return torch.stack(rows).to(torch.bfloat16)


@pytest.mark.parametrize("N,K,seed", [(2048, 2048, 95), (1024, 4096, 96), (512, 8192, 97), (256, 5120, 98)])
@pytest.mark.parametrize("B", [1, 2, 8])
def test_decode_sparse_and_cancelling_activations(dq, oracle, N, K, seed, B):
    """Per-element bound on inputs where nothing averages out: every product must be exact up to fp32
    accumulation, so a few non-zero activations (or two that cancel) meet the same bound as dense rows."""
    W, ref = _layer(oracle, N, K, seed)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    P = _sparse_patterns(K, seed + 1)
    Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(P), ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    Pd = P.to(DEV)
    got = torch.cat([dq.decode_linear(w, Pd[i:i + B]) for i in range(0, P.shape[0], B)])
    _status_ok(dq)
    check_outputs(_f64(got), Yr, S, f"decode, sparse / cancelling activations, batch {B}, {N}x{K}")
    # a single non-zero activation of 1.0 reads one dequantised column: exact after the bf16 rounding
    What = oracle.dequant_lut3(ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    for k in (0, 17, K // 2 + 5, K - 1):
        x = torch.zeros(1, K, dtype=torch.bfloat16)
        x[0, k] = 1.0
        y = _f64(dq.decode_linear(w, x.to(DEV)))[0]
        want = torch.from_numpy(What[:, k]).to(torch.bfloat16).float().numpy().astype(np.float64)
        assert np.array_equal(y, want), f"one-hot column {k}"


def test_decode_lut3_wide_range_activations(dq, oracle):
    """Activations spanning many binades (the kernel rescales them by a power of two into fp16), strided and
    guarded outputs."""
    N, K = 400, 2048
    W, ref = _layer(oracle, N, K, 90)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    for B in (1, 5):
        g = torch.Generator().manual_seed(91 + B)
        X = (torch.randn(B, K, generator=g) * torch.exp2(torch.randint(-20, 12, (B, K), generator=g).float())).to(torch.bfloat16)
        Yr, S = oracle.decode_linear(dq_inputs.bf16_to_f32_numpy(X), ref["lut3_planes"], ref["lut3_scales"], ref["s"])
        out = torch.full((B, N + 8), -3.0, dtype=torch.bfloat16, device=DEV)
        dq.decode_linear(w, X.to(DEV), out=out[:, :N])
        _status_ok(dq)
        assert torch.all(out[:, N:] == -3.0)
        check_outputs(_f64(out[:, :N]), Yr, S, f"lut3 decode, wide-range activations, batch {B}")


_lut2_cache = {}


def _lut2_layer(oracle, N, K, seed):
    key = (N, K, seed)
    if key not in _lut2_cache:
        W = dq_inputs.gaussian_bf16(N, K, 0.02, seed)
        Wf = dq_inputs.bf16_to_f32_numpy(W)
        s = oracle.global_scale(oracle.absmax(Wf))
        _lut2_cache[key] = (W, s) + oracle.quant_lut2(Wf, s)
    return _lut2_cache[key]


@pytest.mark.parametrize("N,K,seed", [(512, 256, 0), (144, 384, 31), (784, 1152, 32)])
def test_pack_lut2_bit_exact(dq, oracle, N, K, seed):
    """LUT2 planes and signed scales against the oracle, alone and next to LUT3 in one handle."""
    W, s, planes, scales = _lut2_layer(oracle, N, K, seed)
    for fmts in (dq.FMT_LUT2, dq.FMT_LUT2 | dq.FMT_LUT3 | dq.FMT_NVFP4):
        w = dq.pack_weights(W.to(DEV), formats=fmts)
        p, sc, s_dev = dq.export_canonical(w, dq.FMT_LUT2)
        _status_ok(dq)
        assert np.float32(_np(s_dev)[0]) == np.float32(s)
        assert _np(p).shape == (N, 2, K // 32)
        assert np.array_equal(_np(sc), scales)
        assert np.array_equal(_np(p).view(np.uint32), planes)
    if fmts & dq.FMT_LUT3:
        _, ref = _layer(oracle, N, K, seed)
        p3, sc3, _ = dq.export_canonical(w, dq.FMT_LUT3)
        assert np.array_equal(_np(p3).view(np.uint32), ref["lut3_planes"]) and np.array_equal(_np(sc3), ref["lut3_scales"])
    # degenerate blocks: zeros, sign ties, one huge outlier
    X = dq_inputs.gaussian_bf16(32, 128, 0.02, 34)
    X[0, :16] = 0
    X[1, 0], X[1, 5] = 0.5, -0.5
    X[3, 7] = 3.0e4
    Xf = dq_inputs.bf16_to_f32_numpy(X)
    s2 = oracle.global_scale(oracle.absmax(Xf))
    rp, rs = oracle.quant_lut2(Xf, s2)
    p, sc, _ = dq.export_canonical(dq.pack_weights(X.to(DEV), formats=dq.FMT_LUT2), dq.FMT_LUT2)
    assert np.array_equal(_np(p).view(np.uint32), rp) and np.array_equal(_np(sc), rs)


@pytest.mark.parametrize("N,K,seed", DECODE_SHAPES + [(272, 17408, 33)])
@pytest.mark.parametrize("B", [1, 2, 3, 8, 17, 64])
def test_decode_lut2_parity(dq, oracle, N, K, seed, B):
    W, s, planes, scales = _lut2_layer(oracle, N, K, seed)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT2)
    X = dq_inputs.gaussian_bf16(B, K, 1.0, 3000 + seed + B)
    out = torch.full((B, N + 8), -3.0, dtype=torch.bfloat16, device=DEV)
    dq.decode_linear_lut2(w, X.to(DEV), out=out[:, :N])
    _status_ok(dq)
    assert torch.all(out[:, N:] == -3.0)
    Yr, S = oracle.decode_linear_lut2(dq_inputs.bf16_to_f32_numpy(X), planes, scales, s)
    check_outputs(_f64(out[:, :N]), Yr, S, f"lut2 decode {B}x{N}x{K}")


def test_decode_lut2_sparse_activations_and_wrong_handle(dq, oracle):
    N, K = 1024, 4096
    W, s, planes, scales = _lut2_layer(oracle, N, K, 96)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT2)
    P = _sparse_patterns(K, 97)
    Yr, S = oracle.decode_linear_lut2(dq_inputs.bf16_to_f32_numpy(P), planes, scales, s)
    for B in (1, 4):
        got = torch.cat([dq.decode_linear_lut2(w, P.to(DEV)[i:i + B]) for i in range(0, P.shape[0], B)])
        _status_ok(dq)
        check_outputs(_f64(got), Yr, S, f"lut2 decode, sparse / cancelling activations, batch {B}")
    with pytest.raises(dq.DQError):
        dq.decode_linear(w, P.to(DEV)[:1])                        # no LUT3 in this handle
    w3 = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    with pytest.raises(dq.DQError):
        dq.decode_linear_lut2(w3, P.to(DEV)[:1])


@pytest.mark.parametrize("N,K,seed", [(144, 384, 31), (784, 1152, 32)])
def test_import_canonical_lut2_round_trip(dq, oracle, N, K, seed):
    """A LUT2 handle built from the oracle's canonical planes and scales exports the same bits again and decodes
    like the handle packed from the master weights (K not a multiple of the 1024-weight slice: padded atoms)."""
    W, s, planes, scales = _lut2_layer(oracle, N, K, seed)
    w_imp = dq.import_canonical_lut2(N, K, s, torch.from_numpy(planes.view(np.int32)).to(DEV).contiguous(),
                                     torch.from_numpy(scales).to(DEV).contiguous())
    p2, s2, g2 = dq.export_canonical(w_imp, dq.FMT_LUT2)
    assert np.float32(g2.cpu().numpy()[0]) == np.float32(s)
    assert np.array_equal(p2.cpu().numpy().view(np.uint32), planes) and np.array_equal(s2.cpu().numpy(), scales)
    w_pack = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT2)
    X = dq_inputs.gaussian_bf16(5, K, 1.0, seed + 700).to(DEV)
    assert torch.equal(dq.decode_linear_lut2(w_imp, X), dq.decode_linear_lut2(w_pack, X))
    Yr, S = oracle.decode_linear_lut2(dq_inputs.bf16_to_f32_numpy(X.cpu()), planes, scales, s)
    check_outputs(_f64(dq.decode_linear_lut2(w_imp, X)), Yr, S, "decode on an imported LUT2 handle")
    _status_ok(dq)
    with pytest.raises(dq.DQError):
        dq.decode_linear(w_imp, X)                                # LUT2 only
    rc = dq.lib().dq_import_canonical_lut2(N, K, None, None, 1.0, None, 0, None, None)
    assert rc == 1


def test_decode_one_hot_and_strided(dq, oracle):
    N, K = 256, 512
    W, ref = _layer(oracle, N, K, 64)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    What = oracle.dequant_lut3(ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    X = torch.zeros(4, K + 8, dtype=torch.bfloat16)
    ks = [0, 17, 130, 511]
    for b, k in enumerate(ks):
        X[b, k] = 1.0
    out = torch.full((4, N + 8), -3.0, dtype=torch.bfloat16, device=DEV)
    dq.decode_linear(w, X.to(DEV)[:, :K], out=out[:, :N])
    _status_ok(dq)
    assert torch.all(out[:, N:] == -3.0)
    got = _f64(out[:, :N])
    for b, k in enumerate(ks):      # one dequantised column, rounded to bf16
        want = torch.from_numpy(What[:, k]).to(torch.bfloat16).float().numpy().astype(np.float64)
        assert np.array_equal(got[b], want)


def test_calls_reject_wrong_handle_use(dq, oracle):
    N, K = 64, 128
    W, _ = _layer(oracle, N, K, 65)
    w_lut = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    w_nv = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4)
    A = dq_inputs.gaussian_bf16(4, K, 1.0, 66).to(DEV)
    with pytest.raises(dq.DQError) as e:
        dq.decode_linear(w_nv, A)
    assert e.value.code == 1
    with pytest.raises(dq.DQError) as e:
        dq.prefill_linear(w_nv, A, 1.0, workspace=torch.empty(1024, dtype=torch.uint8, device=DEV)[:16])
    assert e.value.code in (3, 4)
    with pytest.raises(dq.DQError):
        dq.prefill_linear(w_nv, A, -1.0)
    _status_ok(dq)


def test_calls_replay_from_a_cuda_graph(dq, oracle):
    """Prefill and decode calls neither allocate nor synchronise, so a stream capture records
    them; replays on new inputs (same buffers) give what eager calls give, bit for bit."""
    M, N, K = 384, 512, 1024
    W, ref = _layer(oracle, N, K, 70)
    w = dq.pack_weights(W.to(DEV))
    ws = dq.alloc_workspace(dq.prefill_workspace_bytes(w, M), DEV)
    A = dq_inputs.gaussian_bf16(M, K, 1.0, 71).to(DEV)
    X = dq_inputs.gaussian_bf16(4, K, 1.0, 72).to(DEV)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    Yd = torch.empty(4, N, dtype=torch.bfloat16, device=DEV)
    sa = 4.0 / 2688.0
    dq.prefill_linear(w, A, sa, out=Y, workspace=ws)     # first calls outside capture (one-time set-up)
    dq.decode_linear(w, X, out=Yd)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        dq.prefill_linear(w, A, sa, out=Y, workspace=ws)
        dq.decode_linear(w, X, out=Yd)
    for seed in (73, 74):
        A.copy_(dq_inputs.gaussian_bf16(M, K, 1.0, seed).to(DEV))
        X.copy_(dq_inputs.gaussian_bf16(4, K, 1.0, seed + 10).to(DEV))
        Y.zero_(); Yd.zero_()
        graph.replay()
        torch.cuda.synchronize()
        got, got_d = Y.clone(), Yd.clone()
        want = dq.prefill_linear(w, A, sa, workspace=ws)
        want_d = dq.decode_linear(w, X)
        _status_ok(dq)
        assert torch.equal(got, want) and torch.equal(got_d, want_d)
    Yr, S = oracle.prefill_linear(dq_inputs.bf16_to_f32_numpy(A.cpu()), sa, ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"])
    check_outputs(_f64(Y), Yr, S, "graph replay prefill")


def test_one_handle_serves_several_streams_at_once(dq, oracle):
    """A handle is immutable after packing: prefill calls (each with its own workspace) and decode calls issued on
    three streams at the same time give what the same calls give one after the other, bit for bit."""
    M, N, K = 640, 2048, 2048
    W, _ = _layer(oracle, N, K, 75)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4 | dq.FMT_LUT3 | dq.FMT_LUT2)
    sa = 4.0 / 2688.0
    streams = [torch.cuda.Stream(device=DEV) for _ in range(3)]
    A = [dq_inputs.gaussian_bf16(M, K, 1.0, 760 + i).to(DEV) for i in range(3)]
    X = [dq_inputs.gaussian_bf16(3, K, 1.0, 770 + i).to(DEV) for i in range(3)]
    wss = [dq.alloc_workspace(dq.prefill_workspace_bytes(w, M), DEV) for _ in range(3)]
    want = [(dq.prefill_linear(w, A[i], sa, workspace=wss[i]), dq.decode_linear(w, X[i]), dq.decode_linear_lut2(w, X[i]),
             dq.decode_linear_nvfp4(w, X[i])) for i in range(3)]
    torch.cuda.synchronize()
    got = [None] * 3
    for rep in range(4):                                   # several rounds so that the launches really interleave
        for i, st in enumerate(streams):
            with torch.cuda.stream(st):
                got[i] = (dq.prefill_linear(w, A[i], sa, workspace=wss[i], stream=st), dq.decode_linear(w, X[i], stream=st),
                          dq.decode_linear_lut2(w, X[i], stream=st), dq.decode_linear_nvfp4(w, X[i], stream=st))
    torch.cuda.synchronize()
    _status_ok(dq)
    for i in range(3):
        for a, b in zip(got[i], want[i]):
            assert torch.equal(a, b)


def test_host_buffer_entry_points_match_device_calls(dq, oracle):
    """Pinned host activations in, host outputs back, copies inside the call (row chunks pipelined over
    three streams): same bits as the device-pointer calls; strided host rows; M not a multiple of a chunk."""
    M, N, K = 2500, 512, 1024
    W, _ = _layer(oracle, N, K, 80)
    w = dq.pack_weights(W.to(DEV))
    A_full = dq_inputs.gaussian_bf16(M, K + 64, 1.0, 81).pin_memory()
    A_host = A_full[:, :K]
    sa = dq_inputs.static_act_scale(A_host)
    Y_full = torch.full((M, N + 32), 7.0, dtype=torch.bfloat16).pin_memory()
    staging = dq.alloc_workspace(dq.prefill_host_staging_bytes(w, M), DEV)
    for _ in range(2):                                   # twice in a row on the same stream
        dq.prefill_linear_host(w, A_host, sa, Y_full[:, :N], staging)
    torch.cuda.synchronize()
    want = dq.prefill_linear(w, A_host.contiguous().to(DEV), sa)
    _status_ok(dq)
    assert torch.equal(Y_full[:, :N], want.cpu()) and torch.all(Y_full[:, N:] == 7.0)
    X_host = A_host[:3]
    Yd_host = torch.zeros(3, N, dtype=torch.bfloat16).pin_memory()
    dq.decode_linear_host(w, X_host, Yd_host, staging)
    torch.cuda.synchronize()
    assert torch.equal(Yd_host, dq.decode_linear(w, X_host.contiguous().to(DEV)).cpu())
    with pytest.raises(dq.DQError):
        dq.prefill_linear_host(w, A_host, sa, Y_full[:, :N], staging[:4096])
    _status_ok(dq)


# ---- the tcgen05 decode kernel (test-hook variant 3; batch 1): same arithmetic, other machinery ----

@pytest.mark.parametrize("N,K,seed", DECODE_SHAPES + [(400, 5120, 64), (3072, 12288, 65)])
def test_decode_tcgen05_kernel_parity(dq, oracle, N, K, seed):
    """Levels through tensor memory, one tcgen05.mma per 16-weight block: LUT3 and LUT2 against the oracle, on rows
    that do not fill the last 128-row tile, one to three warpgroups' worth of K, and sparse activations."""
    W, ref = _layer(oracle, N, K, seed)
    W2, s2, planes2, scales2 = _lut2_layer(oracle, N, K, seed)
    assert torch.equal(W, W2)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3 | dq.FMT_LUT2)
    rows = [dq_inputs.gaussian_bf16(1, K, 1.0, seed + 500)]
    if K >= 1024:
        sp = _sparse_patterns(K, seed + 501)
        rows += [sp[0:1], sp[3:4], sp[10:11], sp[13:14]]
    for X in rows:
        Xf = dq_inputs.bf16_to_f32_numpy(X)
        out = torch.full((1, N + 8), -3.0, dtype=torch.bfloat16, device=DEV)
        dq.test_decode_linear(w, dq.FMT_LUT3, X.to(DEV), out=out[:, :N], variant=3)
        _status_ok(dq)
        assert torch.all(out[:, N:] == -3.0)
        Yr, S = oracle.decode_linear(Xf, ref["lut3_planes"], ref["lut3_scales"], ref["s"])
        check_outputs(_f64(out[:, :N]), Yr, S, f"tcgen05 lut3 decode {N}x{K}")
        dq.test_decode_linear(w, dq.FMT_LUT2, X.to(DEV), out=out[:, :N], variant=3)
        _status_ok(dq)
        Yr, S = oracle.decode_linear_lut2(Xf, planes2, scales2, s2)
        check_outputs(_f64(out[:, :N]), Yr, S, f"tcgen05 lut2 decode {N}x{K}")


def test_decode_tcgen05_kernel_limits(dq):
    """Batch 1 only, and rows short enough for its shared-memory layout; anything else is refused, not computed."""
    W = dq_inputs.gaussian_bf16(256, 16384, 0.02, 66)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    X = dq_inputs.gaussian_bf16(2, 16384, 1.0, 67).to(DEV)
    with pytest.raises(dq.DQError):
        dq.test_decode_linear(w, dq.FMT_LUT3, X[:1], variant=3)          # K too long
    W = dq_inputs.gaussian_bf16(256, 1024, 0.02, 68)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3)
    X = dq_inputs.gaussian_bf16(2, 1024, 1.0, 69).to(DEV)
    with pytest.raises(dq.DQError):
        dq.test_decode_linear(w, dq.FMT_LUT3, X, variant=3)              # batch 2
    dq.test_decode_linear(w, dq.FMT_LUT3, X[:1], variant=3)
    _status_ok(dq)


# ---- batches above 8: the kernel that walks K slice by slice with 16 or 32 columns a pass (test-hook variant 4) ----

@pytest.mark.parametrize("N,K,seed", DECODE_SHAPES + [(400, 5120, 64)])
@pytest.mark.parametrize("B", [9, 16, 17, 33, 64])
def test_decode_wide_batch_kernel_parity(dq, oracle, N, K, seed, B):
    """LUT3 and LUT2 against the oracle; activations whose slices differ by many binades (every slice has its own
    power-of-two scale); strided rows and outputs."""
    W, ref = _layer(oracle, N, K, seed)
    W2, s2, planes2, scales2 = _lut2_layer(oracle, N, K, seed)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_LUT3 | dq.FMT_LUT2)
    X = dq_inputs.gaussian_bf16(B, K, 1.0, seed + 600 + B)
    X[:, : K // 2] *= 2.0 ** 20
    X[1] = 0
    Xd = torch.zeros(B, K + 8, dtype=torch.bfloat16, device=DEV)
    Xd[:, :K] = X.to(DEV)
    Xf = dq_inputs.bf16_to_f32_numpy(X)
    out = torch.full((B, N + 8), -3.0, dtype=torch.bfloat16, device=DEV)
    dq.test_decode_linear(w, dq.FMT_LUT3, Xd[:, :K], out=out[:, :N], variant=4)
    _status_ok(dq)
    assert torch.all(out[:, N:] == -3.0)
    Yr, S = oracle.decode_linear(Xf, ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    check_outputs(_f64(out[:, :N]), Yr, S, f"wide lut3 decode {B}x{N}x{K}")
    dq.test_decode_linear(w, dq.FMT_LUT2, Xd[:, :K], out=out[:, :N], variant=4)
    _status_ok(dq)
    Yr, S = oracle.decode_linear_lut2(Xf, planes2, scales2, s2)
    check_outputs(_f64(out[:, :N]), Yr, S, f"wide lut2 decode {B}x{N}x{K}")


def test_measurement_hooks_leave_results_alone(dq, oracle):
    """The measurement hooks (MMA issue sequence alone, streaming read, in-kernel clocks of the last pair GEMM) run, return
    sane values and do not disturb a following prefill: its output is the one from before, bit for bit."""
    M, N, K = 512, 1024, 1024
    W, _ = _layer(oracle, N, K, 90)
    w = dq.pack_weights(W.to(DEV), formats=dq.FMT_NVFP4)
    A = dq_inputs.gaussian_bf16(M, K, 1.0, 91).to(DEV)
    ws = dq.alloc_workspace(dq.prefill_workspace_bytes(w, M), DEV)
    sa = 4.0 / 2688.0
    Y0 = dq.prefill_linear(w, A, sa, workspace=ws)
    cycles, ns = dq.bench_gemm_clocks()
    assert cycles > 0 and ns > 0
    assert 500.0 < cycles / ns * 1e3 < 2500.0                  # an SM clock in MHz
    scratch = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    dq.bench_gemm_mma_only(w, M, scratch, ws)
    c2, n2 = dq.bench_gemm_clocks()
    assert c2 > 0 and n2 > 0 and (c2, n2) != (cycles, ns)
    out = torch.zeros(8, dtype=torch.uint8, device=DEV)
    dq.bench_stream_read(w.packed[: w.packed.numel() // 16 * 16], out)
    _status_ok(dq)
    assert torch.equal(dq.prefill_linear(w, A, sa, workspace=ws), Y0)
    with pytest.raises(dq.DQError):
        dq.bench_gemm_mma_only(w, 64, scratch, ws)             # the measurement mode exists for M > 128 only
