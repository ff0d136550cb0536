"""dq_prefill_linear_static (the entry point for callers that cannot allocate device memory:
the scratch is an array inside the library) must give the same bits as dq_prefill_linear.

Collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test.  It passes alone in a fresh process and after the rest of the suite."""
import pytest
import torch

import dq_inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def dq():
    import __graft_entry__ as g
    g.build()
    import paper_2609_26333_b200 as dq
    assert torch.cuda.is_available()
    return dq


def test_static_scratch_matches_workspace_version_twice_in_a_row(dq):
    N, K = 784, 640
    W = dq_inputs.gaussian_bf16(N, K, 0.02, 901).to(DEV)
    w = dq.pack_weights(W, formats=dq.FMT_NVFP4)
    # second call is smaller than the first, so the scratch still holds the first call's rows
    for M, seed in ((300, 902), (129, 903)):
        A = dq_inputs.gaussian_bf16(M, K, 1.0, seed)
        sa = dq_inputs.static_act_scale(A)
        A = A.to(DEV)
        want = dq.prefill_linear(w, A, sa)
        got = dq.prefill_linear_static(w, A, sa)
        torch.cuda.synchronize()
        st, det = dq.get_status()
        assert st == 0, (st, det)
        assert got.shape == want.shape
        assert torch.equal(got, want), f"M={M}: static-scratch output differs from the workspace version"
        assert torch.isfinite(got.float()).all()


def test_static_scratch_rejects_oversized_problems(dq):
    N, K = 256, 4096
    W = dq_inputs.gaussian_bf16(N, K, 0.02, 904).to(DEV)
    w = dq.pack_weights(W, formats=dq.FMT_NVFP4)
    M = 4096                                   # 4096 x 4096 needs 9 MiB of scratch, the array has 8 MiB
    assert dq.prefill_workspace_bytes(w, M) > 8 * 1024 * 1024
    A = torch.zeros(M, K, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(dq.DQError) as e:
        dq.prefill_linear_static(w, A, 1.0)
    assert e.value.code == 4                   # DQ_ERR_WORKSPACE
    # and a size just inside the limit runs
    M_ok = 2048
    assert dq.prefill_workspace_bytes(w, M_ok) <= 8 * 1024 * 1024
    A = dq_inputs.gaussian_bf16(M_ok, K, 1.0, 905).to(DEV)
    sa = 0.002
    assert torch.equal(dq.prefill_linear_static(w, A, sa), dq.prefill_linear(w, A, sa))
    torch.cuda.synchronize()
    assert dq.get_status()[0] == 0
