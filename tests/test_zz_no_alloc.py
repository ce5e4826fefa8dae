"""The workspace-free trainer log-prob entry point against the regular one (GPU).

ais_logprob_train_static serves callers that own nothing but their inputs and outputs - a callback inside
another framework, or a process whose device memory has all been given to some other pool - and so cannot
supply the workspace that ais_logprob_fwd needs.  It keeps its scratch in a fixed array inside the library.
The array is shared by all calls and keeps old contents, so the check is made on calls in a row with different
shapes: a later one must not be disturbed by what an earlier one left behind, in particular when it streams the
vocabulary in fewer ranges and so leaves planes of the array untouched.  Every call is compared with the regular
entry point and with the float64 oracle.  This file is named to be collected last.
"""

import numpy as np
import pytest
import torch

import workloads
from oracle import ais as oais

pytestmark = pytest.mark.gpu

LP_ATOL = 1e-2          # the log-prob tolerance of the other GPU tests


def _case(ais, w, check_free_memory=False):
    b = workloads.make_batch(w, device="cpu")
    H, W, tok, msk = b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda()
    T = b.T
    step = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block)
    ais.logprob_fwd(step.shape, step.params, H, W, None, None, None, None, tok, msk, step.lp_train, step.lse_train,
                    None, None, step.status, step.workspace)
    lp = torch.full((T,), 7.0, dtype=torch.float32, device="cuda")
    lse = torch.full((T,), 7.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before = torch.cuda.mem_get_info()[0]
    ais.logprob_train_static(step.shape, H, W, tok, msk, lp, lse, status)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before            # nothing was taken from torch's allocator
    if check_free_memory:                                     # nor from the device (not on a device's first call, which
        assert torch.cuda.mem_get_info()[0] == free_before    # may still load the library image with the array in it)
    assert int(status.item()) == 0 and int(step.status.item()) == 0
    assert float((lp - step.lp_train[:T]).abs().max()) <= LP_ATOL
    assert float((lse - step.lse_train[:T]).abs().max()) <= LP_ATOL
    assert torch.all(lp[msk == 0] == 0)
    a = workloads.to_numpy(b)
    ref_lp, ref_lse = oais.logprob_train(a["H"], a["W"], a["tokens"], a["mask"])
    assert np.max(np.abs(lp.cpu().numpy() - ref_lp)) <= LP_ATOL
    assert np.max(np.abs(lse.cpu().numpy() - ref_lse)) <= LP_ATOL
    return lp


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    import paper_2605_13907_b200 as ais
    base = workloads.WORKLOADS["tiny"]
    # first call: several row tiles, ragged vocabulary tail, some rows masked out
    w1 = workloads.scaled(base, d=384, V=1336, P=3, G=4, lengths="uniform:50:200", mask_mode="llada", seed=71)
    lp1 = _case(ais, w1)
    # second call right after it: fewer rows and another vocabulary size, so stale partials lie beyond and beside its own
    w2 = workloads.scaled(base, d=256, V=1024, P=2, G=2, lengths="uniform:10:60", seed=72)
    lp2 = _case(ais, w2, check_free_memory=True)
    # third call: two 256-column tiles only, so the vocabulary goes in 2 ranges and 4 of the 8 planes keep what the
    # calls before wrote there; then a one-range call
    w3 = workloads.scaled(base, d=256, V=512, P=2, G=2, lengths="uniform:20:90", seed=73)
    lp3 = _case(ais, w3, check_free_memory=True)
    w4 = workloads.scaled(base, d=128, V=256, P=1, G=2, lengths="uniform:100:140", seed=74)
    lp4 = _case(ais, w4, check_free_memory=True)
    assert lp1.shape != lp2.shape
    for lp in (lp1, lp2, lp3, lp4):
        assert torch.isfinite(lp).all()


def test_static_scratch_rejects_too_many_rows():
    import paper_2605_13907_b200 as ais
    T = ais.STATIC_MAX_ROWS + 1
    shape = ais.binding.make_shape(T, 256, 1024, 1, 1, 128)
    H = torch.zeros(T, 256, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(1024, 256, dtype=torch.bfloat16, device="cuda")
    tok = torch.zeros(T, dtype=torch.int32, device="cuda")
    msk = torch.ones(T, dtype=torch.uint8, device="cuda")
    lp = torch.zeros(T, dtype=torch.float32, device="cuda")
    with pytest.raises(ais.AisError, match="limit"):
        ais.logprob_train_static(shape, H, W, tok, msk, lp)
