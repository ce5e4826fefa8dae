"""The two conditions that only the device can see, reached without faulting anything: a non-finite value in the
inputs (ordinary floating-point arithmetic carries it to the row's log-prob) and a bounded wait that runs out (the
bound is lowered through the C ABI; the kernels give up in an orderly way and the next call works)."""

import numpy as np
import pytest
import torch

import workloads
from oracle import ais as oais

pytestmark = pytest.mark.gpu

LP_ATOL, ALPHA_ATOL, DH_REL = 1e-2, 1e-3, 1e-2


def _cuda(b):
    return workloads.Batch(b.workload, b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda(), b.seq_offsets, b.rewards)


def test_non_finite_hidden_state_raises_the_flag_and_neutralises_the_row():
    """One valid row of H holds +inf: AIS_FLAG_NONFINITE, lp = 0 for that row in both passes, lse_train = NaN as the
    mark, a zero row of dH; every other row is what the oracle gives for the batch in which that row has
    lp_train = lp_roll = 0 and takes no part in the loss."""
    import paper_2605_13907_b200 as ais
    w = workloads.scaled(workloads.WORKLOADS["tiny"], V=776, P=2, G=4, lengths="uniform:40:90", seed=61)
    clean = workloads.make_batch(w, device="cpu")
    bad = 37
    assert int(clean.mask[bad]) == 1
    a = workloads.to_numpy(clean)
    b = _cuda(clean)
    b.H[bad, 5] = float("inf")
    T = b.T
    step = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block)
    step.step(b.H, b.W, b.tokens, b.mask, b.seq_offsets.cuda(), b.rewards.cuda())
    torch.cuda.synchronize()
    assert int(step.status.item()) == ais.FLAG_NONFINITE
    lp_t = step.lp_train[:T].cpu().numpy().astype(np.float64)
    lp_r = step.lp_roll[:T].cpu().numpy().astype(np.float64)
    lse = step.lse_train[:T].cpu().numpy()
    assert lp_t[bad] == 0 and lp_r[bad] == 0 and np.isnan(lse[bad]) and np.isfinite(np.delete(lse, bad)).all()
    # the other rows do not see the bad one
    ref_t, _ = oais.logprob_train(a["H"], a["W"], a["tokens"], a["mask"])
    ref_r, _, _ = oais.logprob_rollout(a["H"], a["W"], a["tokens"], a["mask"], w.block)
    ref_t[bad] = 0.0
    ref_r[bad] = 0.0
    assert np.max(np.abs(lp_t - ref_t)) <= LP_ATOL and np.max(np.abs(lp_r - ref_r)) <= LP_ATOL
    # diagnostics: the row counts as one with equal log-probs
    adv = oais.advantages(a["rewards"], w.G)
    sid = oais.seq_ids(a["seq_offsets"], T)
    diag = oais.diagnostics(lp_t, lp_r, a["mask"], adv[sid], oais.Params())
    d = step.read_diag()
    assert d["n_valid"] == diag["n_valid"] and abs(d["alpha"] - diag["alpha"]) <= ALPHA_ATOL
    assert float(step.rho[bad]) == 1.0
    # loss and gradient: the row is left out (its count still normalises its sequence)
    _, _, wbar = oais.ratios(lp_t, lp_r, a["mask"], 5.0)
    w_tilde = oais.rectify(wbar, diag["alpha"], a["mask"])
    loss, c = oais.loss_and_coeff(lp_t, lp_t, a["mask"], a["seq_offsets"], adv, w_tilde, w.P, w.G, 0.2)
    n_s = oais.valid_counts(a["mask"], a["seq_offsets"])[sid[bad]]
    loss_without = loss + w_tilde[bad] * adv[sid[bad]] / (w.P * w.G * n_s)
    assert abs(float(step.loss.item()) - loss_without) <= 1e-3 * max(1.0, abs(loss_without))
    c[bad] = 0.0
    dH_ref = oais.grad_hidden(a["H"], a["W"], a["tokens"], c)
    dH = step.dH[:T].float().cpu().numpy().astype(np.float64)
    assert np.all(dH[bad] == 0) and np.isfinite(dH).all()
    assert np.linalg.norm(dH - dH_ref) <= DH_REL * np.linalg.norm(dH_ref)


def test_a_wait_that_runs_out_raises_the_flag_and_the_next_call_is_correct():
    """ais_set_wait_cycles(1): the first wait of every tensor-core pass runs out (a tile copy takes far longer than
    one clock tick), each CTA awaits its copies in flight, frees its tensor memory and ends; the calls return
    AIS_FLAG_TIMEOUT in the status word.  With the default bound restored the same objects give the oracle's results."""
    import paper_2605_13907_b200 as ais
    w = workloads.scaled(workloads.WORKLOADS["tiny"], d=512, V=1336, P=2, G=4, lengths="uniform:40:90", seed=62)
    b = _cuda(workloads.make_batch(w, device="cpu"))
    a = workloads.to_numpy(b)
    offs, rew = b.seq_offsets.cuda(), b.rewards.cuda()
    step = ais.AisStep(b.T, w.d, w.V, w.P, w.G, w.block)
    try:
        ais.set_wait_cycles(1)
        step.forward(b.H, b.W, b.tokens, b.mask)
        torch.cuda.synchronize()
        fwd_status = int(step.status.item())
        step.status.zero_()
        step.lse_train.fill_(3.0)                            # finite values, so that the backward passes have rows to do
        step.lp_train.fill_(-3.0)
        step.lp_roll.fill_(-3.0)
        step.diagnose(b.mask, offs, rew)
        step.backward(b.H, b.W, b.tokens, b.mask, offs)
        torch.cuda.synchronize()
        bwd_status = int(step.status.item())
    finally:
        ais.set_wait_cycles(0)
    assert fwd_status & ais.FLAG_TIMEOUT and bwd_status & ais.FLAG_TIMEOUT
    with pytest.raises(ais.AisError):
        ais.set_wait_cycles(-5)
    # the device and the library are as before: an ordinary step on the same buffers
    step.status.zero_()
    step.step(b.H, b.W, b.tokens, b.mask, offs, rew)
    torch.cuda.synchronize()
    assert int(step.status.item()) == 0
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block)
    T = b.T
    assert np.max(np.abs(step.lp_train[:T].cpu().numpy() - ref["lp_train"])) <= LP_ATOL
    assert np.max(np.abs(step.lp_roll[:T].cpu().numpy() - ref["lp_roll"])) <= LP_ATOL
    assert abs(step.read_diag()["alpha"] - ref["diag"]["alpha"]) <= ALPHA_ATOL
    dH = step.dH[:T].float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(dH - ref["dH"]) <= DH_REL * np.linalg.norm(ref["dH"])
