"""The data-parallel form of the path on one GPU: the split diagnostics API against the fused one, and two prompt
shards processed one after the other (their moment vectors added on the device, as an all-reduce would) against
the oracle's result for the whole batch."""

import numpy as np
import pytest
import torch

import workloads
from oracle import ais as oais
from paper_2605_13907_b200 import dist as adist

pytestmark = pytest.mark.gpu


def _cuda(b):
    return workloads.Batch(b.workload, b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda(), b.seq_offsets, b.rewards)


def test_split_diagnostics_equal_fused_bitwise():
    import paper_2605_13907_b200 as ais
    w = workloads.scaled(workloads.WORKLOADS["tiny"], V=768, lengths="uniform:20:90", seed=61)
    b = _cuda(workloads.make_batch(w, device="cpu"))
    step = ais.AisStep(b.T, w.d, w.V, w.P, w.G, w.block)
    offs, rew = b.seq_offsets.cuda(), b.rewards.cuda()
    step.forward(b.H, b.W, b.tokens, b.mask)
    step.diagnose(b.mask, offs, rew)
    torch.cuda.synchronize()
    fused = (step.read_diag(), step.rho.clone(), step.w_tilde.clone(), step.adv.clone())
    step.rho.zero_(); step.w_tilde.zero_(); step.diag.zero_()
    ais.diag_moments(step.shape, step.params, step.lp_train, step.lp_roll, b.mask, offs, rew, step.adv, step.n_valid_seq,
                     step.moments, step.workspace)
    ais.diag_finalize(step.shape, step.params, step.moments, step.lp_train, step.lp_roll, b.mask, step.rho, step.w_tilde, step.diag)
    torch.cuda.synchronize()
    assert step.read_diag() == fused[0]
    assert torch.equal(step.rho, fused[1]) and torch.equal(step.w_tilde, fused[2]) and torch.equal(step.adv, fused[3])
    assert float(step.moments[0]) == fused[0]["n_valid"] and float(step.moments[10]) == 0.0


def test_two_prompt_shards_reproduce_the_global_batch():
    import paper_2605_13907_b200 as ais
    w = workloads.scaled(workloads.WORKLOADS["tiny"], d=256, V=1024, P=4, G=4, lengths="uniform:20:100", seed=62)
    b = workloads.make_batch(w, device="cpu")
    a = workloads.to_numpy(b)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block)
    world = 2
    W = b.W.cuda()
    shards = []
    for rank in range(world):
        prompts = adist.shard_prompts(w.P, world, rank)
        r0, r1, loffs = adist.shard_rows(b.seq_offsets.numpy(), w.G, prompts)
        st = ais.AisStep(r1 - r0, w.d, w.V, len(prompts), w.G, w.block, P_total=w.P)
        H, tok, msk = b.H[r0:r1].cuda(), b.tokens[r0:r1].cuda(), b.mask[r0:r1].cuda()
        offs = torch.tensor(loffs, dtype=torch.int32, device="cuda")
        rew = b.rewards[prompts.start * w.G:prompts.stop * w.G].cuda()
        st.forward(H, W, tok, msk)
        ais.diag_moments(st.shape, st.params, st.lp_train, st.lp_roll, msk, offs, rew, st.adv, st.n_valid_seq, st.moments,
                         st.workspace)
        shards.append((st, H, tok, msk, offs, r0, r1))
    total = shards[0][0].moments + shards[1][0].moments             # what the all-reduce leaves on every rank
    dH = torch.empty(b.T, w.d, dtype=torch.bfloat16)
    loss = 0.0
    for st, H, tok, msk, offs, r0, r1 in shards:
        st.moments.copy_(total)
        ais.diag_finalize(st.shape, st.params, st.moments, st.lp_train, st.lp_roll, msk, st.rho, st.w_tilde, st.diag)
        st.backward(H, W, tok, msk, offs)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        d = st.read_diag()
        assert abs(d["alpha"] - ref["diag"]["alpha"]) <= 1e-3 and d["n_valid"] == ref["diag"]["n_valid"]
        dH[r0:r1] = st.dH[:r1 - r0].cpu()
        loss += float(st.loss.item())
        assert np.max(np.abs(st.w_tilde[:r1 - r0].cpu().numpy() - ref["w_tilde"][r0:r1])) <= 1e-4
    assert abs(loss - ref["loss"]) <= 1e-3 * max(1.0, abs(ref["loss"]))
    got = dH.float().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref["dH"]) <= 1e-2 * np.linalg.norm(ref["dH"])
