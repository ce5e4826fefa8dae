"""Row compaction for scattered masks (masked-diffusion batches): packing the valid rows, running the path on the
packed batch and scattering back gives the same results as the oracle on the full batch (GPU)."""

import numpy as np
import pytest
import torch

import workloads
from oracle import ais as oais

pytestmark = pytest.mark.gpu


def test_compacted_path_matches_oracle_and_direct_run():
    import paper_2605_13907_b200 as ais
    w = workloads.scaled(workloads.WORKLOADS["tiny"], d=256, V=1024, P=2, G=4, lengths="uniform:60:200", mask_mode="llada", seed=95)
    b = workloads.make_batch(w, device="cpu")
    lo, hi = int(b.seq_offsets[5]), int(b.seq_offsets[6])
    b.mask[lo:hi] = 0                                              # one sequence without any valid row
    a = workloads.to_numpy(b)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block)
    H, W, tok, msk = b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda()
    offs, rew = b.seq_offsets.cuda(), b.rewards.cuda()
    T, N = b.T, int(b.mask.sum())

    rc = ais.RowCompaction(msk, offs, n_packed=N)
    torch.cuda.synchronize()
    # index: exactly the valid rows, in order; offsets: exclusive scan of the per-sequence counts
    want = np.nonzero(a["mask"])[0]
    assert np.array_equal(rc.row_index[:N].cpu().numpy(), want)
    counts = np.array([a["mask"][a["seq_offsets"][s]:a["seq_offsets"][s + 1]].sum() for s in range(w.S)])
    assert np.array_equal(rc.n_valid_seq.cpu().numpy(), counts)
    assert np.array_equal(rc.packed_offsets.cpu().numpy(), np.concatenate([[0], np.cumsum(counts)]))
    assert ais.RowCompaction(msk, offs).n == N                       # read back from the device

    Hp, tokp = rc.gather_rows(H), rc.gather(tok)
    assert torch.equal(Hp[:N], H[torch.as_tensor(want, device="cuda")])
    ones = torch.ones(N, dtype=torch.uint8, device="cuda")
    step = ais.AisStep(N, w.d, w.V, w.P, w.G, w.block)
    step.step(Hp, W, tokp, ones, rc.packed_offsets, rew)
    dH = rc.scatter_rows(step.dH[:N], torch.empty(T, w.d, dtype=torch.bfloat16, device="cuda"))
    lp_t, lp_r = rc.scatter(step.lp_train[:N]), rc.scatter(step.lp_roll[:N])
    rho, wt = rc.scatter(step.rho[:N], fill=1.0), rc.scatter(step.w_tilde[:N], fill=1.0)
    torch.cuda.synchronize()
    assert int(step.status.item()) == 0
    valid = a["mask"].astype(bool)
    assert np.max(np.abs(lp_t.cpu().numpy() - ref["lp_train"])) <= 1e-2
    assert np.max(np.abs(lp_r.cpu().numpy() - ref["lp_roll"])) <= 1e-2
    assert np.max(np.abs(rho.cpu().numpy() - ref["rho"]) / ref["rho"]) <= 2e-2
    assert np.all(lp_t.cpu().numpy()[~valid] == 0) and np.all(rho.cpu().numpy()[~valid] == 1) and np.all(wt.cpu().numpy()[~valid] == 1)
    d = step.read_diag()
    assert abs(d["alpha"] - ref["diag"]["alpha"]) <= 1e-3 and d["n_valid"] == N
    assert abs(float(step.loss.item()) - ref["loss"]) <= 1e-3 * max(1.0, abs(ref["loss"]))
    got = dH.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref["dH"]) <= 1e-2 * np.linalg.norm(ref["dH"])
    assert np.all(got[~valid] == 0)

    # the direct run on the full batch with its mask agrees with the packed one
    direct = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block)
    direct.step(H, W, tok, msk, offs, rew)
    torch.cuda.synchronize()
    assert float((direct.lp_train[:T] - lp_t).abs().max()) <= 1e-5
    assert abs(direct.read_diag()["alpha"] - d["alpha"]) <= 1e-6


def test_compaction_argument_errors():
    import paper_2605_13907_b200 as ais
    msk = torch.ones(64, dtype=torch.uint8, device="cuda")
    offs = torch.tensor([0, 64], dtype=torch.int32, device="cuda")
    rc = ais.RowCompaction(msk, offs, n_packed=64)
    src = torch.zeros(64, 24, dtype=torch.bfloat16, device="cuda")   # 48-byte rows: multiple of 16, fine
    assert rc.gather_rows(src).shape == (64, 24)
    bad = torch.zeros(64, 20, dtype=torch.bfloat16, device="cuda")   # 40-byte rows: refused
    with pytest.raises(ais.AisError):
        rc.gather_rows(bad)
