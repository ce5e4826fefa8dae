"""Data-parallel host logic on CPU: two gloo ranks shard a batch by prompts, all-reduce the moment vector and
arrive at the oracle's global diagnostics (no GPU involved; the moments here are computed by the test itself)."""

import math
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import ais as oais
from paper_2605_13907_b200 import dist as adist


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _problem():
    rng = np.random.default_rng(123)
    P, G = 5, 3
    lengths = rng.integers(3, 20, P * G)
    offs = np.concatenate([[0], np.cumsum(lengths)])
    T = int(offs[-1])
    lp_t = -np.abs(rng.normal(4, 1.5, T))
    lp_r = lp_t + rng.normal(0, 0.05, T)
    mask = (rng.random(T) < 0.85).astype(np.uint8)
    rewards = (rng.random(P * G) < 0.4).astype(np.float64)
    return P, G, offs, lp_t, lp_r, mask, rewards


def _local_moments(lp_t, lp_r, mask, adv_tok, C=5.0):
    """The 12 masked sums, written from their definition in include/ais.h."""
    v = mask.astype(bool)
    d = (lp_t - lp_r)[v]
    w = np.exp(np.minimum(d, math.log(C)))
    A = adv_tok[v]
    m = [v.sum(), w.sum(), (w * w).sum(), np.abs(d).sum(), A.sum(), (A * A).sum(), (A * w).sum(), ((A * w) ** 2).sum(),
         (-d).sum(), np.abs(np.exp(lp_t[v]) - np.exp(lp_r[v])).sum(), 0.0, 0.0]
    return torch.tensor(m, dtype=torch.float64)


def _alpha_from_moments(m, p=oais.Params()):
    N = m[0]
    mu = m[1] / N
    cv2 = (m[2] / N - mu * mu) / (mu * mu)
    a_ess = (1 + cv2) ** -0.5
    a_mis = min(1.0, (m[3] / N) / p.delta)
    sA = math.sqrt(max(m[5] / N - (m[4] / N) ** 2, 0.0))
    sAw = math.sqrt(max(m[7] / N - (m[6] / N) ** 2, 0.0))
    a_var = max(0.0, (sAw / (sA + p.eps) - p.gamma) / p.gamma)
    return min(1.0, max(0.0, a_ess - p.beta_var * a_var)) * a_mis


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        P, G, offs, lp_t, lp_r, mask, rewards = _problem()
        prompts = adist.shard_prompts(P, world, rank)
        r0, r1, local_offs = adist.shard_rows(offs, G, prompts)
        adv = oais.advantages(rewards[prompts.start * G:prompts.stop * G], G)      # groups stay whole on a rank
        sid = oais.seq_ids(np.array(local_offs), r1 - r0)
        m = _local_moments(lp_t[r0:r1], lp_r[r0:r1], mask[r0:r1], adv[sid])
        adist.allreduce_moments(m)
        out[rank] = (m.tolist(), (prompts.start, prompts.stop), (r0, r1))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reach_the_global_alpha():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    P, G, offs, lp_t, lp_r, mask, rewards = _problem()
    adv = oais.advantages(rewards, G)
    sid = oais.seq_ids(offs, len(mask))
    ref = oais.diagnostics(lp_t, lp_r, mask, adv[sid], oais.Params())
    m0, pr0, rows0 = out[0]
    m1, pr1, rows1 = out[1]
    assert m0 == m1                                             # every rank holds the same global sums
    assert pr0[1] == pr1[0] and pr0[0] == 0 and pr1[1] == P and rows0[1] == rows1[0] and rows1[1] == len(mask)
    assert m0[0] == ref["n_valid"]
    assert _alpha_from_moments(m0) == pytest.approx(ref["alpha"], abs=1e-12)
    assert m0[3] / m0[0] == pytest.approx(ref["d_bar"], rel=1e-12)


def test_shard_prompts_partitions_everything():
    for P in (1, 7, 8, 64):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(adist.shard_prompts(P, world, r))
            assert seen == list(range(P))
            sizes = [len(adist.shard_prompts(P, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        adist.shard_prompts(4, 2, 2)


def test_allreduce_is_identity_without_a_group():
    m = torch.arange(12, dtype=torch.float64)
    assert torch.equal(adist.allreduce_moments(m.clone()), m)
    with pytest.raises(TypeError):
        adist.allreduce_moments(torch.zeros(12))
