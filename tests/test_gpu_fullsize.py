"""GPU parity at the full sizes of the five workloads, in the launch configuration the benchmark times.

The float64 oracle cannot run whole batches of these sizes, so the comparison is staged:
  * FP8 codes and scales: bit-exact on ALL of W and on a seeded sample of H rows;
  * log-probs, ratios and dH rows: on that sample of rows (rows are independent at the LM head), each oracle
    row computed against the whole vocabulary;
  * the reductions (advantages, diagnostics, alpha, w_tilde, loss, c_t): the oracle's float64 reductions run on
    the GPU's full [T] log-prob vectors, so every row takes part in that check.
The oracle's work over W is spread over a spawn-ed process pool in row chunks; the chunks are independent.
"""

import multiprocessing as mp
import os

import numpy as np
import pytest
import torch

import workloads
from oracle import ais as oais
from oracle import e4m3

pytestmark = pytest.mark.gpu

LP_ATOL, RHO_RTOL, ALPHA_ATOL, DH_REL = 1e-2, 2e-2, 1e-3, 1e-2
W_CHUNK = 4096


def _w_chunk_job(args):
    """Oracle work for one chunk of vocabulary rows: quantise, dequantise, logits of the sampled rows."""
    Wc, Hs, Hq, block = args
    qc, sc = e4m3.quantize_blocks(Wc, block)
    Wq = e4m3.dequantize_blocks(qc, sc, block)
    return qc, sc, oais.logits(Hs, Wc), oais.logits(Hq, Wq)


def _sample_rows(batch, n, rng):
    T = batch.T
    offs = batch.seq_offsets.numpy().astype(np.int64)
    rows = {0, T - 1, max(0, T - 2), (T // 128) * 128 - 1 if T >= 128 else 0, min(T - 1, (T // 128) * 128)}
    for s in rng.choice(len(offs) - 1, size=min(len(offs) - 1, 24), replace=False):
        lo, hi = offs[s], offs[s + 1]
        if hi > lo:
            rows.update(int(x) for x in rng.integers(lo, hi, 3))
    while len(rows) < n:
        rows.add(int(rng.integers(0, T)))
    return np.array(sorted(rows))[:n]


@pytest.mark.parametrize("name", ["qwen3_8b", "llada_8b", "long_cot", "large_vocab"])
def test_fullsize_sampled_parity(name):
    import paper_2605_13907_b200 as ais
    w = workloads.WORKLOADS[name]
    ctx = mp.get_context("spawn")
    pool = ctx.Pool(max(1, min(16, len(os.sched_getaffinity(0)))))
    try:
        batch = workloads.make_batch(w, device="cuda")
        T = batch.T
        params = ais.default_params(vocab_chunk=w.vocab_chunk)
        step = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block, params=params, workspace_bytes_cap=48 << 30)
        offs_d, rew_d = batch.seq_offsets.cuda(), batch.rewards.cuda()
        step.step(batch.H, batch.W, batch.tokens, batch.mask, offs_d, rew_d)
        torch.cuda.synchronize()
        assert int(step.status.item()) == 0

        rng = np.random.default_rng(w.seed + 17)
        rows = _sample_rows(batch, 160, rng)
        a = workloads.to_numpy(batch, rows=rows)
        Hs, tok_s, msk_s = a["H"], a["tokens"], a["mask"]
        valid_s = msk_s.astype(bool)

        # ---- H codes / scales on the sample
        qHs, sHs = e4m3.quantize_blocks(Hs, w.block)
        idx = torch.as_tensor(rows, device="cuda")
        assert np.array_equal(step.qH[idx].cpu().numpy(), qHs)
        assert np.array_equal(step.sH[:, idx].cpu().numpy().T.view(np.uint32), sHs.view(np.uint32))
        Hq = e4m3.dequantize_blocks(qHs, sHs, w.block)

        # ---- all of W through the oracle, chunk by chunk; logits of the sampled rows
        Wf = a["W"]
        jobs = [(Wf[v0:v0 + W_CHUNK], Hs, Hq, w.block) for v0 in range(0, w.V, W_CHUNK)]
        z_t = np.empty((len(rows), w.V))
        z_r = np.empty((len(rows), w.V))
        for j, (qc, sc, zt, zr) in enumerate(pool.imap(_w_chunk_job, jobs)):
            v0 = j * W_CHUNK
            v1 = min(v0 + W_CHUNK, w.V)
            assert np.array_equal(step.qW[v0:v1].cpu().numpy(), qc), f"W codes differ in rows {v0}..{v1}"
            assert np.array_equal(step.sW[:, v0:v1].cpu().numpy().T.view(np.uint32), sc.view(np.uint32))
            z_t[:, v0:v1] = zt
            z_r[:, v0:v1] = zr
        lp_t, lse_t = oais.log_softmax_gather(z_t, tok_s, msk_s)
        lp_r, _ = oais.log_softmax_gather(z_r, tok_s, msk_s)
        g_lp_t = step.lp_train[idx].cpu().numpy().astype(np.float64)
        g_lp_r = step.lp_roll[idx].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(g_lp_t - lp_t)) <= LP_ATOL
        assert np.max(np.abs(g_lp_r - lp_r)) <= LP_ATOL
        assert np.max(np.abs(step.lse_train[idx].cpu().numpy() - lse_t)) <= LP_ATOL
        _, rho, _ = oais.ratios(lp_t, lp_r, msk_s, 5.0)
        g_rho = step.rho[idx].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(g_rho - rho) / rho) <= RHO_RTOL
        assert np.all(g_lp_t[~valid_s] == 0) and np.all(g_rho[~valid_s] == 1)

        # ---- reductions on the full vectors
        full_lt = step.lp_train[:T].cpu().numpy().astype(np.float64)
        full_lr = step.lp_roll[:T].cpu().numpy().astype(np.float64)
        mask = batch.mask.cpu().numpy()
        offs = batch.seq_offsets.numpy().astype(np.int64)
        adv = oais.advantages(batch.rewards.numpy(), w.G)
        sid = oais.seq_ids(offs, T)
        diag = oais.diagnostics(full_lt, full_lr, mask, adv[sid], oais.Params())
        d = step.read_diag()
        assert abs(d["alpha"] - diag["alpha"]) <= ALPHA_ATOL
        for k in ("n_valid", "alpha_ess", "d_bar", "alpha_mis", "delta_sigma", "alpha_var", "ess_ratio"):
            assert d[k] == pytest.approx(diag[k], rel=1e-6, abs=1e-9), k
        assert 1e-3 < d["d_bar"] < 0.3                             # FP8 perturbation in the expected band
        assert np.allclose(step.adv.cpu().numpy(), adv, atol=1e-6)
        _, _, wbar = oais.ratios(full_lt, full_lr, mask, 5.0)
        w_tilde = oais.rectify(wbar, diag["alpha"], mask)
        assert np.max(np.abs(step.w_tilde[:T].cpu().numpy() - w_tilde)) <= 1e-4
        loss, c = oais.loss_and_coeff(full_lt, full_lt, mask, offs, adv, w_tilde, w.P, w.G, 0.2)
        assert abs(float(step.loss.item()) - loss) <= 1e-4 * max(1.0, abs(loss))

        # ---- dH on the sampled rows
        dH_ref = oais.grad_hidden(Hs, Wf, tok_s, c[rows])
        dH = step.dH[idx].float().cpu().numpy().astype(np.float64)
        nz = np.linalg.norm(dH_ref, axis=1) > 0
        assert np.linalg.norm(dH - dH_ref) <= DH_REL * np.linalg.norm(dH_ref)
        assert np.all(dH[~valid_s] == 0)
        if nz.any():      # row by row as well, so that one bad row cannot hide in the norm of the others
            rel = np.linalg.norm((dH - dH_ref)[nz], axis=1) / np.linalg.norm(dH_ref[nz], axis=1)
            assert rel.max() <= 2 * DH_REL

        # ---- dW at full size: two identities that hold at any size.  The oracle cannot form dW here (it needs the
        # softmax of every row), so: columns of dW sum to zero over the vocabulary (rows of softmax - onehot do), and
        # <dW, W> = sum_t g_t . z_t = <dH, H> ties dW to the dH that was checked row by row above.
        if name in ("qwen3_8b", "llada_8b"):
            dW = torch.empty(w.V, w.d, dtype=torch.float32, device="cuda")
            step.backward(batch.H, batch.W, batch.tokens, batch.mask, offs_d, dW=dW)
            torch.cuda.synchronize()
            assert int(step.status.item()) == 0
            norm = float(dW.double().norm())
            assert norm > 0 and float(dW.double().sum(dim=0).norm()) <= 2e-2 * norm
            ip_w = float((dW.double() * batch.W.double()).sum())
            ip_h = float((step.dH[:T].double() * batch.H.double()).sum())
            assert abs(ip_w - ip_h) <= 1e-2 * max(abs(ip_h), 1e-12)
    finally:
        pool.terminate()
        pool.join()
