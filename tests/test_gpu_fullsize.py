"""GPU parity at the full sizes of the five workloads, in the launch configuration the benchmark times.

The float64 oracle cannot run whole batches of these sizes, so the comparison is staged:
  * FP8 codes and scales: bit-exact on ALL of W and on a seeded sample of H rows;
  * log-probs, ratios and dH rows: on that sample of rows (rows are independent at the LM head), each oracle
    row computed against the whole vocabulary.  The sample holds at least eight rows of every sequence on the
    workloads with up to 128 sequences (4096 rows), and 1024 rows (two per sequence) on the long
    chain-of-thought workload;
  * the reductions (advantages, diagnostics, alpha, w_tilde, loss, c_t): the oracle's float64 reductions run on
    the GPU's full [T] log-prob vectors, so every row takes part in that check.
The oracle's quantiser (elementwise numpy, one core per call) runs over W in a spawn-ed process pool, chunk by
chunk; its matrix products run in this process on the BLAS threads, 1024 sampled rows at a time so that the
[rows, V] float64 logits stay near 2.5 GB.
"""

import multiprocessing as mp
import os

import numpy as np
import pytest
import torch

import row_sampling
import workloads
from oracle import ais as oais
from oracle import e4m3

pytestmark = pytest.mark.gpu

LP_ATOL, RHO_RTOL, ALPHA_ATOL, DH_REL = 1e-2, 2e-2, 1e-3, 1e-2
W_CHUNK = 4096
ROW_GROUP = 1024
SAMPLE = {"qwen3_8b": 4096, "llada_8b": 4096, "long_cot": 1024, "large_vocab": 1024}


def _quantise_chunk(args):
    Wc, block = args
    return e4m3.quantize_blocks(Wc, block)


def _padded_copy(batch, L):
    """The same batch in the padded [S, L] form: sequence s occupies rows s L .. s L + len_s - 1, the tail rows
    are masked and hold other values (they must not matter)."""
    w = batch.workload
    offs = batch.seq_offsets.numpy().astype(np.int64)
    S = len(offs) - 1
    dev = batch.H.device
    g = torch.Generator(device=dev).manual_seed(99)
    H = (torch.randn(S * L, w.d, generator=g, device=dev, dtype=torch.float32) * 3).to(torch.bfloat16)
    tok = torch.randint(0, w.V, (S * L,), generator=g, device=dev, dtype=torch.int32)
    mask = torch.zeros(S * L, dtype=torch.uint8, device=dev)
    index = np.empty(batch.T, dtype=np.int64)                # padded row of every packed row
    for s in range(S):
        n = offs[s + 1] - offs[s]
        H[s * L:s * L + n] = batch.H[offs[s]:offs[s + 1]]
        tok[s * L:s * L + n] = batch.tokens[offs[s]:offs[s + 1]]
        mask[s * L:s * L + n] = batch.mask[offs[s]:offs[s + 1]]
        index[offs[s]:offs[s + 1]] = s * L + np.arange(n)
    poffs = torch.arange(0, S * L + 1, L, dtype=torch.int32)
    return workloads.Batch(w, H, batch.W, tok, mask, poffs, batch.rewards), index


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
        offs = batch.seq_offsets.numpy().astype(np.int64)
        rows = row_sampling.sample_rows(offs, T, SAMPLE[name], rng)
        assert len(rows) >= SAMPLE[name]
        if SAMPLE[name] >= 4096:
            per_seq = row_sampling.rows_per_sequence(rows, offs)
            assert per_seq.min() >= 8, per_seq.min()
        a = workloads.to_numpy(batch, rows=rows)
        Hs, tok_s, msk_s = a["H"], a["tokens"], a["mask"]
        valid_s = msk_s.astype(bool)
        Wf = a["W"]

        # ---- H codes / scales on the sample
        qHs, sHs = e4m3.quantize_blocks(Hs, w.block)
        idx = torch.as_tensor(rows, device="cuda")
        assert np.array_equal(step.qH[idx].cpu().numpy(), qHs)
        assert np.array_equal(step.sH[:, idx].cpu().numpy().T.view(np.uint32), sHs.view(np.uint32))
        Hq = e4m3.dequantize_blocks(qHs, sHs, w.block)

        # ---- all of W through the oracle's quantiser, chunk by chunk: codes and scales bit-exact
        starts = list(range(0, w.V, W_CHUNK))
        qW, sW = [], []
        for v0, (qc, sc) in zip(starts, pool.imap(_quantise_chunk, [(Wf[v0:v0 + W_CHUNK], w.block) for v0 in starts])):
            v1 = min(v0 + W_CHUNK, w.V)
            assert np.array_equal(step.qW[v0:v1].cpu().numpy(), qc), f"W codes differ in rows {v0}..{v1}"
            assert np.array_equal(step.sW[:, v0:v1].cpu().numpy().T.view(np.uint32), sc.view(np.uint32))
            qW.append(qc)
            sW.append(sc)

        # ---- reductions on the full vectors (they give the alpha and the c_t that the sampled dH rows need)
        full_lt = step.lp_train[:T].cpu().numpy().astype(np.float64)
        full_lr = step.lp_roll[:T].cpu().numpy().astype(np.float64)
        mask = batch.mask.cpu().numpy()
        adv = oais.advantages(batch.rewards.numpy(), w.G)
        sid = oais.seq_ids(offs, T)
        diag = oais.diagnostics(full_lt, full_lr, mask, adv[sid], oais.Params())
        d = step.read_diag()
        assert abs(d["alpha"] - diag["alpha"]) <= ALPHA_ATOL
        for k in ("n_valid", "alpha_ess", "d_bar", "alpha_mis", "delta_sigma", "alpha_var", "ess_ratio", "kl_k1", "mean_abs_dp"):
            assert d[k] == pytest.approx(diag[k], rel=1e-5, abs=1e-9), k
        assert 1e-3 < d["d_bar"] < 0.3                             # FP8 perturbation in the expected band
        assert np.allclose(step.adv.cpu().numpy(), adv, atol=1e-6)
        _, _, wbar = oais.ratios(full_lt, full_lr, mask, 5.0)
        w_tilde = oais.rectify(wbar, diag["alpha"], mask)
        assert np.max(np.abs(step.w_tilde[:T].cpu().numpy() - w_tilde)) <= 1e-4
        loss, c = oais.loss_and_coeff(full_lt, full_lt, mask, offs, adv, w_tilde, w.P, w.G, 0.2)
        assert abs(float(step.loss.item()) - loss) <= 1e-4 * max(1.0, abs(loss))

        # ---- log-probs, ratios and dH of the sampled rows, one group of rows at a time
        g_lp_t = step.lp_train[idx].cpu().numpy().astype(np.float64)
        g_lp_r = step.lp_roll[idx].cpu().numpy().astype(np.float64)
        g_lse = step.lse_train[idx].cpu().numpy().astype(np.float64)
        g_rho = step.rho[idx].cpu().numpy().astype(np.float64)
        g_dH = step.dH[idx].float().cpu().numpy().astype(np.float64)
        lp_t_all = np.empty(len(rows))
        lp_r_all = np.empty(len(rows))
        dH_all = np.empty((len(rows), w.d))
        for r0 in range(0, len(rows), ROW_GROUP):
            sl = slice(r0, min(r0 + ROW_GROUP, len(rows)))
            n = sl.stop - sl.start
            z_t = np.empty((n, w.V))
            z_r = np.empty((n, w.V))
            for j, v0 in enumerate(starts):
                v1 = min(v0 + W_CHUNK, w.V)
                z_t[:, v0:v1] = oais.logits(Hs[sl], Wf[v0:v1])
                z_r[:, v0:v1] = oais.logits(Hq[sl], e4m3.dequantize_blocks(qW[j], sW[j], w.block))
            lp_t, lse_t = oais.log_softmax_gather(z_t, tok_s[sl], msk_s[sl])
            lp_r, _ = oais.log_softmax_gather(z_r, tok_s[sl], msk_s[sl])
            assert np.max(np.abs(g_lp_t[sl] - lp_t)) <= LP_ATOL
            assert np.max(np.abs(g_lp_r[sl] - lp_r)) <= LP_ATOL
            assert np.max(np.abs(g_lse[sl] - lse_t)) <= LP_ATOL
            _, rho, _ = oais.ratios(lp_t, lp_r, msk_s[sl], 5.0)
            assert np.max(np.abs(g_rho[sl] - rho) / rho) <= RHO_RTOL
            lp_t_all[sl], lp_r_all[sl] = lp_t, lp_r
            gz = oais.logit_gradient(z_t, tok_s[sl], c[rows[sl]])
            dH_ref = np.zeros((n, w.d))
            for v0 in starts:
                v1 = min(v0 + W_CHUNK, w.V)
                dH_ref += gz[:, v0:v1] @ Wf[v0:v1].astype(np.float64)
            dH_all[sl] = dH_ref
        assert np.all(g_lp_t[~valid_s] == 0) and np.all(g_rho[~valid_s] == 1)
        nz = np.linalg.norm(dH_all, axis=1) > 0
        assert np.linalg.norm(g_dH - dH_all) <= DH_REL * np.linalg.norm(dH_all)
        assert np.all(g_dH[~valid_s] == 0)
        if nz.any():      # row by row as well, so that one bad row cannot hide in the norm of the others
            rel = np.linalg.norm((g_dH - dH_all)[nz], axis=1) / np.linalg.norm(dH_all[nz], axis=1)
            assert rel.max() <= DH_REL, rel.max()

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
            del dW

        # ---- the padded [S, 2048] form of the same batch (response lengths with a padding mask): the sampled rows
        # against the oracle values found above, every valid row against the packed run, neutral values in the padding
        if name == "qwen3_8b":
            L = 2048
            pb, index = _padded_copy(batch, L)
            pstep = ais.AisStep(pb.T, w.d, w.V, w.P, w.G, w.block, params=params, workspace_bytes_cap=48 << 30)
            pstep.step(pb.H, pb.W, pb.tokens, pb.mask, pb.seq_offsets.cuda(), rew_d)
            torch.cuda.synchronize()
            assert int(pstep.status.item()) == 0
            pidx = torch.as_tensor(index[rows], device="cuda")
            assert np.max(np.abs(pstep.lp_train[pidx].cpu().numpy() - lp_t_all)) <= LP_ATOL
            assert np.max(np.abs(pstep.lp_roll[pidx].cpu().numpy() - lp_r_all)) <= LP_ATOL
            pd = pstep.read_diag()
            assert pd["n_valid"] == d["n_valid"] and abs(pd["alpha"] - diag["alpha"]) <= ALPHA_ATOL
            for k in ("alpha_ess", "d_bar", "delta_sigma", "ess_ratio"):
                assert pd[k] == pytest.approx(diag[k], rel=1e-5, abs=1e-9), k
            pdH = pstep.dH[pidx].float().cpu().numpy().astype(np.float64)
            assert np.linalg.norm(pdH - dH_all) <= DH_REL * np.linalg.norm(dH_all)
            allidx = torch.as_tensor(index, device="cuda")
            assert float((pstep.lp_train[allidx] - step.lp_train[:T]).abs().max()) <= 1e-5
            assert float((pstep.lp_roll[allidx] - step.lp_roll[:T]).abs().max()) <= 1e-5
            assert float((pstep.w_tilde[allidx] - step.w_tilde[:T]).abs().max()) <= 1e-5
            pad = pb.mask == 0
            assert int(pad.sum()) == pb.T - T
            assert bool((pstep.lp_train[:pb.T][pad] == 0).all()) and bool((pstep.rho[:pb.T][pad] == 1).all())
            assert bool((pstep.w_tilde[:pb.T][pad] == 1).all()) and bool((pstep.dH[:pb.T][pad] == 0).all())
            assert abs(float(pstep.loss.item()) - loss) <= 1e-4 * max(1.0, abs(loss))
            del pstep, pb

        # ---- the same head stored [d, V] (ais_shape.w_layout = AIS_W_DV) at full size: both log-prob vectors must be the
        # same bits as with the [V, d] head that was checked against the oracle above, codes and scales too
        if name == "qwen3_8b":
            Wdv = batch.W.t().contiguous()
            dstep = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block, params=params, workspace_bytes_cap=48 << 30, w_layout=ais.W_DV)
            dstep.step(batch.H, Wdv, batch.tokens, batch.mask, offs_d, rew_d)
            torch.cuda.synchronize()
            assert int(dstep.status.item()) == 0
            assert torch.equal(dstep.qW, step.qW) and torch.equal(dstep.sW[:, :w.V], step.sW[:, :w.V])
            assert torch.equal(dstep.lp_train[:T], step.lp_train[:T]) and torch.equal(dstep.lp_roll[:T], step.lp_roll[:T])
            assert dstep.read_diag()["alpha"] == d["alpha"]
            ddH = dstep.dH[idx].float().cpu().numpy().astype(np.float64)
            assert np.linalg.norm(ddH - dH_all) <= DH_REL * np.linalg.norm(dH_all)
    finally:
        pool.terminate()
        pool.join()
