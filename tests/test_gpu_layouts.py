"""Layouts of the same batch must not change the result: sequences packed back to back against the same sequences
padded to a common length with masked rows, and the batch reductions on vectors that do not start on a 16-byte
boundary (the kernels then read row by row instead of four rows per load) and whose length is not a multiple of 4."""

import ctypes

import numpy as np
import pytest
import torch

import workloads
from oracle import ais as oais

pytestmark = pytest.mark.gpu


def test_padded_sequences_equal_packed_sequences():
    import paper_2605_13907_b200 as ais
    w = workloads.scaled(workloads.WORKLOADS["tiny"], d=256, V=1280, P=3, G=4, lengths="uniform:30:200", seed=71)
    b = workloads.make_batch(w, device="cpu")
    offs = b.seq_offsets.numpy().astype(np.int64)
    S, lens = w.P * w.G, np.diff(offs)
    L = int(lens.max()) + 7                                   # padded length, not a multiple of anything
    g = torch.Generator().manual_seed(3)
    Hp = torch.randn(S * L, w.d, generator=g).to(torch.bfloat16)        # padding rows hold arbitrary hidden states
    tokp = torch.randint(0, w.V, (S * L,), generator=g, dtype=torch.int32)
    mskp = torch.zeros(S * L, dtype=torch.uint8)
    rows = np.concatenate([s * L + np.arange(lens[s]) for s in range(S)])   # where the packed rows sit in the padded batch
    Hp[rows] = b.H
    tokp[rows] = b.tokens
    mskp[rows] = b.mask
    offp = torch.arange(0, S * L + 1, L, dtype=torch.int32)

    W = b.W.cuda()
    rew = b.rewards.cuda()
    packed = ais.AisStep(b.T, w.d, w.V, w.P, w.G, w.block)
    packed.step(b.H.cuda(), W, b.tokens.cuda(), b.mask.cuda(), b.seq_offsets.cuda(), rew)
    padded = ais.AisStep(S * L, w.d, w.V, w.P, w.G, w.block)
    padded.step(Hp.cuda(), W, tokp.cuda(), mskp.cuda(), offp.cuda(), rew)
    torch.cuda.synchronize()
    assert int(packed.status.item()) == 0 and int(padded.status.item()) == 0

    r = torch.as_tensor(rows)
    # a row's logits do not depend on its neighbours: the per-row results are the same bits
    for name in ("lp_train", "lse_train", "lp_roll", "rho"):
        assert torch.equal(getattr(packed, name)[:b.T].cpu(), getattr(padded, name).cpu()[r]), name
    dp, dq = packed.read_diag(), padded.read_diag()
    assert dp["n_valid"] == dq["n_valid"] == float(b.mask.sum())
    for k in ("alpha", "d_bar", "cv2", "ess", "delta_sigma", "loss"):
        assert abs(dp[k] - dq[k]) <= 1e-6 * max(1.0, abs(dp[k])), k
    assert torch.equal(packed.n_valid_seq.cpu(), padded.n_valid_seq.cpu())
    dH_packed = packed.dH[:b.T].float().cpu()
    dH_padded = padded.dH.float().cpu()
    assert float((dH_packed - dH_padded[r]).norm()) <= 1e-3 * float(dH_packed.norm())      # alpha differs in the last bits
    pad = torch.ones(S * L, dtype=torch.bool)
    pad[r] = False
    assert torch.all(dH_padded[pad] == 0) and torch.all(padded.lp_train.cpu()[pad] == 0) and torch.all(padded.rho.cpu()[pad] == 1)
    # and both agree with the oracle on the packed batch
    a = workloads.to_numpy(b)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block)
    assert abs(dq["alpha"] - ref["diag"]["alpha"]) <= 1e-3
    assert np.linalg.norm(dH_padded[r].numpy().astype(np.float64) - ref["dH"]) <= 1e-2 * np.linalg.norm(ref["dH"])


@pytest.mark.parametrize("T,shift,S", [(1, 0, 6), (3, 1, 6), (1027, 0, 6), (1027, 1, 6), (4101, 3, 6), (4101, 0, 6),
                                       (5 * 2048 + 77, 0, 1600), (3 * 2048, 0, 8), (20 * 2048 + 1, 0, 400)])
def test_batch_reductions_on_unaligned_and_ragged_vectors(T, shift, S):
    """S = 6: a few sequences with boundaries anywhere.  Larger S on aligned storage: the kernel that stages 2048-row tiles
    in shared memory, with sequences of a few rows (several boundaries inside one thread's eight rows), empty sequences,
    masked stretches longer than a tile and a ragged tail."""
    import paper_2605_13907_b200 as ais
    rng = np.random.default_rng(100 + T + shift + S)
    G = 2
    P = S // G
    # sequence boundaries anywhere, some of the sequences empty
    cuts = np.sort(rng.integers(0, T + 1, S - 1))
    cuts[1] = cuts[0]
    cuts[-1] = T
    if S > 100:
        cuts[S // 2:S // 2 + 5] = cuts[S // 2]              # a run of empty sequences in the middle
    offs = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    lp_t = -rng.uniform(0.1, 6.0, T).astype(np.float32)
    lp_r = (lp_t + rng.normal(0, 0.3, T)).astype(np.float32)
    mask = (rng.random(T) < 0.7).astype(np.uint8)
    if T > 3 * 2048:
        mask[2048 - 100:2 * 2048 + 300] = 0                 # more than one whole tile without a valid row
        mask[T // 2] = 7                                     # any non-zero byte counts as valid
        lp_t[2048:2048 + 8] = np.float32(-np.inf)            # masked rows may hold anything
        lp_r[2048 + 8:2048 + 16] = np.float32(np.nan)
    rew = (rng.random(S) < 0.5).astype(np.float32)
    params = ais.default_params()
    op = oais.Params()
    ref_adv = oais.advantages(rew.astype(np.float64), G)
    ref_diag = oais.diagnostics(lp_t, lp_r, mask, ref_adv[oais.seq_ids(offs, T)], op)
    _, ref_rho, ref_wbar = oais.ratios(lp_t, lp_r, mask, op.C)
    ref_wt = oais.rectify(ref_wbar, ref_diag["alpha"], mask)

    def shifted(x):                                          # same values, storage starting `shift` elements later
        buf = torch.empty(x.size + 8, dtype=torch.from_numpy(x).dtype, device="cuda")
        v = buf[shift:shift + x.size]
        v.copy_(torch.from_numpy(x))
        return v

    shape = ais.make_shape(T, 128, 1024, P, G, 128)
    ws = torch.empty(ais.workspace_min_bytes(shape, params), dtype=torch.uint8, device="cuda")
    d_lp_t, d_lp_r, d_mask = shifted(lp_t), shifted(lp_r), shifted(mask)
    adv = torch.empty(S, device="cuda")
    nseq = torch.full((S,), -1, dtype=torch.int32, device="cuda")
    rho, wt = shifted(np.zeros(T, np.float32)), shifted(np.zeros(T, np.float32))
    diag = torch.zeros(32, dtype=torch.float64, device="cuda")
    ais.diagnostics(shape, params, d_lp_t, d_lp_r, d_mask, torch.from_numpy(offs).cuda(), torch.from_numpy(rew).cuda(), adv, nseq,
                    rho, wt, diag, ws)
    torch.cuda.synchronize()
    d = ais.Diag.from_buffer_copy(diag.cpu().numpy().tobytes()[:ctypes.sizeof(ais.Diag)]).as_dict()
    valid = mask.astype(bool)
    counts = np.array([(mask[offs[s]:offs[s + 1]] != 0).sum() for s in range(S)], np.int32)
    assert np.array_equal(nseq.cpu().numpy(), counts)
    assert d["n_valid"] == float(valid.sum())
    for k in ("alpha", "alpha_ess", "alpha_mis", "alpha_var", "d_bar", "cv2", "delta_sigma", "mean_abs_dp", "kl_k1"):
        assert abs(d[k] - ref_diag[k]) <= 1e-4 * max(1.0, abs(ref_diag[k])), (k, d[k], ref_diag[k])
    assert np.allclose(adv.cpu().numpy(), ref_adv, atol=1e-6)
    got_rho, got_wt = rho.cpu().numpy(), wt.cpu().numpy()
    assert np.allclose(got_rho[valid], ref_rho[valid], rtol=1e-5) and np.all(got_rho[~valid] == 1)
    assert np.allclose(got_wt[valid], ref_wt[valid], rtol=1e-4, atol=1e-5) and np.all(got_wt[~valid] == 1)


@pytest.mark.parametrize("T,shift", [(3 * 2048 + 77, 0), (1027, 1), (1, 0)])
def test_small_but_non_zero_variance_is_kept(T, shift):
    """Every valid row carries the same advantage (the other response of each prompt has no valid row) and a weight of
    1 +- 1e-4: std(A) is exactly 0 and std(A w) is 0.5e-4, which the eps of the variance-amplification ratio turns into
    Delta-sigma = 50, so alpha is 0 (Eq. alpha-var).  Sums of squares rounded to fp32 lose this variance (1e-8 of the
    mean square); the kernels' shifted sums must not.  T = 1 is the case of one valid row, where every variance is 0."""
    import paper_2605_13907_b200 as ais
    rng = np.random.default_rng(7 + T)
    S, G = 4, 2
    cuts = np.sort(rng.integers(0, T + 1, S - 1))
    offs = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    lp_t = -rng.uniform(0.5, 4.0, T).astype(np.float32)
    lp_r = (lp_t.astype(np.float64) - 1e-4 * rng.choice([-1.0, 1.0], T)).astype(np.float32)
    mask = np.zeros(T, np.uint8)
    for s in (0, 2):
        mask[offs[s]:offs[s + 1]] = (rng.random(offs[s + 1] - offs[s]) < 0.8)
    if T == 1:
        offs = np.array([0, 1, 1, 1, 1], np.int32)
        mask[:] = 1
    rew = np.array([1, 0, 1, 0], np.float32)
    op = oais.Params()
    ref_adv = oais.advantages(rew.astype(np.float64), G)
    ref = oais.diagnostics(lp_t, lp_r, mask, ref_adv[oais.seq_ids(offs, T)], op)
    if T > 1:
        assert ref["std_A"] == 0.0 and 20 < ref["delta_sigma"] < 80 and ref["alpha"] == 0.0 and ref["alpha_ess"] > 0.99

    def shifted(x):
        buf = torch.empty(x.size + 8, dtype=torch.from_numpy(x).dtype, device="cuda")
        v = buf[shift:shift + x.size]
        v.copy_(torch.from_numpy(x))
        return v

    params = ais.default_params()
    shape = ais.make_shape(T, 128, 1024, S // G, G, 128)
    ws = torch.empty(ais.workspace_min_bytes(shape, params), dtype=torch.uint8, device="cuda")
    adv = torch.empty(S, device="cuda")
    nseq = torch.zeros(S, dtype=torch.int32, device="cuda")
    rho, wt = torch.zeros(T, device="cuda"), torch.zeros(T, device="cuda")
    diag = torch.zeros(32, dtype=torch.float64, device="cuda")
    ais.diagnostics(shape, params, shifted(lp_t), shifted(lp_r), shifted(mask), torch.from_numpy(offs).cuda(),
                    torch.from_numpy(rew).cuda(), adv, nseq, rho, wt, diag, ws)
    torch.cuda.synchronize()
    d = ais.Diag.from_buffer_copy(diag.cpu().numpy().tobytes()[:ctypes.sizeof(ais.Diag)]).as_dict()
    assert d["n_valid"] == ref["n_valid"] and d["std_A"] == 0.0
    assert abs(d["alpha"] - ref["alpha"]) <= 1e-3
    for k in ("cv2", "std_Aw", "delta_sigma", "alpha_var", "alpha_ess"):
        assert d[k] == pytest.approx(ref[k], rel=1e-5, abs=1e-15), (k, d[k], ref[k])


def test_sequence_level_weights_on_gpu():
    """params.seq_level_weights: every valid row carries min(prod_t rho_t, C) of its sequence (Eq. is-weight).  The
    fused call and the split pair agree with the oracle's sequence-level variant; d_bar and rho stay per token."""
    import paper_2605_13907_b200 as ais
    w = workloads.scaled(workloads.WORKLOADS["tiny"], d=256, V=1280, P=3, G=4, lengths="uniform:3:70", seed=77)
    b = workloads.make_batch(w, device="cpu")
    a = workloads.to_numpy(b)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block,
                         params=oais.Params(seq_level=True))
    tok = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block,
                         want_grad=False)
    assert abs(ref["diag"]["cv2"] - tok["diag"]["cv2"]) > 1e-4          # the two variants really differ on this batch
    params = ais.default_params(seq_level_weights=1)
    step = ais.AisStep(b.T, w.d, w.V, w.P, w.G, w.block, params=params)
    offs, rew = b.seq_offsets.cuda(), b.rewards.cuda()
    H, W, tokens, mask = b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda()
    step.step(H, W, tokens, mask, offs, rew)
    torch.cuda.synchronize()
    d = step.read_diag()
    T = b.T
    for k in ("alpha", "alpha_ess", "alpha_var", "cv2", "d_bar", "delta_sigma"):
        assert abs(d[k] - ref["diag"][k]) <= 1e-3 * max(1.0, abs(ref["diag"][k])), (k, d[k], ref["diag"][k])
    assert np.max(np.abs(step.w_tilde.cpu().numpy()[:T] - ref["w_tilde"])) <= 2e-2 * np.max(ref["w_tilde"])
    assert np.max(np.abs(step.rho.cpu().numpy()[:T] - ref["rho"]) / ref["rho"]) <= 2e-2
    dH = step.dH.float().cpu().numpy()[:T].astype(np.float64)
    assert np.linalg.norm(dH - ref["dH"]) <= 1e-2 * np.linalg.norm(ref["dH"])
    fused = (d, step.w_tilde.clone())
    # the split pair gives the same bits
    step.w_tilde.zero_(); step.diag.zero_()
    ais.diag_moments(step.shape, step.params, step.lp_train, step.lp_roll, mask, offs, rew, step.adv, step.n_valid_seq,
                     step.moments, step.workspace, seq_logw=step.seq_logw)
    ais.diag_finalize(step.shape, step.params, step.moments, step.lp_train, step.lp_roll, mask, step.rho, step.w_tilde, step.diag,
                      seq_offsets=offs, seq_logw=step.seq_logw)
    torch.cuda.synchronize()
    d2 = step.read_diag()
    for k in ("alpha", "cv2", "d_bar", "delta_sigma", "n_valid"):
        assert d2[k] == fused[0][k], k
    assert torch.equal(step.w_tilde, fused[1])


def test_sequence_level_reductions_over_several_tiles():
    """The sequence-level variant of the batch reductions on a batch long enough for the kernel that stages 2048-row
    tiles in shared memory (the end-to-end test of the variant above is smaller than one tile): split pair
    ais_diag_moments / ais_diag_finalize against the oracle's sequence-level weights."""
    import paper_2605_13907_b200 as ais
    rng = np.random.default_rng(4242)
    T, S, G = 4 * 2048 + 321, 60, 4
    P = S // G
    cuts = np.sort(rng.integers(0, T + 1, S - 1))
    cuts[7] = cuts[6]                                         # an empty sequence
    offs = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    lp_t = -rng.uniform(0.1, 6.0, T).astype(np.float32)
    lp_r = (lp_t + rng.normal(0, 0.02, T)).astype(np.float32)  # small per-token gaps: the sequence products stay moderate
    mask = (rng.random(T) < 0.8).astype(np.uint8)
    rew = (rng.random(S) < 0.5).astype(np.float32)
    op = oais.Params(seq_level=True)
    ref_adv = oais.advantages(rew.astype(np.float64), G)
    ref_logw, ref_wbar = oais.ratios_sequence(lp_t, lp_r, mask, offs, op.C)
    ref = oais.diagnostics(lp_t, lp_r, mask, ref_adv[oais.seq_ids(offs, T)], op, wbar_rows=ref_wbar)
    ref_wt = oais.rectify(ref_wbar, ref["alpha"], mask)

    params = ais.default_params(seq_level_weights=1)
    shape = ais.make_shape(T, 128, 1024, P, G, 128)
    ws = torch.empty(ais.workspace_min_bytes(shape, params), dtype=torch.uint8, device="cuda")
    c = lambda x: torch.from_numpy(x).cuda()
    d_lp_t, d_lp_r, d_mask, d_offs = c(lp_t), c(lp_r), c(mask), c(offs)
    adv = torch.empty(S, device="cuda")
    nseq = torch.full((S,), -1, dtype=torch.int32, device="cuda")
    logw = torch.zeros(S, device="cuda")
    moments = torch.zeros(16, dtype=torch.float64, device="cuda")
    rho, wt = torch.zeros(T, device="cuda"), torch.zeros(T, device="cuda")
    diag = torch.zeros(32, dtype=torch.float64, device="cuda")
    ais.diag_moments(shape, params, d_lp_t, d_lp_r, d_mask, d_offs, c(rew), adv, nseq, moments, ws, seq_logw=logw)
    ais.diag_finalize(shape, params, moments, d_lp_t, d_lp_r, d_mask, rho, wt, diag, seq_offsets=d_offs, seq_logw=logw)
    torch.cuda.synchronize()
    d = ais.Diag.from_buffer_copy(diag.cpu().numpy().tobytes()[:ctypes.sizeof(ais.Diag)]).as_dict()
    valid = mask.astype(bool)
    counts = np.array([(mask[offs[s]:offs[s + 1]] != 0).sum() for s in range(S)], np.int32)
    assert np.array_equal(nseq.cpu().numpy(), counts)
    assert np.allclose(logw.cpu().numpy(), ref_logw, rtol=1e-5, atol=1e-5)
    assert d["n_valid"] == float(valid.sum())
    for k in ("alpha", "alpha_ess", "alpha_mis", "alpha_var", "d_bar", "cv2", "delta_sigma", "mean_abs_dp", "kl_k1"):
        assert abs(d[k] - ref[k]) <= 1e-4 * max(1.0, abs(ref[k])), (k, d[k], ref[k])
    got_wt = wt.cpu().numpy()
    assert np.allclose(got_wt[valid], ref_wt[valid], rtol=1e-4, atol=1e-5) and np.all(got_wt[~valid] == 1)


@pytest.mark.parametrize("case", ["ragged", "block32"])
def test_head_stored_d_by_v_gives_the_same_results(case):
    """ais_shape.w_layout = AIS_W_DV: the LM head as [d, V] (the form in which the paper writes it) with a padded row
    stride.  Codes and scales of the column-block quantiser equal the row quantiser's on the transposed matrix, the
    log-probs of both passes are the same bits as with the [V, d] head, dH and dW (which comes out [d, V]) agree with
    the oracle."""
    import paper_2605_13907_b200 as ais
    base = workloads.WORKLOADS["tiny"]
    w = workloads.scaled(base, d=384, V=1336, P=3, G=4, lengths="uniform:5:90", seed=21) if case == "ragged" else \
        workloads.scaled(base, d=256, V=2048, P=2, G=4, block=32, lengths="uniform:40:120", seed=22)
    b = workloads.make_batch(w, device="cpu")
    a = workloads.to_numpy(b)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block)
    H, W, tok, msk = b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda()
    offs, rew = b.seq_offsets.cuda(), b.rewards.cuda()
    T = b.T
    ldw = w.V + 24                                            # padded row stride of the [d, V] head
    Wbig = torch.randn(w.d, ldw).to(torch.bfloat16).cuda()
    Wbig[:, :w.V] = W.t()
    Wdv = Wbig[:, :w.V]

    vd = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block)
    dW_vd = torch.zeros(w.V, w.d, dtype=torch.float32, device="cuda")
    vd.forward(H, W, tok, msk)
    vd.diagnose(msk, offs, rew)
    vd.backward(H, W, tok, msk, offs, dW=dW_vd)
    dv = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block, ldw=ldw, w_layout=ais.W_DV)
    dW_dv = torch.full((w.d, w.V), 3.0, dtype=torch.float32, device="cuda")
    dv.forward(H, Wdv, tok, msk)
    dv.diagnose(msk, offs, rew)
    dv.backward(H, Wdv, tok, msk, offs, dW=dW_dv)
    torch.cuda.synchronize()
    assert int(vd.status.item()) == 0 and int(dv.status.item()) == 0
    # quantiser: bit-exact against the oracle (and therefore against the row quantiser)
    assert np.array_equal(dv.qW.cpu().numpy(), ref["qW"])
    assert np.array_equal(dv.sW.cpu().numpy()[:, :w.V].T.view(np.uint32), ref["sW"].view(np.uint32))
    assert torch.equal(dv.qW, vd.qW) and torch.equal(dv.sW[:, :w.V], vd.sW[:, :w.V])
    # log-probs: the same bits whichever way W is stored
    for name in ("lp_train", "lse_train", "lp_roll"):
        assert torch.equal(getattr(dv, name)[:T], getattr(vd, name)[:T]), name
    assert np.max(np.abs(dv.lp_train[:T].cpu().numpy() - ref["lp_train"])) <= 1e-2
    assert np.max(np.abs(dv.lp_roll[:T].cpu().numpy() - ref["lp_roll"])) <= 1e-2
    assert dv.read_diag()["alpha"] == vd.read_diag()["alpha"]
    dH = dv.dH[:T].float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(dH - ref["dH"]) <= 1e-2 * np.linalg.norm(ref["dH"])
    assert float((dv.dH[:T].float() - vd.dH[:T].float()).norm()) <= 2e-3 * float(vd.dH[:T].float().norm())
    got = dW_dv.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref["dW"].T) <= 1e-2 * np.linalg.norm(ref["dW"])
    assert float((dW_dv - dW_vd.t()).norm()) <= 2e-3 * float(dW_vd.norm())
