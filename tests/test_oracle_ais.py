"""Pins for the float64 oracle of the AIS-GRPO path (CPU only).

Each test checks the oracle against something fixed outside it: hand-worked closed forms
(tests/golden/diag_closed_forms.txt), identities and bounds the paper states, brute force on a
tiny vocabulary, exact rational arithmetic, and central finite differences.
"""

import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import ais, e4m3

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
P0 = ais.Params()


def _golden():
    out = {}
    for line in open(os.path.join(GOLDEN, "diag_closed_forms.txt")):
        line = line.split("#")[0].strip()
        if line:
            case, key, val = line.split()
            out[(case, key)] = float(val)
    return out


def _diag_from_w(w, delta=None, A=None, p=P0):
    """Feed chosen weights through the oracle: lp_roll = 0, lp_train = log w (or a given Delta)."""
    w = np.asarray(w, dtype=np.float64)
    d = np.log(w) if delta is None else np.asarray(delta, dtype=np.float64)
    A = np.ones_like(d) if A is None else np.asarray(A, dtype=np.float64)
    return ais.diagnostics(d, np.zeros_like(d), np.ones(len(d), np.uint8), A, p)


# ------------------------------------------------------------------ diagnostics: closed forms
def test_golden_closed_forms():
    g = _golden()
    d = _diag_from_w([1.0, 3.0] * 50)
    for k in ("cv2", "ess_ratio", "alpha_ess"):
        assert d[k] == pytest.approx(g[("two_point", k)], abs=1e-12)
    d = _diag_from_w([1.0, 1.0, 1.0, 5.0] * 25)
    for k in ("cv2", "ess_ratio", "alpha_ess"):
        assert d[k] == pytest.approx(g[("three_to_one", k)], abs=1e-12)
    d = _diag_from_w(None, delta=[0.01, -0.01] * 32)
    assert d["d_bar"] == pytest.approx(g[("half_delta", "d_bar")], abs=1e-15)
    assert d["alpha_mis"] == pytest.approx(g[("half_delta", "alpha_mis")], abs=1e-12)


def test_alpha_ess_identity_and_bounds():
    """sqrt(ESS_ratio) == (1 + CV^2)^(-1/2)  (Eq. alpha-ess); ESS in [1, N]."""
    rng = np.random.default_rng(0)
    for n in (1, 2, 17, 1000):
        w = np.minimum(np.exp(rng.normal(0, 1.0, n)), 5.0)
        d = _diag_from_w(w)
        assert math.sqrt(d["ess_ratio"]) == pytest.approx(d["alpha_ess"], abs=1e-12)
        assert 1.0 - 1e-12 <= d["ess"] <= n + 1e-9
        assert n ** -0.5 - 1e-12 <= d["alpha_ess"] <= 1.0 + 1e-12
        assert 0.0 <= d["alpha"] <= 1.0


def test_constant_weights_and_degenerate_weights():
    d = _diag_from_w([2.5] * 64)
    assert d["cv2"] == pytest.approx(0.0, abs=1e-15) and d["alpha_ess"] == pytest.approx(1.0, abs=1e-15)
    assert d["ess"] == pytest.approx(64.0)
    # one token at the cap, the others vanishing: ESS -> 1
    w = np.full(256, 1e-9)
    w[0] = 5.0
    d = _diag_from_w(w)
    assert d["ess"] == pytest.approx(1.0, abs=1e-6)


def test_truncation_at_C():
    d = _diag_from_w([100.0] * 8 + [1.0] * 8)            # rho = 100 is cut to 5
    assert d["mean_w"] == pytest.approx(3.0)
    delta, rho, wbar = ais.ratios(np.log([100.0, 2.0]), np.zeros(2), np.ones(2), 5.0)
    assert rho == pytest.approx([100.0, 2.0]) and wbar == pytest.approx([5.0, 2.0])
    assert np.isfinite(ais.ratios(np.array([800.0]), np.zeros(1), np.ones(1), 5.0)[2]).all()


def test_alpha_mis_branches():
    assert _diag_from_w(None, delta=[0.0] * 10)["alpha_mis"] == 0.0
    assert _diag_from_w(None, delta=[0.02, -0.02] * 5)["alpha_mis"] == pytest.approx(1.0)
    assert _diag_from_w(None, delta=[0.3, -0.5] * 5)["alpha_mis"] == 1.0
    assert _diag_from_w(None, delta=[0.005] * 10)["alpha_mis"] == pytest.approx(0.25)


def test_alpha_var_branches():
    A = np.array([1.0, -1.0] * 32)
    # constant w_bar = 3: Delta sigma = 3 std/(std+eps) ~ 3 -> alpha_var = (3-1.2)/1.2 = 1.5 -> alpha = 0
    d = _diag_from_w([3.0] * 64, A=A)
    assert d["std_A"] == pytest.approx(1.0)
    assert d["delta_sigma"] == pytest.approx(3.0 / (1.0 + 1e-6), abs=1e-12)
    assert d["alpha_var"] == pytest.approx((3.0 / (1.0 + 1e-6) - 1.2) / 1.2, abs=1e-12)
    assert d["alpha"] == 0.0
    # constant w_bar = 1.1: below the tolerance gamma -> no penalty
    d = _diag_from_w([1.1] * 64, A=A)
    assert d["alpha_var"] == 0.0
    # all advantages zero
    d = _diag_from_w([1.0, 3.0] * 32, A=np.zeros(64))
    assert d["delta_sigma"] == 0.0 and d["alpha_var"] == 0.0


def test_alpha_final_product_form():
    """alpha = clip(alpha_ess - beta alpha_var, 0, 1) * alpha_mis, and it collapses when either gate is 0."""
    rng = np.random.default_rng(1)
    delta = rng.normal(0, 0.004, 500)
    A = rng.choice([-0.3, 0.7], 500)
    d = _diag_from_w(None, delta=delta, A=A)
    exp = min(1, max(0, d["alpha_ess"] - 1.0 * d["alpha_var"])) * d["alpha_mis"]
    assert d["alpha"] == pytest.approx(exp, abs=1e-15)
    assert 0 < d["alpha_mis"] < 1 and 0 < d["alpha"] < 1
    assert _diag_from_w(None, delta=np.zeros(50), A=A[:50])["alpha"] == 0.0
    p = ais.Params(beta_var=2.0)
    d2 = _diag_from_w(None, delta=delta * 300, A=A, p=p)
    assert d2["alpha"] == pytest.approx(min(1, max(0, d2["alpha_ess"] - 2.0 * d2["alpha_var"])) * d2["alpha_mis"])


def test_on_policy_recovery():
    """Rollout == trainer: rho = w_bar = 1 exactly, d_bar = 0, alpha = 0, weight 1 (Proposition 'on-policy recovery')."""
    rng = np.random.default_rng(2)
    lp = -np.abs(rng.normal(5, 2, 100))
    mask = np.ones(100, np.uint8)
    _, rho, wbar = ais.ratios(lp, lp, mask, 5.0)
    assert np.all(rho == 1.0) and np.all(wbar == 1.0)
    d = ais.diagnostics(lp, lp, mask, rng.normal(size=100), P0)
    assert d["d_bar"] == 0.0 and d["alpha"] == 0.0 and d["alpha_ess"] == 1.0
    for a in (0.0, 0.3, 1.0):
        assert np.all(ais.rectify(wbar, a, mask) == 1.0)


def test_rectified_weight_bounds():
    """0 <= 1 - alpha + alpha w_bar <= 1 + alpha (C - 1)  (Proposition 'bounded second moment')."""
    rng = np.random.default_rng(3)
    delta = rng.normal(0, 2.0, 2000)
    _, _, wbar = ais.ratios(delta, np.zeros(2000), np.ones(2000), 5.0)
    for a in (0.0, 0.25, 1.0):
        wt = ais.rectify(wbar, a, np.ones(2000))
        assert np.all(wt >= 0) and np.all(wt <= 1 + a * 4.0 + 1e-12)


def test_diagnostics_against_exact_rationals():
    """Independent second implementation straight from the equations with exact fractions."""
    rng = np.random.default_rng(4)
    for trial in range(5):
        n = int(rng.integers(3, 48))
        # weights chosen as small rationals so every moment is exact
        wn = rng.integers(1, 40, n)
        w = [Fraction(int(k), 8) for k in wn]
        A = [Fraction(int(k), 4) for k in rng.integers(-4, 5, n)]
        wc = [min(x, Fraction(5)) for x in w]                  # w_bar = min(w, C)
        Aw = [a * x for a, x in zip(A, wc)]
        mu = sum(wc) / n
        var = sum((x - mu) ** 2 for x in wc) / n
        cv2 = var / mu ** 2
        ess = sum(wc) ** 2 / sum(x * x for x in wc)
        mA = sum(A) / n
        vA = sum((a - mA) ** 2 for a in A) / n
        mAw = sum(Aw) / n
        vAw = sum((a - mAw) ** 2 for a in Aw) / n
        d = _diag_from_w([float(x) for x in w], A=[float(a) for a in A])
        assert d["cv2"] == pytest.approx(float(cv2), rel=1e-12, abs=1e-14)
        assert d["ess"] == pytest.approx(float(ess), rel=1e-12)
        assert d["std_A"] == pytest.approx(math.sqrt(float(vA)), rel=1e-12, abs=1e-14)
        assert d["std_Aw"] == pytest.approx(math.sqrt(float(vAw)), rel=1e-12, abs=1e-14)
        dbar = math.fsum(abs(math.log(float(x))) for x in w) / n
        assert d["d_bar"] == pytest.approx(dbar, rel=1e-12)


def test_masked_tokens_are_ignored():
    rng = np.random.default_rng(5)
    lt, lr = rng.normal(-3, 1, 40), rng.normal(-3, 1, 40)
    A = rng.normal(size=40)
    mask = (rng.random(40) < 0.5).astype(np.uint8)
    full = ais.diagnostics(lt, lr, mask, A, P0)
    sel = mask.astype(bool)
    sub = ais.diagnostics(lt[sel], lr[sel], np.ones(sel.sum(), np.uint8), A[sel], P0)
    for k in sub:
        assert full[k] == pytest.approx(sub[k], rel=1e-13, abs=1e-15)
    empty = ais.diagnostics(lt, lr, np.zeros(40, np.uint8), A, P0)
    assert empty["alpha"] == 0.0 and empty["n_valid"] == 0


def test_monitor_outputs_hand_numbers_and_direction():
    """kl_k1 = mean(log pi_roll - log pi_train) over the valid rows, the sample estimate of KL(pi_roll || pi_train)
    on tokens drawn from the rollout policy, and mean_abs_dp = mean |pi_train - pi_roll| of the sampled tokens
    (caption of the training-behaviour figure).  Hand numbers from tests/golden/diag_closed_forms.txt; a swap of
    the two arguments or a flipped sign changes the asymmetric case; masked rows hold garbage."""
    g = _golden()
    one = np.ones(2, np.uint8)
    d = ais.diagnostics(np.log([0.5, 0.25]), np.log([0.25, 0.5]), one, np.ones(2), P0)
    assert d["mean_abs_dp"] == pytest.approx(g[("monitor_swap", "mean_abs_dp")], abs=1e-15)
    assert d["kl_k1"] == pytest.approx(g[("monitor_swap", "kl_k1")], abs=1e-15)
    lt = np.array([math.log(0.5), 7.0, math.log(0.5), -50.0])
    lr = np.array([math.log(0.25), -3.0, math.log(0.125), 2.0])
    d = ais.diagnostics(lt, lr, np.array([1, 0, 1, 0], np.uint8), np.ones(4), P0)
    assert d["mean_abs_dp"] == pytest.approx(g[("monitor_down", "mean_abs_dp")], abs=1e-15)
    assert d["kl_k1"] == pytest.approx(g[("monitor_down", "kl_k1")], abs=1e-15)
    assert d["kl_k1"] < 0


def test_kl_monitor_equals_the_textbook_divergence_on_an_exact_sample():
    """Tokens that occur exactly in proportion to pi_roll make the sample mean the expectation: kl_k1 then equals
    sum_v pi_roll(v) log(pi_roll(v) / pi_train(v)) -- the divergence from the rollout to the trainer, not the other
    direction -- and mean_abs_dp equals sum_v pi_roll(v) |pi_train(v) - pi_roll(v)|."""
    p_roll = np.array([0.5, 0.25, 0.125, 0.125])
    p_train = np.array([0.1, 0.2, 0.3, 0.4])
    tok = np.array([0, 0, 0, 0, 1, 1, 2, 3])                 # counts 4 : 2 : 1 : 1 = pi_roll
    d = ais.diagnostics(np.log(p_train[tok]), np.log(p_roll[tok]), np.ones(8, np.uint8), np.ones(8), P0)
    kl_roll_train = math.fsum(q * math.log(q / p) for q, p in zip(p_roll, p_train))
    kl_train_roll = math.fsum(p * math.log(p / q) for q, p in zip(p_roll, p_train))
    assert d["kl_k1"] == pytest.approx(kl_roll_train, rel=1e-13)
    assert abs(d["kl_k1"] - kl_train_roll) > 0.05 and kl_roll_train > 0
    assert d["mean_abs_dp"] == pytest.approx(math.fsum(q * abs(p - q) for q, p in zip(p_roll, p_train)), rel=1e-13)


# ------------------------------------------------------------------ advantages
def test_advantages():
    r = np.array([1, 0, 0, 1, 1, 1, 1, 1, 0, 0, 0, 0], dtype=np.float64)
    a = ais.advantages(r, 4)
    assert a.reshape(3, 4).sum(axis=1) == pytest.approx([0, 0, 0], abs=1e-15)
    assert a[:4] == pytest.approx([0.5, -0.5, -0.5, 0.5])
    assert np.all(a[4:] == 0)                                    # all-equal groups -> zero advantage
    an = ais.advantages(r, 4, adv_std_norm=True, eps=1e-6)
    assert an[:4] == pytest.approx(np.array([1, -1, -1, 1]) / (1 + 2e-6), rel=1e-5)


# ------------------------------------------------------------------ log-probs
def test_softmax_rows_sum_to_one_and_naive_form():
    rng = np.random.default_rng(6)
    H = rng.normal(size=(20, 8))
    W = rng.normal(size=(16, 8)) * 0.3
    z = ais.logits(H, W)
    # every token in turn: exp(lp) over the whole vocabulary sums to 1 (brute force over V = 16)
    tot = np.zeros(20)
    best = np.full(20, -np.inf)
    arg = np.zeros(20, dtype=int)
    for v in range(16):
        lp, lse = ais.log_softmax_gather(z, np.full(20, v), np.ones(20))
        tot += np.exp(lp)
        arg = np.where(lp > best, v, arg)
        best = np.maximum(best, lp)
        naive = z[:, v] - np.log(np.exp(z).sum(axis=1))          # no max shift
        assert lp == pytest.approx(naive, abs=1e-12)
    assert tot == pytest.approx(np.ones(20), abs=1e-12)
    assert np.array_equal(arg, z.argmax(axis=1))
    # the matmul orientation: z[t, v] = sum_k H[t,k] W[v,k]
    assert z[3, 5] == pytest.approx(sum(H[3, k] * W[5, k] for k in range(8)), abs=1e-13)


def test_large_logits_do_not_overflow():
    z = np.array([[1000.0, 999.0, -1000.0]])
    lp, lse = ais.log_softmax_gather(z, [0], [1])
    assert lse[0] == pytest.approx(1000.0 + math.log(1 + math.exp(-1)), abs=1e-12)
    assert lp[0] == pytest.approx(-math.log(1 + math.exp(-1)), abs=1e-12)


def test_masked_rows_zero():
    rng = np.random.default_rng(7)
    z = rng.normal(size=(6, 9))
    lp, lse = ais.log_softmax_gather(z, [1] * 6, [1, 0, 1, 0, 0, 1])
    assert lp[1] == 0 and lse[3] == 0 and lp[0] != 0


def _lossless_operands(rng, rows, d, block):
    """Values that quantise without error: E4M3 grid values times a power-of-two scale, block amax = 448 * 2^e."""
    grid = e4m3.decode(np.arange(0x08, 0x7F, dtype=np.uint8))
    grid = grid[(np.arange(0x08, 0x7F) & 0x7) % 2 == 0]            # keep bf16-exact products trivially
    x = np.zeros((rows, d))
    for r in range(rows):
        for b in range(d // block):
            e = int(rng.integers(-12, -6))
            vals = rng.choice(grid, block) * rng.choice([-1.0, 1.0], block)
            vals[int(rng.integers(block))] = 448.0
            x[r, b * block:(b + 1) * block] = vals * 2.0 ** e
    return x


def test_lossless_quantisation_gives_identical_passes():
    rng = np.random.default_rng(8)
    H = _lossless_operands(rng, 12, 64, 32)
    W = _lossless_operands(rng, 24, 64, 32)
    tok = rng.integers(0, 24, 12)
    mask = np.ones(12, np.uint8)
    lp_t, _ = ais.logprob_train(H, W, tok, mask)
    lp_r, _, (qH, sH, qW, sW) = ais.logprob_rollout(H, W, tok, mask, 32)
    assert np.array_equal(e4m3.dequantize_blocks(qH, sH, 32), H)
    assert np.array_equal(lp_t, lp_r)


def test_rollout_perturbation_sanity_band():
    """N(0,1) hidden, N(0,1/d) weights at d=256: FP8 noise moves log-probs by a few 1e-2, not by 1 and not by 1e-5."""
    import torch
    rng = np.random.default_rng(9)
    H = torch.tensor(rng.normal(size=(64, 256)), dtype=torch.float32).to(torch.bfloat16).float().numpy()
    W = torch.tensor(rng.normal(size=(512, 256)) / 16, dtype=torch.float32).to(torch.bfloat16).float().numpy()
    tok = rng.integers(0, 512, 64)
    mask = np.ones(64, np.uint8)
    lp_t, _ = ais.logprob_train(H, W, tok, mask)
    lp_r, _, _ = ais.logprob_rollout(H, W, tok, mask, 128)
    dbar = np.mean(np.abs(lp_t - lp_r))
    assert 3e-3 < dbar < 2e-1


# ------------------------------------------------------------------ loss and gradient
def _tiny_problem(seed=10, T=12, d=6, V=11, P=2, G=2):
    rng = np.random.default_rng(seed)
    H = rng.normal(size=(T, d))
    W = rng.normal(size=(V, d)) * 0.5
    tok = rng.integers(0, V, T)
    mask = (rng.random(T) < 0.8).astype(np.uint8)
    mask[0] = 1
    offs = np.array([0, 3, 6, 10, 12])
    rewards = np.array([1.0, 0.0, 0.0, 1.0])
    return H, W, tok, mask, offs, rewards, P, G


def _loss_of_H(H, W, tok, mask, offs, adv, w_tilde, lp_old, P, G, clip):
    lp, _ = ais.logprob_train(H, W, tok, mask)
    loss, _ = ais.loss_and_coeff(lp, lp_old, mask, offs, adv, w_tilde, P, G, clip)
    return loss


@pytest.mark.parametrize("shift_old", [0.0, 0.35])
def test_gradient_matches_central_differences(shift_old):
    H, W, tok, mask, offs, rewards, P, G = _tiny_problem()
    rng = np.random.default_rng(11)
    adv = ais.advantages(rewards, G)
    w_tilde = 1.0 + 0.7 * (np.minimum(np.exp(rng.normal(0, 0.5, len(tok))), 5.0) - 1.0)
    lp0, _ = ais.logprob_train(H, W, tok, mask)
    lp_old = lp0 + shift_old * rng.choice([-1.0, 1.0], len(tok))   # shift 0.35 -> rho_on outside [0.8, 1.2]
    loss, c = ais.loss_and_coeff(lp0, lp_old, mask, offs, adv, w_tilde, P, G, 0.2)
    if shift_old:
        assert np.any((c == 0) & (mask == 1) & (adv[ais.seq_ids(offs, len(tok))] != 0))   # clip is active somewhere
    dH = ais.grad_hidden(H, W, tok, c)
    num = np.zeros_like(H)
    h = 1e-5
    for t in range(H.shape[0]):
        for k in range(H.shape[1]):
            Hp, Hm = H.copy(), H.copy()
            Hp[t, k] += h
            Hm[t, k] -= h
            num[t, k] = (_loss_of_H(Hp, W, tok, mask, offs, adv, w_tilde, lp_old, P, G, 0.2)
                         - _loss_of_H(Hm, W, tok, mask, offs, adv, w_tilde, lp_old, P, G, 0.2)) / (2 * h)
    assert np.linalg.norm(dH - num) <= 1e-6 * max(np.linalg.norm(num), 1e-12) + 1e-10
    assert np.all(dH[mask == 0] == 0)


def test_kl_term_value_sign_and_gradient():
    """kl_t = r - log r - 1 >= 0 with equality at r = 1; closed form on hand values; the gradient including the
    KL term matches central differences (the reference log-probs come from a second, perturbed LM head)."""
    H, W, tok, mask, offs, rewards, P, G = _tiny_problem(seed=16)
    rng = np.random.default_rng(17)
    adv = ais.advantages(rewards, G)
    w_tilde = np.ones(len(tok))
    lp0, _ = ais.logprob_train(H, W, tok, mask)
    W_ref = W + rng.normal(0, 0.2, W.shape)
    lp_ref, _ = ais.logprob_train(H, W_ref, tok, mask)
    # value: identical policies give zero, otherwise positive; one token worked by hand
    assert ais.kl_term(lp0, lp0, mask, offs, P, G) == 0.0
    assert ais.kl_term(lp0, lp_ref, mask, offs, P, G) > 0.0
    one = ais.kl_term(np.array([math.log(0.5)]), np.array([math.log(0.25)]), np.ones(1), np.array([0, 1]), 1, 1)
    assert one == pytest.approx(0.5 - math.log(0.5) - 1.0, abs=1e-15)            # r = 1/2
    beta = 0.7
    l0, c0 = ais.loss_and_coeff(lp0, lp0, mask, offs, adv, w_tilde, P, G, 0.2)
    l1, c1 = ais.loss_and_coeff(lp0, lp0, mask, offs, adv, w_tilde, P, G, 0.2, lp_ref=lp_ref, beta_kl=beta)
    assert l1 - l0 == pytest.approx(beta * ais.kl_term(lp0, lp_ref, mask, offs, P, G), abs=1e-14)
    dH = ais.grad_hidden(H, W, tok, c1)
    num = np.zeros_like(H)
    h = 1e-5

    def f(Hx):
        lp, _ = ais.logprob_train(Hx, W, tok, mask)
        return ais.loss_and_coeff(lp, lp0, mask, offs, adv, w_tilde, P, G, 0.2, lp_ref=lp_ref, beta_kl=beta)[0]
    for t in range(H.shape[0]):
        for k in range(H.shape[1]):
            Hp, Hm = H.copy(), H.copy()
            Hp[t, k] += h
            Hm[t, k] -= h
            num[t, k] = (f(Hp) - f(Hm)) / (2 * h)
    assert np.linalg.norm(dH - num) <= 1e-6 * np.linalg.norm(num) + 1e-10
    assert np.linalg.norm(ais.grad_hidden(H, W, tok, c1 - c0)) > 0                 # the KL part is not a no-op


def test_weight_gradient_matches_central_differences():
    """dW against central differences of the loss in every entry of W (clip active, KL term on)."""
    H, W, tok, mask, offs, rewards, P, G = _tiny_problem(seed=18, T=12, d=5, V=7)
    rng = np.random.default_rng(19)
    adv = ais.advantages(rewards, G)
    w_tilde = 1.0 + 0.5 * (np.minimum(np.exp(rng.normal(0, 0.5, len(tok))), 5.0) - 1.0)
    lp0, _ = ais.logprob_train(H, W, tok, mask)
    lp_old = lp0 + 0.3 * rng.choice([-1.0, 1.0], len(tok))
    lp_ref = lp0 + rng.normal(0, 0.3, len(tok))

    def f(Wx):
        lp, _ = ais.logprob_train(H, Wx, tok, mask)
        return ais.loss_and_coeff(lp, lp_old, mask, offs, adv, w_tilde, P, G, 0.2, lp_ref=lp_ref, beta_kl=0.3)[0]
    _, c = ais.loss_and_coeff(lp0, lp_old, mask, offs, adv, w_tilde, P, G, 0.2, lp_ref=lp_ref, beta_kl=0.3)
    dW = ais.grad_weight(H, W, tok, c)
    assert dW.shape == W.shape
    num = np.zeros_like(W)
    h = 1e-5
    for v in range(W.shape[0]):
        for k in range(W.shape[1]):
            Wp, Wm = W.copy(), W.copy()
            Wp[v, k] += h
            Wm[v, k] -= h
            num[v, k] = (f(Wp) - f(Wm)) / (2 * h)
    assert np.linalg.norm(dW - num) <= 1e-6 * np.linalg.norm(num) + 1e-10
    # columns of (p - onehot) sum to zero over the vocabulary, so the rows of dW sum to zero over v
    assert np.abs(dW.sum(axis=0)).max() < 1e-12


def test_logit_gradient_rows_sum_to_zero_and_weight_layout():
    H, W, tok, mask, offs, rewards, P, G = _tiny_problem(seed=12)
    c = np.random.default_rng(0).normal(size=len(tok))
    # dH = (c (p - onehot)) W ; with W = identity-like columns the row sums of (p - onehot) show through
    Wones = np.ones_like(W)
    assert np.abs(ais.grad_hidden(H, Wones, tok, c)).max() < 1e-12     # rows of (p - e_y) sum to 0
    dH = ais.grad_hidden(H, W, tok, c)
    t = 4
    z = H[t] @ W.T
    p = np.exp(z - z.max())
    p /= p.sum()
    p[tok[t]] -= 1
    assert dH[t] == pytest.approx(c[t] * (p @ W), abs=1e-12)


def test_alpha_endpoints_and_linearity():
    """alpha = 0 is plain GRPO, alpha = 1 is truncated IS (Eq. token-level-tis), and
    g(alpha) = (1 - alpha) g(0) + alpha g(1)  (Appendix, mixed estimator)."""
    H, W, tok, mask, offs, rewards, P, G = _tiny_problem(seed=13)
    T = len(tok)
    rng = np.random.default_rng(14)
    lp_t, _ = ais.logprob_train(H, W, tok, mask)
    lp_r = lp_t + rng.normal(0, 0.8, T)
    adv = ais.advantages(rewards, G)
    sid = ais.seq_ids(offs, T)
    n = ais.valid_counts(mask, offs)
    _, rho, wbar = ais.ratios(lp_t, lp_r, mask, 5.0)
    grads, losses = {}, {}
    for a in (0.0, 0.37, 1.0):
        wt = ais.rectify(wbar, a, mask)
        losses[a], c = ais.loss_and_coeff(lp_t, lp_t, mask, offs, adv, wt, P, G, 0.2)
        grads[a] = ais.grad_hidden(H, W, tok, c)
    # independent statements of the two endpoints
    norm = mask / (P * G * np.maximum(n[sid], 1))
    c_grpo = adv[sid] * norm
    c_tis = np.minimum(rho, 5.0) * adv[sid] * norm
    assert grads[0.0] == pytest.approx(ais.grad_hidden(H, W, tok, c_grpo), abs=1e-14)
    assert grads[1.0] == pytest.approx(ais.grad_hidden(H, W, tok, c_tis), abs=1e-14)
    assert grads[0.37] == pytest.approx(0.63 * grads[0.0] + 0.37 * grads[1.0], abs=1e-14)
    assert losses[0.37] == pytest.approx(0.63 * losses[0.0] + 0.37 * losses[1.0], abs=1e-14)
    # with rho_on = 1 the objective is sum_s A_s / (P G n_s) * sum_t w_tilde_t
    J = sum(adv[s] / (P * G * n[s]) * wbar[(sid == s) & (mask == 1)].sum() for s in range(4) if n[s])
    assert losses[1.0] == pytest.approx(-J, abs=1e-14)


def test_empty_sequence_contributes_nothing():
    H, W, tok, mask, offs, rewards, P, G = _tiny_problem(seed=15)
    mask[:] = 1
    mask[3:6] = 0                                              # sequence 1 has no valid position
    lp, _ = ais.logprob_train(H, W, tok, mask)
    adv = ais.advantages(rewards, G)
    loss, c = ais.loss_and_coeff(lp, lp, mask, offs, adv, np.ones(len(tok)), P, G, 0.2)
    assert np.all(c[3:6] == 0) and np.isfinite(loss)


def test_full_path_runs_on_tiny_workload():
    import workloads
    b = workloads.make_batch(workloads.scaled(workloads.WORKLOADS["tiny"], V=256, lengths="const:16"))
    a = workloads.to_numpy(b)
    w = b.workload
    out = ais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block)
    assert out["dH"].shape == a["H"].shape
    assert 0 <= out["diag"]["alpha"] <= 1
    assert 1e-3 < out["diag"]["d_bar"] < 0.3


def test_microscaling_rollout_equals_trainer_when_lossless():
    """Every block on the E4M3 grid times a power of two: the microscaling rollout pass sees the same operands as
    the trainer pass (zero divergence), and otherwise it differs by a small, non-zero amount."""
    rng = np.random.default_rng(31)
    T, d, V = 6, 64, 24
    def lossless(rows):
        codes = rng.integers(0, 256, size=(rows, d)).astype(np.uint8)
        codes[(codes & 0x7F) == 0x7F] = 0x28
        codes[(codes & 0x78) == 0x78] &= 0xBF                      # keep |values| <= 120 so that bf16 holds them exactly
        codes[:, ::32] = 0x7E
        k = rng.integers(-12, -6, size=(rows, d // 32))
        return np.ldexp(e4m3.decode(codes).reshape(rows, d // 32, 32), k[:, :, None]).reshape(rows, d)
    H, W = lossless(T), lossless(V)
    tok = rng.integers(0, V, T)
    mask = np.ones(T, np.uint8)
    lp_t, _ = ais.logprob_train(H, W, tok, mask)
    lp_r, _, _ = ais.logprob_rollout(H, W, tok, mask, ais.MX32)
    assert np.array_equal(lp_t, lp_r)
    H2 = np.asarray(rng.normal(size=(T, d)), np.float32).astype(np.float64)
    lp_t2, _ = ais.logprob_train(H2, W, tok, mask)
    lp_r2, _, _ = ais.logprob_rollout(H2, W, tok, mask, ais.MX32)
    dlt = np.abs(lp_t2 - lp_r2)
    assert 0 < dlt.max() < 0.5


def test_sequence_level_weight_is_the_product_of_token_ratios():
    """Eq. is-weight with hand numbers: rho = (2, 1/2, 3) gives w = 3; truncation at C; a masked position drops out;
    sequences of one token reproduce the token-level weights; equal policies give weight 1."""
    lp_r = np.zeros(7)
    lp_t = np.log(np.array([2.0, 0.5, 3.0, 7.0, 1.0, 4.0, 4.0]))
    mask = np.array([1, 1, 1, 0, 1, 1, 1], np.uint8)
    offs = np.array([0, 4, 5, 7])
    logw, wbar = ais.ratios_sequence(lp_t, lp_r, mask, offs, C=5.0)
    assert np.allclose(np.exp(logw), [3.0, 1.0, 16.0])
    assert np.allclose(wbar, [3, 3, 3, 1, 1, 5, 5])                     # row 3 is masked; 16 is truncated to C
    _, wbar2 = ais.ratios_sequence(lp_t, lp_r, mask, offs, C=2.0)
    assert np.allclose(wbar2, [2, 2, 2, 1, 1, 2, 2])
    one = np.arange(8)
    _, _, tok = ais.ratios(lp_t, lp_r, np.ones(7, np.uint8), 5.0)
    _, seq = ais.ratios_sequence(lp_t, lp_r, np.ones(7, np.uint8), one, 5.0)
    assert np.allclose(tok, seq)
    _, same = ais.ratios_sequence(lp_t, lp_t, mask, offs, 5.0)
    assert np.all(same == 1.0)


def test_sequence_level_path_constant_drift():
    """Delta = delta on every token of sequences of length L: w_bar = min(e^{L delta}, C) on every row, so the
    weights are constant within the batch only if all lengths agree: CV = 0, alpha_ess = 1."""
    T, L = 24, 6
    offs = np.arange(0, T + 1, L)
    lp_r = -np.ones(T)
    lp_t = lp_r + 0.1
    mask = np.ones(T, np.uint8)
    _, wbar = ais.ratios_sequence(lp_t, lp_r, mask, offs, 5.0)
    assert np.allclose(wbar, math.exp(0.6))
    adv_tok = np.repeat([0.5, -0.5, 0.5, -0.5], L)
    d = ais.diagnostics(lp_t, lp_r, mask, adv_tok, ais.Params(seq_level=True), wbar_rows=wbar)
    assert abs(d["cv2"]) < 1e-20 and abs(d["alpha_ess"] - 1) < 1e-12 and abs(d["d_bar"] - 0.1) < 1e-12
    assert abs(d["delta_sigma"] - math.exp(0.6) * 0.5 / (0.5 + 1e-6)) < 1e-9
