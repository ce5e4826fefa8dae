"""AIS-GRPO hot path in float64 numpy (oracle; test infrastructure only).

Every function states the passage of the paper it follows.  Nothing here is
blocked, fused or reordered: each routine is the definition written out, with
numpy's float64 matmul / exp / log as the library steps.

Conventions shared with the GPU library
---------------------------------------
H       [T, d]   hidden states (bf16-representable values)
W       [V, d]   LM head, one row per vocabulary entry (so logits z = H @ W.T)
tokens  [T]      sampled token ids
mask    [T]      1 = position takes part, 0 = padding / unmasked position
seq_offsets [S+1] row offsets of the S = P*G sequences; the G sequences of one
                 prompt are consecutive
"""

from __future__ import annotations

from dataclasses import dataclass
import math

import numpy as np

from . import e4m3


@dataclass
class Params:
    """Hyper-parameters (Appendix 'AIS hyperparameters' and Table of GRPO settings).

    beta_var is listed by Algorithm 1 but the paper prints no value for it;
    1.0 is the reading taken here.  alpha_override = None keeps the adaptive
    coefficient; a number forces alpha (0 = plain GRPO, 1 = truncated IS).
    """
    C: float = 5.0
    delta: float = 0.02
    gamma: float = 1.2
    eps: float = 1e-6
    beta_var: float = 1.0
    clip_eps: float = 0.2
    alpha_override: float | None = None
    adv_std_norm: bool = False
    seq_level: bool = False          # importance weight per sequence (Eq. is-weight) instead of per token


# --------------------------------------------------------------------------- log-probs
def logits(H, W) -> np.ndarray:
    """z = H W^T in float64 (Eq. logit-mismatch: f(x; theta) at the LM head)."""
    return np.asarray(H, dtype=np.float64) @ np.asarray(W, dtype=np.float64).T


def log_softmax_gather(z, tokens, mask):
    """lse_t = log sum_v exp z_tv ; lp_t = z[t, y_t] - lse_t   (Algorithm 1, 'full-precision log-probs').

    Rows with mask 0 give lp = 0 and lse = 0.
    """
    z = np.asarray(z, dtype=np.float64)
    T = z.shape[0]
    m = np.max(z, axis=1)
    lse = m + np.log(np.sum(np.exp(z - m[:, None]), axis=1))
    lp = z[np.arange(T), np.asarray(tokens, dtype=np.int64)] - lse
    valid = np.asarray(mask).astype(bool)
    return np.where(valid, lp, 0.0), np.where(valid, lse, 0.0)


def logprob_train(H, W, tokens, mask):
    """Trainer pass: bf16 operands, wide accumulation, temperature 1."""
    return log_softmax_gather(logits(H, W), tokens, mask)


MX32 = -32        # `block` value selecting microscaling FP8 (E8M0 scale per 32 elements)
MXFP4 = -4        # `block` value selecting microscaling FP4 (E2M1 elements, E8M0 scale per 32 elements)


def logprob_rollout(H, W, tokens, mask, block: int):
    """Rollout pass: weights and activations quantised to E4M3 per block along d
    (Section 2.1: 'we quantize both the weights and activations of the rollout model'),
    then the same log-softmax.  block = 0 selects one scale per tensor (Appendix 'FP8 rollout': per-tensor
    dynamic scaling); block = MX32 selects power-of-two scales per 32 elements (the microscaling format named as
    future work in the paper's limitations).  Returns (lp, lse, (qH, sH, qW, sW))."""
    if block == MXFP4:
        qH, sH = e4m3.quantize_mxfp4(H)
        qW, sW = e4m3.quantize_mxfp4(W)
        Hq = e4m3.dequantize_mxfp4(qH, sH)
        Wq = e4m3.dequantize_mxfp4(qW, sW)
    elif block == MX32:
        qH, sH = e4m3.quantize_mx(H)
        qW, sW = e4m3.quantize_mx(W)
        Hq = e4m3.dequantize_mx(qH, sH)
        Wq = e4m3.dequantize_mx(qW, sW)
    elif block == 0:
        qH, sH = e4m3.quantize_tensor(H)
        qW, sW = e4m3.quantize_tensor(W)
        Hq = e4m3.decode(qH) * np.float64(sH)
        Wq = e4m3.decode(qW) * np.float64(sW)
    else:
        qH, sH = e4m3.quantize_blocks(H, block)
        qW, sW = e4m3.quantize_blocks(W, block)
        Hq = e4m3.dequantize_blocks(qH, sH, block)
        Wq = e4m3.dequantize_blocks(qW, sW, block)
    lp, lse = log_softmax_gather(logits(Hq, Wq), tokens, mask)
    return lp, lse, (qH, sH, qW, sW)


# --------------------------------------------------------------------------- ratios
def ratios(lp_train, lp_roll, mask, C: float):
    """Delta_t, rho_t = exp(Delta_t) (Algorithm 1, sampler-trainer ratio) and
    w_bar_t = min(rho_t, C) (Eq. ais-components).  Invalid rows: Delta 0, rho 1, w_bar 1."""
    valid = np.asarray(mask).astype(bool)
    delta = np.where(valid, np.asarray(lp_train, np.float64) - np.asarray(lp_roll, np.float64), 0.0)
    with np.errstate(over="ignore"):
        rho = np.exp(delta)
    wbar = np.exp(np.minimum(delta, math.log(C)))
    return delta, rho, wbar


def ratios_sequence(lp_train, lp_roll, mask, seq_offsets, C: float):
    """Sequence-level importance weight of Eq. is-weight, w(x) = prod_t rho_t over the valid positions of a
    sequence, truncated as in Eq. ais-components, w_bar(x) = min(w(x), C), and handed to every position of the
    sequence.  Returns (log w per sequence, w_bar per row); invalid rows get 1.  The paper states this form and
    then argues for per-token truncation; it is offered as a variant."""
    valid = np.asarray(mask).astype(bool)
    delta = np.where(valid, np.asarray(lp_train, np.float64) - np.asarray(lp_roll, np.float64), 0.0)
    off = np.asarray(seq_offsets, dtype=np.int64)
    logw = np.array([delta[off[s]:off[s + 1]].sum() for s in range(len(off) - 1)])
    wbar_seq = np.exp(np.minimum(logw, math.log(C)))
    wbar = np.ones(len(delta))
    for s in range(len(off) - 1):
        wbar[off[s]:off[s + 1]] = wbar_seq[s]
    return logw, np.where(valid, wbar, 1.0)


# --------------------------------------------------------------------------- advantages
def advantages(rewards, G: int, adv_std_norm: bool = False, eps: float = 1e-6) -> np.ndarray:
    """A_i = r_i - mean_j r_j over the G responses of one prompt (Eq. grpo_adv, unnormalised form).
    adv_std_norm divides by (population std of the group + eps); not the paper's default."""
    r = np.asarray(rewards, dtype=np.float64).reshape(-1, G)
    a = r - r.mean(axis=1, keepdims=True)
    if adv_std_norm:
        a = a / (r.std(axis=1, keepdims=True) + eps)
    return a.reshape(-1)


def seq_ids(seq_offsets, T: int) -> np.ndarray:
    """Sequence index of every row."""
    off = np.asarray(seq_offsets, dtype=np.int64)
    ids = np.zeros(T, dtype=np.int64)
    for s in range(len(off) - 1):
        ids[off[s]:off[s + 1]] = s
    return ids


def valid_counts(mask, seq_offsets) -> np.ndarray:
    """n_s = number of valid positions of sequence s (|o_i| of the AIS-GRPO objective)."""
    off = np.asarray(seq_offsets, dtype=np.int64)
    m = np.asarray(mask).astype(np.int64)
    return np.array([m[off[s]:off[s + 1]].sum() for s in range(len(off) - 1)], dtype=np.int64)


# --------------------------------------------------------------------------- diagnostics
def diagnostics(lp_train, lp_roll, mask, adv_tok, p: Params, wbar_rows=None) -> dict:
    """The three signals and the mixing coefficient over the valid token set
    (Eqs. alpha-ess, discrepancy, alpha-mis, variance-amplification ratio, alpha-var, alpha-final).

    All moments are population moments (divide by N): the identity
    sqrt(ESS_ratio) = (1 + CV^2)^(-1/2) printed with Eq. alpha-ess only holds for those.
    """
    valid = np.asarray(mask).astype(bool)
    N = int(valid.sum())
    out = dict(n_valid=float(N))
    if N == 0:
        out.update(mean_w=1.0, cv2=0.0, ess=0.0, ess_ratio=1.0, alpha_ess=1.0, d_bar=0.0,
                   alpha_mis=0.0, std_A=0.0, std_Aw=0.0, delta_sigma=0.0, alpha_var=0.0,
                   alpha=0.0, alpha_adaptive=0.0, kl_k1=0.0, mean_abs_dp=0.0)
        if p.alpha_override is not None:
            out["alpha"] = float(p.alpha_override)
        return out
    delta, _, wbar = ratios(lp_train, lp_roll, mask, p.C)
    if wbar_rows is not None:             # sequence-level variant: every valid row carries its sequence's weight
        wbar = np.asarray(wbar_rows, np.float64)
    d = delta[valid]
    w = wbar[valid]
    A = np.asarray(adv_tok, dtype=np.float64)[valid]

    mu = w.mean()
    var = np.mean((w - mu) ** 2)
    cv2 = var / (mu * mu)
    ess = w.sum() ** 2 / np.sum(w * w)
    alpha_ess = (1.0 + cv2) ** -0.5

    d_bar = np.mean(np.abs(d))
    alpha_mis = min(1.0, d_bar / p.delta)

    Aw = A * w
    std_A = math.sqrt(np.mean((A - A.mean()) ** 2))
    std_Aw = math.sqrt(np.mean((Aw - Aw.mean()) ** 2))
    delta_sigma = std_Aw / (std_A + p.eps)
    alpha_var = max(0.0, (delta_sigma - p.gamma) / p.gamma)

    alpha = min(1.0, max(0.0, alpha_ess - p.beta_var * alpha_var)) * alpha_mis
    lt = np.asarray(lp_train, np.float64)[valid]
    lr = np.asarray(lp_roll, np.float64)[valid]
    out.update(mean_w=float(mu), cv2=float(cv2), ess=float(ess), ess_ratio=float(ess / N),
               alpha_ess=float(alpha_ess), d_bar=float(d_bar), alpha_mis=float(alpha_mis),
               std_A=float(std_A), std_Aw=float(std_Aw), delta_sigma=float(delta_sigma),
               alpha_var=float(alpha_var), alpha_adaptive=float(alpha), alpha=float(alpha),
               kl_k1=float(np.mean(lr - lt)),
               mean_abs_dp=float(np.mean(np.abs(np.exp(lt) - np.exp(lr)))))
    if p.alpha_override is not None:
        out["alpha"] = float(p.alpha_override)
    return out


def rectify(wbar, alpha: float, mask) -> np.ndarray:
    """w_tilde = 1 + alpha (w_bar - 1)  (Algorithm 1, rectification weight); 1 on invalid rows."""
    valid = np.asarray(mask).astype(bool)
    return np.where(valid, 1.0 + alpha * (np.asarray(wbar, np.float64) - 1.0), 1.0)


# --------------------------------------------------------------------------- loss / gradient
def surrogate_terms(lp_theta, lp_old, adv_tok, clip_eps: float):
    """Per token: rho_on, min(rho_on A, clip(rho_on, 1-eps, 1+eps) A) and the indicator that
    the unclipped branch is the active one (ties count as unclipped)."""
    rho_on = np.exp(np.asarray(lp_theta, np.float64) - np.asarray(lp_old, np.float64))
    A = np.asarray(adv_tok, np.float64)
    un = rho_on * A
    cl = np.clip(rho_on, 1.0 - clip_eps, 1.0 + clip_eps) * A
    sur = np.minimum(un, cl)
    active = (un <= cl)
    return rho_on, sur, active


def loss_and_coeff(lp_theta, lp_old, mask, seq_offsets, adv, w_tilde, P: int, G: int, clip_eps: float,
                   lp_ref=None, beta_kl: float = 0.0):
    """loss = -J with J = sum_s 1/(P G n_s) sum_{t in s, valid} [w_tilde_t * sur_t - beta_kl * kl_t]
    (AIS-GRPO objective; the expectation over prompts is the mean over the P prompts, |o_i| = n_s).

    kl_t is the per-token estimate of D_KL(pi_theta || pi_ref).  The paper writes the term but not its
    estimator; the reading here is the one of the GRPO paper it builds on,
    kl_t = r - log r - 1 with r = pi_ref / pi_theta = exp(lp_ref - lp_theta), which is non-negative and
    zero only when the two log-probs agree.  lp_ref = None (or beta_kl = 0) drops the term.

    Also returns c_t, the per-token factor of the logit gradient
    d loss / d z[t, :] = c_t (softmax(z_t) - onehot(y_t)), with w_tilde, A and lp_old held constant
    (the diagnostics are computed from detached tensors, Appendix 'AIS hyperparameters').
    """
    T = len(mask)
    valid = np.asarray(mask).astype(bool)
    sid = seq_ids(seq_offsets, T)
    n = valid_counts(mask, seq_offsets)
    adv_tok = np.asarray(adv, np.float64)[sid]
    rho_on, sur, active = surrogate_terms(lp_theta, lp_old, adv_tok, clip_eps)
    n_tok = np.maximum(n[sid], 1).astype(np.float64)
    norm = 1.0 / (P * G * n_tok)
    wt = np.asarray(w_tilde, np.float64)
    J = np.sum(np.where(valid, wt * sur * norm, 0.0))
    c = np.where(valid & active, wt * adv_tok * rho_on * norm, 0.0)
    if lp_ref is not None and beta_kl != 0.0:
        log_r = np.asarray(lp_ref, np.float64) - np.asarray(lp_theta, np.float64)
        r = np.exp(log_r)
        kl = r - log_r - 1.0
        J = J - beta_kl * np.sum(np.where(valid, kl * norm, 0.0))
        # d kl / d lp_theta = 1 - r ; d loss / d lp_theta = +beta * norm * (1 - r) ; d lp / d z = onehot - p
        c = c - np.where(valid, beta_kl * (1.0 - r) * norm, 0.0)
    return -J, c


def kl_term(lp_theta, lp_ref, mask, seq_offsets, P: int, G: int) -> float:
    """sum_s 1/(P G n_s) sum_t kl_t : the value of the KL term of the objective (without beta)."""
    T = len(mask)
    valid = np.asarray(mask).astype(bool)
    sid = seq_ids(seq_offsets, T)
    n_tok = np.maximum(valid_counts(mask, seq_offsets)[sid], 1).astype(np.float64)
    log_r = np.asarray(lp_ref, np.float64) - np.asarray(lp_theta, np.float64)
    kl = np.exp(log_r) - log_r - 1.0
    return float(np.sum(np.where(valid, kl / (P * G * n_tok), 0.0)))


def logit_gradient(z, tokens, c) -> np.ndarray:
    """d loss / d z[t, :] = c_t (softmax(z_t) - onehot(y_t)): the gradient of -c_t log softmax(z_t)[y_t], the form every
    term of the objective takes once w_tilde, A and lp_old are held constant."""
    z = np.asarray(z, dtype=np.float64)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    T = z.shape[0]
    p[np.arange(T), np.asarray(tokens, np.int64)] -= 1.0
    p *= np.asarray(c, np.float64)[:, None]
    return p


def grad_hidden(H, W, tokens, c) -> np.ndarray:
    """dH[t, :] = c_t (softmax(z_t) - onehot(y_t)) W   in float64."""
    return logit_gradient(logits(H, W), tokens, c) @ np.asarray(W, np.float64)


def grad_weight(H, W, tokens, c) -> np.ndarray:
    """dW[v, :] = sum_t c_t (softmax(z_t)[v] - [v = y_t]) H[t, :]   in float64 (same layout as W: [V, d])."""
    return logit_gradient(logits(H, W), tokens, c).T @ np.asarray(H, np.float64)


# --------------------------------------------------------------------------- whole path
def full_path(H, W, tokens, mask, seq_offsets, rewards, P: int, G: int, block: int,
              params: Params | None = None, lp_old=None, want_grad: bool = True, lp_ref=None, beta_kl: float = 0.0) -> dict:
    """Algorithm 1, 'Adaptive Coefficient Estimation' through 'Policy Update' (loss and dH only)."""
    p = params or Params()
    T = np.asarray(H).shape[0]
    lp_t, lse_t = logprob_train(H, W, tokens, mask)
    lp_r, lse_r, (qH, sH, qW, sW) = logprob_rollout(H, W, tokens, mask, block)
    adv = advantages(rewards, G, p.adv_std_norm, p.eps)
    sid = seq_ids(seq_offsets, T)
    adv_tok = adv[sid]
    delta, rho, wbar = ratios(lp_t, lp_r, mask, p.C)
    if p.seq_level:
        _, wbar = ratios_sequence(lp_t, lp_r, mask, seq_offsets, p.C)
    diag = diagnostics(lp_t, lp_r, mask, adv_tok, p, wbar_rows=wbar if p.seq_level else None)
    w_tilde = rectify(wbar, diag["alpha"], mask)
    old = lp_t if lp_old is None else lp_old
    loss, c = loss_and_coeff(lp_t, old, mask, seq_offsets, adv, w_tilde, P, G, p.clip_eps, lp_ref=lp_ref, beta_kl=beta_kl)
    diag["loss"] = float(loss)
    out = dict(lp_train=lp_t, lse_train=lse_t, lp_roll=lp_r, lse_roll=lse_r, qH=qH, sH=sH, qW=qW, sW=sW,
               adv=adv, rho=rho, wbar=wbar, w_tilde=w_tilde, diag=diag, loss=loss, c=c)
    if want_grad:
        out["dH"] = grad_hidden(H, W, tokens, c)
        out["dW"] = grad_weight(H, W, tokens, c)
    return out
