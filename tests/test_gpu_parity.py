"""GPU parity: the CUDA library (through its C ABI) against the float64 oracle on the same seeded inputs.

Tolerances (stated with the workloads): FP8 codes and scales bit-exact; log-probs 1e-2 absolute; ratios 2e-2
relative; mixing coefficient 1e-3 absolute; hidden-state gradient 1e-2 relative Frobenius error.
"""

import math

import numpy as np
import pytest
import torch

import workloads
from oracle import ais as oais
from oracle import e4m3

pytestmark = pytest.mark.gpu

LP_ATOL = 1e-2
RHO_RTOL = 2e-2
ALPHA_ATOL = 1e-3
DH_REL = 1e-2


def _lib():
    import paper_2605_13907_b200 as ais
    return ais


def _rel_fro(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def _run_gpu(batch, params=None, lp_old=None, ws_cap=None):
    ais = _lib()
    w = batch.workload
    dev = batch.H.device
    step = ais.AisStep(batch.T, w.d, w.V, w.P, w.G, w.block, device=dev, params=params, workspace_bytes_cap=ws_cap)
    offs = batch.seq_offsets.to(dev)
    rew = batch.rewards.to(dev)
    step.step(batch.H, batch.W, batch.tokens, batch.mask, offs, rew, lp_old=lp_old)
    torch.cuda.synchronize()
    return step


def _oracle(batch, params=None, lp_old=None, rows=None):
    a = workloads.to_numpy(batch)
    w = batch.workload
    return a, oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block,
                             params=params, lp_old=lp_old)


def _compare_all(batch, step, ref, a, check_grad=True):
    T = batch.T
    valid = a["mask"].astype(bool)
    # FP8 codes and scales: bit-exact
    assert np.array_equal(step.qH.cpu().numpy()[:T], ref["qH"])
    assert np.array_equal(step.qW.cpu().numpy(), ref["qW"])
    assert np.array_equal(step.sH.cpu().numpy()[:, :T].T.view(np.uint32), ref["sH"].view(np.uint32))
    assert np.array_equal(step.sW.cpu().numpy()[:, :batch.W.shape[0]].T.view(np.uint32), ref["sW"].view(np.uint32))
    lp_t = step.lp_train.cpu().numpy()[:T].astype(np.float64)
    lp_r = step.lp_roll.cpu().numpy()[:T].astype(np.float64)
    assert np.max(np.abs(lp_t - ref["lp_train"])) <= LP_ATOL
    assert np.max(np.abs(lp_r - ref["lp_roll"])) <= LP_ATOL
    assert np.max(np.abs(step.lse_train.cpu().numpy()[:T] - ref["lse_train"])) <= LP_ATOL
    assert np.all(lp_t[~valid] == 0) and np.all(lp_r[~valid] == 0)
    rho = step.rho.cpu().numpy()[:T].astype(np.float64)
    assert np.max(np.abs(rho - ref["rho"]) / ref["rho"]) <= RHO_RTOL
    assert np.all(rho[~valid] == 1)
    w_tilde = step.w_tilde.cpu().numpy()[:T].astype(np.float64)
    assert np.max(np.abs(w_tilde - ref["w_tilde"]) / ref["w_tilde"]) <= RHO_RTOL      # 1 + alpha (min(rho, C) - 1)
    assert np.all(w_tilde[~valid] == 1)
    d = step.read_diag()
    assert abs(d["alpha"] - ref["diag"]["alpha"]) <= ALPHA_ATOL
    assert d["n_valid"] == ref["diag"]["n_valid"]
    assert np.allclose(step.adv.cpu().numpy(), ref["adv"], atol=1e-6)
    assert int(step.status.item()) == 0 and d["status_flags"] == 0
    if check_grad:
        dH = step.dH.float().cpu().numpy()[:T].astype(np.float64)
        assert _rel_fro(dH, ref["dH"]) <= DH_REL
        assert np.all(dH[~valid] == 0)
        assert abs(float(step.loss.item()) - ref["loss"]) <= 1e-3 * max(1.0, abs(ref["loss"]))
    return d


# ------------------------------------------------------------------ quantiser
@pytest.mark.parametrize("block", [32, 64, 128])
def test_quantize_bit_exact_adversarial(block):
    ais = _lib()
    g = torch.Generator().manual_seed(5)
    rows, cols = 77, 640                                    # ragged row count, several blocks per row
    x = torch.randn(rows, cols, generator=g) * torch.exp(torch.randn(rows, 1, generator=g) * 3)
    x[3] = 0.0                                              # all-zero row -> scale 1, codes 0
    x[4, :block] = 0.0
    x[5, 7] = 3.0e38                                        # huge amax
    x[6] = x[6] * 1e-38                                     # bf16 subnormals
    x[7, :block] = 3.5 * torch.linspace(-1, 1, block)       # near power-of-two scale
    x[8, 0] = -0.0
    xb = x.to(torch.bfloat16).cuda()
    codes, scales = ais.quantize_fp8(xb, block)
    torch.cuda.synchronize()
    rc, rs = e4m3.quantize_blocks(xb.float().cpu().numpy(), block)
    assert np.array_equal(scales.cpu().numpy()[:, :rows].T.view(np.uint32), rs.view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), rc)


def test_quantize_every_bf16_value():
    """All finite bf16 bit patterns, several scales: the hardware conversion agrees with the oracle's codec."""
    ais = _lib()
    bits = torch.arange(0, 1 << 16, dtype=torch.int32)
    vals = (bits << 16).view(torch.float32)
    vals = vals[torch.isfinite(vals)]
    n = (vals.numel() // 128) * 128
    for amax in (448.0, 1.0, 3.0e-3, 1.7e5):
        x = vals[:n].clone().reshape(-1, 128)
        x = torch.where(x.abs() > amax, torch.zeros_like(x), x)
        x[:, 0] = amax                                      # fixes every block's scale
        xb = x.to(torch.bfloat16).cuda()
        codes, scales = ais.quantize_fp8(xb, 128)
        torch.cuda.synchronize()
        rc, rs = e4m3.quantize_blocks(xb.float().cpu().numpy(), 128)
        assert np.array_equal(codes.cpu().numpy(), rc)
        assert np.array_equal(scales.cpu().numpy()[:, :x.shape[0]].T.view(np.uint32), rs.view(np.uint32))


def test_quantize_every_bf16_value_random_scales():
    """Every finite bf16 value against 60 block scales spread over 60 decades (the quotient x / s must be the
    correctly rounded one for the code to match, whatever the scale's mantissa)."""
    ais = _lib()
    bits = torch.arange(0, 1 << 16, dtype=torch.int32)
    vals = (bits << 16).view(torch.float32)
    vals = vals[torch.isfinite(vals)]
    n = (vals.numel() // 127) * 127
    rng = np.random.default_rng(0)
    for _ in range(60):
        amax = float(torch.tensor(np.exp(rng.uniform(np.log(1e-30), np.log(1e30))), dtype=torch.float32).to(torch.bfloat16))
        x = vals[:n].clone().reshape(-1, 127)
        x = torch.where(x.abs() > amax, torch.full_like(x, amax * 0.5), x)
        x = torch.cat([torch.full((x.shape[0], 1), amax), x], dim=1).to(torch.bfloat16).cuda()
        codes, scales = ais.quantize_fp8(x, 128)
        torch.cuda.synchronize()
        rc, rs = e4m3.quantize_blocks(x.float().cpu().numpy(), 128)
        assert np.array_equal(codes.cpu().numpy(), rc)
        assert np.array_equal(scales.cpu().numpy()[:, :x.shape[0]].T.view(np.uint32), rs.view(np.uint32))


# ------------------------------------------------------------------ whole path
def test_tiny_config_full_parity():
    batch = workloads.make_batch(workloads.WORKLOADS["tiny"], device="cpu")
    batch = _to_cuda(batch)
    step = _run_gpu(batch)
    a, ref = _oracle(batch)
    d = _compare_all(batch, step, ref, a)
    assert 0.0 <= d["alpha"] <= 1.0


def _to_cuda(b):
    return workloads.Batch(b.workload, b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda(), b.seq_offsets, b.rewards)


@pytest.mark.parametrize("case", ["ragged", "block32", "masked", "chunked"])
def test_small_shapes_full_parity(case):
    base = workloads.WORKLOADS["tiny"]
    if case == "ragged":      # T not a multiple of 128, V not a multiple of 256, several row tiles
        w = workloads.scaled(base, d=384, V=1336, P=3, G=4, lengths="uniform:5:90", seed=21)
    elif case == "block32":
        w = workloads.scaled(base, d=256, V=2048, P=2, G=4, block=32, lengths="uniform:40:120", seed=22)
    elif case == "masked":    # LLaDA-style scattered validity, one sequence with no valid row at all
        w = workloads.scaled(base, d=256, V=1024, P=2, G=4, lengths="const:96", mask_mode="llada", seed=23)
    else:                     # explicit vocabulary chunks with a ragged last chunk
        w = workloads.scaled(base, d=512, V=5000 // 8 * 8, P=2, G=2, lengths="uniform:100:300", vocab_chunk=1024, seed=24)
    batch = workloads.make_batch(w, device="cpu")
    if case == "masked":
        lo, hi = int(batch.seq_offsets[2]), int(batch.seq_offsets[3])
        batch.mask[lo:hi] = 0
    batch = _to_cuda(batch)
    ais = _lib()
    params = ais.default_params(vocab_chunk=w.vocab_chunk)
    step = _run_gpu(batch, params=params)
    a, ref = _oracle(batch)
    _compare_all(batch, step, ref, a)


def test_alpha_endpoints_and_clip_on_gpu():
    """alpha_override 0 / 1 reproduce the plain GRPO and truncated-IS gradients; lp_old != lp_train exercises the clip."""
    ais = _lib()
    w = workloads.scaled(workloads.WORKLOADS["tiny"], V=768, lengths="uniform:30:70", seed=31)
    batch = _to_cuda(workloads.make_batch(w, device="cpu"))
    a = workloads.to_numpy(batch)
    grads = {}
    for alpha in (0.0, 1.0, 0.4):
        step = _run_gpu(batch, params=ais.default_params(alpha_override=alpha))
        _, ref = _oracle(batch, params=oais.Params(alpha_override=alpha))
        _compare_all(batch, step, ref, a)
        grads[alpha] = step.dH.float().cpu().numpy().astype(np.float64)
    mix = 0.6 * grads[0.0] + 0.4 * grads[1.0]
    assert _rel_fro(grads[0.4], mix) <= 2e-2                    # bf16 outputs: linear up to output rounding
    # clip: shift lp_old so that rho_on leaves [0.8, 1.2] on many tokens
    _, ref0 = _oracle(batch)
    rng = np.random.default_rng(3)
    lp_old = ref0["lp_train"] + 0.3 * rng.choice([-1.0, 1.0], batch.T)
    lp_old_gpu = torch.tensor(lp_old, dtype=torch.float32, device="cuda")
    step = _run_gpu(batch, lp_old=lp_old_gpu)
    _, ref = _oracle(batch, lp_old=lp_old_gpu.cpu().numpy().astype(np.float64))
    assert np.any((ref["c"] == 0) & (a["mask"] == 1))
    _compare_all(batch, step, ref, a)


@pytest.mark.parametrize("C", [2.0, 10.0])
def test_truncation_threshold_sweep_on_gpu(C):
    """C = 2 and C = 10 (the thresholds of the paper's variation analysis besides the default 5) through
    ais_diagnostics and ais_loss_bwd on a batch whose ratios exceed both: the rollout log-probs of some rows are pushed
    down by 1 .. 3.5 nats, so rho reaches 2.7 .. 33 there.  Prop. 'bounded second moment': 0 <= w_tilde <= 1 + alpha (C - 1)."""
    ais = _lib()
    w = workloads.scaled(workloads.WORKLOADS["tiny"], V=768, P=3, G=4, lengths="uniform:30:70", seed=35)
    batch = _to_cuda(workloads.make_batch(w, device="cpu"))
    a = workloads.to_numpy(batch)
    T = batch.T
    step = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block, params=ais.default_params(C=C))
    step.forward(batch.H, batch.W, batch.tokens, batch.mask)
    torch.cuda.synchronize()
    rng = np.random.default_rng(36)
    shift = np.where(rng.random(T) < 0.15, rng.uniform(1.0, 3.5, T), 0.0)
    step.lp_roll[:T] -= torch.tensor(shift, dtype=torch.float32, device="cuda")
    offs, rew = batch.seq_offsets.cuda(), batch.rewards.cuda()
    step.diagnose(batch.mask, offs, rew)
    step.backward(batch.H, batch.W, batch.tokens, batch.mask, offs)
    torch.cuda.synchronize()
    assert int(step.status.item()) == 0
    lt = step.lp_train[:T].cpu().numpy().astype(np.float64)
    lr = step.lp_roll[:T].cpu().numpy().astype(np.float64)
    p = oais.Params(C=C)
    adv = oais.advantages(a["rewards"], w.G)
    _, rho, wbar = oais.ratios(lt, lr, a["mask"], C)
    assert np.sum(rho > C) >= 5 and np.sum(rho > 10.0) >= 1
    diag = oais.diagnostics(lt, lr, a["mask"], adv[oais.seq_ids(a["seq_offsets"], T)], p)
    w_tilde = oais.rectify(wbar, diag["alpha"], a["mask"])
    d = step.read_diag()
    assert abs(d["alpha"] - diag["alpha"]) <= ALPHA_ATOL
    for k in ("mean_w", "cv2", "ess_ratio", "alpha_ess", "d_bar", "delta_sigma", "alpha_var"):
        assert d[k] == pytest.approx(diag[k], rel=1e-4, abs=1e-7), k
    g_wt = step.w_tilde[:T].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(g_wt - w_tilde) / w_tilde) <= RHO_RTOL
    assert g_wt.min() >= 0.0 and g_wt.max() <= 1.0 + diag["alpha"] * (C - 1.0) + 1e-5
    assert np.max(np.abs(step.rho[:T].cpu().numpy() - rho) / rho) <= RHO_RTOL
    loss, c = oais.loss_and_coeff(lt, lt, a["mask"], a["seq_offsets"], adv, w_tilde, w.P, w.G, p.clip_eps)
    assert abs(float(step.loss.item()) - loss) <= 1e-3 * max(1.0, abs(loss))
    dH_ref = oais.grad_hidden(a["H"], a["W"], a["tokens"], c)
    assert _rel_fro(step.dH.float().cpu().numpy()[:T].astype(np.float64), dH_ref) <= DH_REL


def test_kl_term_on_gpu():
    """Eq. ais-grpo with its KL term: reference log-probs from a perturbed LM head (computed by the library's own
    forward pass on the GPU side and by the oracle on the CPU side), beta_kl = 0.5."""
    ais = _lib()
    w = workloads.scaled(workloads.WORKLOADS["tiny"], V=768, lengths="uniform:30:70", seed=33)
    batch = _to_cuda(workloads.make_batch(w, device="cpu"))
    a = workloads.to_numpy(batch)
    g = torch.Generator().manual_seed(7)
    W_ref = (batch.W.float().cpu() + 0.02 * torch.randn(batch.W.shape, generator=g)).to(torch.bfloat16)
    lp_ref_oracle, _ = oais.logprob_train(a["H"], W_ref.float().numpy(), a["tokens"], a["mask"])
    # reference pass on the GPU: the trainer kernel with the reference weights
    ref_step = ais.AisStep(batch.T, w.d, w.V, w.P, w.G, w.block)
    ais.logprob_fwd(ref_step.shape, ref_step.params, batch.H, W_ref.cuda(), None, None, None, None, batch.tokens, batch.mask,
                    ref_step.lp_train, ref_step.lse_train, None, None, ref_step.status, ref_step.workspace)
    torch.cuda.synchronize()
    assert np.max(np.abs(ref_step.lp_train.cpu().numpy()[:batch.T] - lp_ref_oracle)) <= LP_ATOL
    beta = 0.5
    step = ais.AisStep(batch.T, w.d, w.V, w.P, w.G, w.block, params=ais.default_params(beta_kl=beta))
    step.step(batch.H, batch.W, batch.tokens, batch.mask, batch.seq_offsets.cuda(), batch.rewards.cuda(),
              lp_ref=ref_step.lp_train)
    torch.cuda.synchronize()
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block,
                         lp_ref=lp_ref_oracle, beta_kl=beta)
    d = _compare_all(batch, step, ref, a)
    kl = oais.kl_term(ref["lp_train"], lp_ref_oracle, a["mask"], a["seq_offsets"], w.P, w.G)
    assert kl > 1e-4 and abs(d["kl_ref"] - kl) <= 2e-2 * kl + 1e-6
    # the term really moves the gradient: without it dH differs
    plain = _run_gpu(batch)
    assert _rel_fro(plain.dH.float().cpu().numpy(), step.dH.float().cpu().numpy()) > 1e-2


@pytest.mark.parametrize("case", ["tiny", "ragged"])
def test_per_tensor_fp8_scaling(case):
    """fp8_block = 0: one scale per tensor (the paper's own rollout setting).  Codes and the two scales bit-exact,
    the rest of the path within the usual tolerances."""
    ais = _lib()
    base = workloads.WORKLOADS["tiny"]
    w = workloads.scaled(base, block=0) if case == "tiny" else \
        workloads.scaled(base, block=0, d=384, V=1336, P=3, G=4, lengths="uniform:5:90", seed=81)
    batch = _to_cuda(workloads.make_batch(w, device="cpu"))
    step = _run_gpu(batch)
    a = workloads.to_numpy(batch)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, 0)
    T = batch.T
    assert np.array_equal(step.qH.cpu().numpy()[:T], ref["qH"]) and np.array_equal(step.qW.cpu().numpy(), ref["qW"])
    assert np.float32(step.sH[0, 0].item()).view(np.uint32) == np.float32(ref["sH"]).view(np.uint32)
    assert np.float32(step.sW[0, 0].item()).view(np.uint32) == np.float32(ref["sW"]).view(np.uint32)
    assert np.max(np.abs(step.lp_roll.cpu().numpy()[:T] - ref["lp_roll"])) <= LP_ATOL
    assert np.max(np.abs(step.lp_train.cpu().numpy()[:T] - ref["lp_train"])) <= LP_ATOL
    d = step.read_diag()
    assert abs(d["alpha"] - ref["diag"]["alpha"]) <= ALPHA_ATOL and int(step.status.item()) == 0
    dH = step.dH.float().cpu().numpy()[:T].astype(np.float64)
    assert _rel_fro(dH, ref["dH"]) <= DH_REL
    # degenerate input: an all-zero tensor gets scale 1 and zero codes
    z = torch.zeros(8, 128, dtype=torch.bfloat16, device="cuda")
    codes, scale = ais.quantize_fp8(z, 0)
    assert float(scale[0, 0]) == 1.0 and not codes.any()


@pytest.mark.parametrize("case", ["tiny", "ragged_chunked"])
def test_weight_gradient_on_gpu(case):
    """dW = U^T H against the oracle; with the minimum workspace the rows go through in 128-row passes that
    accumulate into dW; dw_accumulate adds a second micro-batch on top."""
    ais = _lib()
    base = workloads.WORKLOADS["tiny"]
    w = base if case == "tiny" else workloads.scaled(base, d=384, V=1336, P=3, G=4, lengths="uniform:20:90", seed=91)
    batch = _to_cuda(workloads.make_batch(w, device="cpu"))
    a, ref = _oracle(batch)
    step = ais.AisStep(batch.T, w.d, w.V, w.P, w.G, w.block, workspace_bytes_cap=(1 if case != "tiny" else None))
    offs, rew = batch.seq_offsets.cuda(), batch.rewards.cuda()
    dW = torch.full((w.V, w.d), 7.0, dtype=torch.float32, device="cuda")          # must be overwritten, not added to
    step.forward(batch.H, batch.W, batch.tokens, batch.mask)
    step.diagnose(batch.mask, offs, rew)
    step.backward(batch.H, batch.W, batch.tokens, batch.mask, offs, dW=dW)
    torch.cuda.synchronize()
    assert int(step.status.item()) == 0
    got = dW.cpu().numpy().astype(np.float64)
    assert _rel_fro(got, ref["dW"]) <= DH_REL
    dH = step.dH.float().cpu().numpy()[:batch.T].astype(np.float64)
    assert _rel_fro(dH, ref["dH"]) <= DH_REL
    step.backward(batch.H, batch.W, batch.tokens, batch.mask, offs, dW=dW, dw_accumulate=True)
    torch.cuda.synchronize()
    assert _rel_fro(dW.cpu().numpy().astype(np.float64), 2 * ref["dW"]) <= DH_REL


def test_padded_leading_dimensions_and_empty_batch_of_rows():
    """H and W as column slices of wider buffers (ldh, ldw > d): codes, dH and every tensor map follow the strides.
    Also T = 0: every entry point accepts it and alpha comes out 0 with the EMPTY flag."""
    ais = _lib()
    w = workloads.scaled(workloads.WORKLOADS["tiny"], d=256, V=776, lengths="uniform:20:70", seed=97)
    b = workloads.make_batch(w, device="cpu")
    a, ref = _oracle(b)
    ldh, ldw = w.d + 64, w.d + 128
    Hbig = torch.randn(b.T, ldh).to(torch.bfloat16).cuda()
    Wbig = torch.randn(w.V, ldw).to(torch.bfloat16).cuda()
    Hbig[:, :w.d] = b.H.cuda()
    Wbig[:, :w.d] = b.W.cuda()
    H, W = Hbig[:, :w.d], Wbig[:, :w.d]
    step = ais.AisStep(b.T, w.d, w.V, w.P, w.G, w.block, ldh=ldh, ldw=ldw)
    step.dH.fill_(3.0)
    dW = torch.zeros(w.V, w.d, dtype=torch.float32, device="cuda")
    step.forward(H, W, b.tokens.cuda(), b.mask.cuda())
    step.diagnose(b.mask.cuda(), b.seq_offsets.cuda(), b.rewards.cuda())
    step.backward(H, W, b.tokens.cuda(), b.mask.cuda(), b.seq_offsets.cuda(), dW=dW)
    torch.cuda.synchronize()
    batch = workloads.Batch(w, H, W, b.tokens.cuda(), b.mask.cuda(), b.seq_offsets, b.rewards)
    _compare_all(batch, step, ref, a)
    assert _rel_fro(dW.cpu().numpy().astype(np.float64), ref["dW"]) <= DH_REL
    # T = 0
    e = ais.AisStep(0, w.d, w.V, w.P, w.G, w.block)
    z8 = torch.zeros(1, dtype=torch.uint8, device="cuda")
    offs0 = torch.zeros(w.S + 1, dtype=torch.int32, device="cuda")
    e.step(torch.zeros(1, w.d, dtype=torch.bfloat16, device="cuda"), b.W.cuda(), torch.zeros(1, dtype=torch.int32, device="cuda"),
           z8, offs0, b.rewards.cuda())
    torch.cuda.synchronize()
    d = e.read_diag()
    assert d["alpha"] == 0.0 and d["status_flags"] & ais.FLAG_EMPTY and float(e.loss.item()) == 0.0


def test_whole_row_tiles_without_work_are_skipped_correctly():
    """A group with equal rewards (zero advantage over ~800 consecutive rows) and a long stretch of masked rows: the
    tensor-core passes skip such 128-row tiles; outputs must still be exact zeros there and right everywhere else,
    including dW, which contracts over the skipped rows."""
    ais = _lib()
    w = workloads.scaled(workloads.WORKLOADS["tiny"], d=256, V=776, P=3, G=4, lengths="const:200", seed=99)
    b = workloads.make_batch(w, device="cpu")
    b.rewards[4:8] = 1.0                                   # prompt 1: all responses rewarded -> A = 0 on rows 800..1599
    b.rewards[0:4] = torch.tensor([1.0, 0.0, 0.0, 1.0])
    b.mask[130:520] = 0                                    # rows 130..519 masked: tiles 2 and 3 hold no valid row
    batch = _to_cuda(b)
    a, ref = _oracle(batch)
    assert np.all(ref["c"][800:1600] == 0) and np.any(ref["c"][:130] != 0)
    step = ais.AisStep(batch.T, w.d, w.V, w.P, w.G, w.block)
    step.dH.fill_(5.0)
    dW = torch.full((w.V, w.d), 5.0, dtype=torch.float32, device="cuda")
    offs, rew = batch.seq_offsets.cuda(), batch.rewards.cuda()
    step.forward(batch.H, batch.W, batch.tokens, batch.mask)
    step.diagnose(batch.mask, offs, rew)
    step.backward(batch.H, batch.W, batch.tokens, batch.mask, offs, dW=dW)
    torch.cuda.synchronize()
    _compare_all(batch, step, ref, a)
    dH = step.dH.float().cpu().numpy()
    assert np.all(dH[800:1600] == 0) and np.all(dH[130:520] == 0)
    assert _rel_fro(dW.cpu().numpy().astype(np.float64), ref["dW"]) <= DH_REL


def test_on_policy_recovery_on_gpu():
    """Feeding the trainer's log-probs as the rollout's: rho == 1 exactly, alpha == 0 (Proposition 'on-policy recovery')."""
    ais = _lib()
    batch = _to_cuda(workloads.make_batch(workloads.WORKLOADS["tiny"], device="cpu"))
    step = _run_gpu(batch)
    offs, rew = batch.seq_offsets.cuda(), batch.rewards.cuda()
    ais.diagnostics(step.shape, step.params, step.lp_train, step.lp_train, batch.mask, offs, rew, step.adv, step.n_valid_seq,
                    step.rho, step.w_tilde, step.diag, step.workspace)
    torch.cuda.synchronize()
    d = step.read_diag()
    assert torch.all(step.rho == 1.0) and torch.all(step.w_tilde == 1.0)
    assert d["alpha"] == 0.0 and d["d_bar"] == 0.0 and d["alpha_ess"] == 1.0


def test_small_workspace_chunks_rows_and_is_deterministic():
    """The minimum workspace forces the backward pass through one 128-row chunk at a time; results do not change."""
    ais = _lib()
    w = workloads.scaled(workloads.WORKLOADS["tiny"], V=1024, lengths="uniform:60:120", seed=41)
    batch = _to_cuda(workloads.make_batch(w, device="cpu"))
    big = _run_gpu(batch)
    small = _run_gpu(batch, ws_cap=1)
    again = _run_gpu(batch)
    assert torch.equal(big.dH, small.dH)
    assert torch.equal(big.dH, again.dH) and torch.equal(big.lp_roll, again.lp_roll)
    assert big.read_diag() == again.read_diag()


def test_empty_batch_and_bad_tokens_flags():
    ais = _lib()
    w = workloads.scaled(workloads.WORKLOADS["tiny"], V=512, lengths="const:32", seed=51)
    batch = _to_cuda(workloads.make_batch(w, device="cpu"))
    batch.mask.zero_()
    step = _run_gpu(batch)
    d = step.read_diag()
    assert d["status_flags"] & ais.FLAG_EMPTY and d["alpha"] == 0.0 and float(step.loss.item()) == 0.0
    assert torch.all(step.dH == 0) and torch.all(step.lp_train == 0)
    batch.mask.fill_(1)
    batch.tokens[5] = w.V + 3
    batch.tokens[9] = -1
    step = _run_gpu(batch)
    assert int(step.status.item()) & ais.FLAG_TOKEN_RANGE
    assert float(step.lp_train[5]) == 0.0 and float(step.lp_roll[9]) == 0.0


def test_host_side_argument_errors():
    ais = _lib()
    batch = _to_cuda(workloads.make_batch(workloads.scaled(workloads.WORKLOADS["tiny"], V=512, lengths="const:32"), device="cpu"))
    step = ais.AisStep(batch.T, 256, 512, 2, 4, 128)
    with pytest.raises(ais.AisError):
        ais.logprob_fwd(step.shape, step.params, batch.H, batch.W, step.qH, step.sH, step.qW, step.sW, None, batch.mask,
                        step.lp_train, step.lse_train, step.lp_roll, step.lse_roll, step.status, step.workspace)
    with pytest.raises(ais.AisError):                        # workspace too small
        ais.loss_bwd(step.shape, step.params, batch.H, batch.W, batch.tokens, batch.mask, batch.seq_offsets.cuda(),
                     step.lse_train, step.lp_train, None, step.adv, step.w_tilde, step.dH, step.loss, step.diag, step.status,
                     step.workspace[:256])
    bad = ais.binding.make_shape(batch.T, 200, 512, 2, 4, 128)   # d not a multiple of 128
    with pytest.raises(ais.AisError):
        ais.diagnostics(bad, step.params, step.lp_train, step.lp_roll, batch.mask, batch.seq_offsets.cuda(),
                        batch.rewards.cuda(), step.adv, step.n_valid_seq, step.rho, step.w_tilde, step.diag, step.workspace)
    with pytest.raises(ais.AisError):
        ais.quantize_fp8(batch.H.cpu(), 128)
