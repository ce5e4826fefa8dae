"""Microscaling FP8 rollout pass (power-of-two E8M0 scale per 32 elements, applied by the block-scaled tensor-core
instruction) against the oracle: codes and packed scale bytes bit-exact, log-probs and the rest of the path within the
usual tolerances."""

import numpy as np
import pytest
import torch

import abi_layout
import row_sampling
import workloads
from oracle import ais as oais
from oracle import e4m3

pytestmark = pytest.mark.gpu

LP_ATOL = 1e-2
ALPHA_ATOL = 1e-3
DH_REL = 1e-2


def _cuda(b):
    return workloads.Batch(b.workload, b.H.cuda(), b.W.cuda(), b.tokens.cuda(), b.mask.cuda(), b.seq_offsets, b.rewards)


def test_mx_quantiser_bit_exact():
    import paper_2605_13907_b200 as ais
    g = torch.Generator().manual_seed(11)
    rows, cols = 301, 384                                   # three row chunks (the last ragged), three chunk columns
    x = torch.randn(rows, cols, generator=g) * torch.exp(torch.randn(rows, 1, generator=g) * 4)
    x[5] = 0.0                                              # zero blocks -> neutral scale
    x[6, :32] = 1e-39                                       # bf16 subnormals: scale code clamps at 0
    x[7, 40] = 3.0e38                                       # largest exponents
    x[8, :64] = torch.tensor([480.0, -500.0, 447.0, 449.0] * 16)        # the (448, 512) clipping band
    x[9] = -0.0
    xb = x.to(torch.bfloat16)
    codes, packed = ais.quantize_fp8(xb.cuda(), ais.FP8_MX32)
    torch.cuda.synchronize()
    ref_c, ref_s = e4m3.quantize_mx(xb.float().numpy())
    assert np.array_equal(codes.cpu().numpy(), ref_c)
    assert packed.numel() == abi_layout.mx_scale_bytes(rows, cols) == ais.mx_scale_bytes(rows, cols)
    got = packed.cpu().numpy()
    assert np.array_equal(abi_layout.unpack_mx_scales(got, rows, cols), ref_s)
    assert np.all(abi_layout.mx_scale_padding(got, rows, cols) == 127)


@pytest.mark.parametrize("case", ["tiny", "ragged"])
def test_mx_rollout_path(case):
    import paper_2605_13907_b200 as ais
    base = workloads.WORKLOADS["tiny"]
    w = workloads.scaled(base, block=ais.FP8_MX32) if case == "tiny" else \
        workloads.scaled(base, block=ais.FP8_MX32, d=384, V=1336, P=3, G=4, lengths="uniform:5:90", seed=83)
    b = _cuda(workloads.make_batch(w, device="cpu"))
    step = ais.AisStep(b.T, w.d, w.V, w.P, w.G, w.block)
    step.step(b.H, b.W, b.tokens, b.mask, b.seq_offsets.cuda(), b.rewards.cuda())
    torch.cuda.synchronize()
    a = workloads.to_numpy(b)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, oais.MX32)
    T = b.T
    assert int(step.status.item()) == 0
    assert np.array_equal(step.qH.cpu().numpy()[:T], ref["qH"]) and np.array_equal(step.qW.cpu().numpy(), ref["qW"])
    assert np.array_equal(abi_layout.unpack_mx_scales(step.sW.cpu().numpy(), w.V, w.d), ref["sW"])
    assert np.array_equal(abi_layout.unpack_mx_scales(step.sH.cpu().numpy(), T, w.d), ref["sH"])
    err = np.abs(step.lp_roll.cpu().numpy()[:T] - ref["lp_roll"])
    assert err.max() <= LP_ATOL, err.max()
    assert err.max() <= 1e-4                                 # power-of-two scales are exact: only fp32 accumulation differs
    assert np.max(np.abs(step.lp_train.cpu().numpy()[:T] - ref["lp_train"])) <= LP_ATOL
    d = step.read_diag()
    assert abs(d["alpha"] - ref["diag"]["alpha"]) <= ALPHA_ATOL
    assert abs(d["d_bar"] - ref["diag"]["d_bar"]) <= 1e-4
    dH = step.dH.float().cpu().numpy()[:T].astype(np.float64)
    assert np.linalg.norm(dH - ref["dH"]) <= DH_REL * np.linalg.norm(ref["dH"])


@pytest.mark.parametrize("fmt", ["fp8", "fp4"])
def test_mx_fullsize_sampled_rows(fmt):
    """qwen3_8b shape in the launch configuration the benchmark's --fp8-mx / --fp4-mx variants time: all of W's codes and
    scale bytes bit-exact, and the rollout log-probs of a seeded sample of rows against the oracle over the whole
    vocabulary."""
    import paper_2605_13907_b200 as ais
    fp4 = fmt == "fp4"
    quant = e4m3.quantize_mxfp4 if fp4 else e4m3.quantize_mx
    dequant = e4m3.dequantize_mxfp4 if fp4 else e4m3.dequantize_mx
    plain = abi_layout.unpack_fp4_pairs if fp4 else (lambda c: c)
    w = workloads.scaled(workloads.WORKLOADS["qwen3_8b"], block=ais.FP4_MX32 if fp4 else ais.FP8_MX32)
    batch = workloads.make_batch(w, device="cuda")
    T = batch.T
    step = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block, want_grad=False)
    step.forward(batch.H, batch.W, batch.tokens, batch.mask)
    torch.cuda.synchronize()
    assert int(step.status.item()) == 0
    rows = row_sampling.sample_rows(batch.seq_offsets.numpy(), T, 1024, np.random.default_rng(5))     # >= 8 of each sequence
    assert row_sampling.rows_per_sequence(rows, batch.seq_offsets.numpy()).min() >= 8
    Hs = batch.H[torch.as_tensor(rows, device="cuda")].float().cpu().numpy().astype(np.float64)
    qHs, sHs = quant(Hs)
    assert np.array_equal(plain(step.qH.cpu().numpy()[rows]), qHs)
    Hq = dequant(qHs, sHs)
    sH_gpu = abi_layout.unpack_mx_scales(step.sH.cpu().numpy(), T, w.d)
    assert np.array_equal(sH_gpu[rows], sHs)
    qW_gpu = step.qW.cpu().numpy()
    sW_gpu = abi_layout.unpack_mx_scales(step.sW.cpu().numpy(), w.V, w.d)
    z = np.empty((len(rows), w.V))
    CH = 4096                                               # a multiple of 256: whole scale groups per piece
    for v0 in range(0, w.V, CH):
        Wc = batch.W[v0:v0 + CH].float().cpu().numpy().astype(np.float64)
        qc, sc = quant(Wc)
        assert np.array_equal(plain(qW_gpu[v0:v0 + CH]), qc), v0
        n = Wc.shape[0]
        assert np.array_equal(sW_gpu[v0:v0 + n], sc), v0
        z[:, v0:v0 + n] = Hq @ dequant(qc, sc).T
    tok = batch.tokens.cpu().numpy()[rows]
    msk = batch.mask.cpu().numpy()[rows]
    lp_ref, _ = oais.log_softmax_gather(z, tok, msk)
    got = step.lp_roll.cpu().numpy()[rows]
    assert np.max(np.abs(got - lp_ref)) <= 1e-3, np.max(np.abs(got - lp_ref))


# --------------------------------------------------------------------------- FP4 elements
def test_mxfp4_quantiser_bit_exact():
    import paper_2605_13907_b200 as ais
    g = torch.Generator().manual_seed(12)
    rows, cols = 301, 512
    x = torch.randn(rows, cols, generator=g) * torch.exp(torch.randn(rows, 1, generator=g) * 4)
    x[5] = 0.0
    x[6, :32] = 1e-39
    x[7, 40] = 3.0e38
    x[8, :64] = torch.tensor([7.0, -6.5, 5.0, 2.5, 0.25, 0.75, 1.25, 3.5] * 8)      # clipping band and every tie
    x[9] = -0.0
    xb = x.to(torch.bfloat16)
    codes, packed = ais.quantize_fp8(xb.cuda(), ais.FP4_MX32)
    torch.cuda.synchronize()
    ref_c, ref_s = e4m3.quantize_mxfp4(xb.float().numpy())
    assert codes.shape == (rows, cols // 2)
    assert np.array_equal(abi_layout.unpack_fp4_pairs(codes.cpu().numpy()), ref_c)
    got = packed.cpu().numpy()
    assert np.array_equal(abi_layout.unpack_mx_scales(got, rows, cols), ref_s)
    assert np.all(abi_layout.mx_scale_padding(got, rows, cols) == 127)


@pytest.mark.parametrize("case", ["tiny", "ragged"])
def test_mxfp4_rollout_path(case):
    """FP4 rollouts are far from the trainer (d_bar of order 1), which is the regime where the mixing coefficient
    saturates; what is checked is parity with the oracle on the same codes."""
    import paper_2605_13907_b200 as ais
    base = workloads.WORKLOADS["tiny"]
    w = workloads.scaled(base, block=ais.FP4_MX32) if case == "tiny" else \
        workloads.scaled(base, block=ais.FP4_MX32, d=512, V=1336, P=3, G=4, lengths="uniform:5:90", seed=84)
    b = _cuda(workloads.make_batch(w, device="cpu"))
    step = ais.AisStep(b.T, w.d, w.V, w.P, w.G, w.block)
    step.step(b.H, b.W, b.tokens, b.mask, b.seq_offsets.cuda(), b.rewards.cuda())
    torch.cuda.synchronize()
    a = workloads.to_numpy(b)
    ref = oais.full_path(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, oais.MXFP4)
    T = b.T
    assert int(step.status.item()) == 0
    assert np.array_equal(abi_layout.unpack_fp4_pairs(step.qH.cpu().numpy()[:T]), ref["qH"])
    assert np.array_equal(abi_layout.unpack_fp4_pairs(step.qW.cpu().numpy()), ref["qW"])
    assert np.array_equal(abi_layout.unpack_mx_scales(step.sW.cpu().numpy(), w.V, w.d), ref["sW"])
    err = np.abs(step.lp_roll.cpu().numpy()[:T] - ref["lp_roll"])
    assert err.max() <= 1e-3, err.max()
    d = step.read_diag()
    assert abs(d["alpha"] - ref["diag"]["alpha"]) <= ALPHA_ATOL
    assert abs(d["d_bar"] - ref["diag"]["d_bar"]) <= 1e-3 * max(1.0, ref["diag"]["d_bar"])
    dH = step.dH.float().cpu().numpy()[:T].astype(np.float64)
    assert np.linalg.norm(dH - ref["dH"]) <= DH_REL * np.linalg.norm(ref["dH"])
