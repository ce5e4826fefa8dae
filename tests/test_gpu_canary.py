"""Nothing is written outside the buffers the caller hands over: every output (and the workspace) is a view into a
larger allocation filled with a canary byte, with padding between the rows of the two-dimensional ones, and after a
whole pass of the path the canary is intact everywhere outside the documented extents while the results are the
bits an ordinary run gives."""

import numpy as np
import pytest
import torch

import workloads

pytestmark = pytest.mark.gpu

CANARY = 0xA5
GUARD = 4096                      # bytes before and after every buffer (keeps the 256-byte alignment of the allocation)


class Guarded:
    """A tensor of the given shape and row stride inside a canary-filled allocation."""

    def __init__(self, shape, dtype, ld=None, device="cuda"):
        es = torch.empty((), dtype=dtype).element_size()
        rows = shape[0] if len(shape) == 2 else 1
        cols = shape[-1]
        self.ld = ld if ld is not None else cols
        self.rows, self.cols, self.es = rows, cols, es
        body = rows * self.ld * es
        self.raw = torch.full((GUARD + body + GUARD,), CANARY, dtype=torch.uint8, device=device)
        inner = self.raw[GUARD:GUARD + body].view(dtype)
        self.t = inner.view(rows, self.ld)[:, :cols] if len(shape) == 2 else inner

    def check(self, name, rows_written=None):
        """Front and back guards, the padding columns of every row, and the rows past rows_written."""
        raw = self.raw.cpu().numpy()
        assert (raw[:GUARD] == CANARY).all(), name + ": bytes before the buffer were written"
        assert (raw[-GUARD:] == CANARY).all(), name + ": bytes after the buffer were written"
        body = raw[GUARD:-GUARD].reshape(self.rows, self.ld * self.es)
        assert (body[:, self.cols * self.es:] == CANARY).all(), name + ": row padding was written"
        if rows_written is not None:
            assert (body[rows_written:] == CANARY).all(), name + ": rows past the extent were written"


def _swap_in_guarded(step, T, d, V, S, ldh, extra_rows):
    """Replaces the step's outputs by guarded views; returns {name: (Guarded, rows the library may write)}."""
    g = {}
    for name in ("lp_train", "lse_train", "lp_roll", "lse_roll", "rho", "w_tilde"):
        g[name] = (Guarded((T + extra_rows,), torch.float32), None)
    g["adv"] = (Guarded((S,), torch.float32), None)
    g["n_valid_seq"] = (Guarded((S,), torch.int32), None)
    g["dH"] = (Guarded((T + extra_rows, d), torch.bfloat16, ld=ldh), T)
    g["qH"] = (Guarded((T + extra_rows, step.qH.shape[1]), torch.uint8, ld=step.qH.stride(0)), T)
    g["qW"] = (Guarded(tuple(step.qW.shape), torch.uint8, ld=step.qW.stride(0)), None)
    g["sH"] = (Guarded(tuple(step.sH.shape), step.sH.dtype, ld=step.sH.stride(0) if step.sH.dim() == 2 else None), None)
    g["sW"] = (Guarded(tuple(step.sW.shape), step.sW.dtype, ld=step.sW.stride(0) if step.sW.dim() == 2 else None), None)
    g["workspace"] = (Guarded((step.workspace.numel(),), torch.uint8), None)
    for name, (buf, _) in g.items():
        setattr(step, name, buf.t)
    return g


CASES = {
    # name: (workload overrides, fp8 block, W layout is [d, V], row stride padding of H / dH)
    "block128_ragged": (dict(d=512, V=1336, P=2, G=4, lengths="uniform:40:117", seed=81), 128, False, 64),
    "block32_dv_head": (dict(d=256, V=776, P=2, G=3, lengths="uniform:20:150", seed=82), 32, True, 16),
    "mxfp8": (dict(d=256, V=1040, P=1, G=4, lengths="uniform:33:99", seed=83), "mx8", False, 0),
    "three_rows": (dict(d=128, V=264, P=1, G=2, lengths="uniform:1:2", seed=84), 128, False, 0),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_no_write_outside_the_callers_buffers(case):
    import paper_2605_13907_b200 as ais
    over, block, dv, pad = CASES[case]
    block = ais.FP8_MX32 if block == "mx8" else block
    w = workloads.scaled(workloads.WORKLOADS["tiny"], block=block, **over)
    b = workloads.make_batch(w, device="cpu")
    T, S = b.T, w.P * w.G
    ldh = w.d + pad
    H = Guarded((T, w.d), torch.bfloat16, ld=ldh)
    H.t.copy_(b.H)
    Wsrc = b.W.t().contiguous() if dv else b.W
    W = Wsrc.cuda()
    layout = ais.W_DV if dv else ais.W_VD
    tok, msk, offs, rew = b.tokens.cuda(), b.mask.cuda(), b.seq_offsets.cuda(), b.rewards.cuda()

    def run(guarded):
        step = ais.AisStep(T, w.d, w.V, w.P, w.G, block, ldh=ldh, w_layout=layout)
        g = _swap_in_guarded(step, T, w.d, w.V, S, ldh, extra_rows=5) if guarded else None
        dW = Guarded(tuple(Wsrc.shape), torch.float32, ld=Wsrc.shape[1] + 4) if guarded else \
            Guarded(tuple(Wsrc.shape), torch.float32)
        step.step(H.t, W, tok, msk, offs, rew)
        step.backward(H.t, W, tok, msk, offs, dW=dW.t)
        torch.cuda.synchronize()
        assert int(step.status.item()) == 0
        return step, g, dW

    plain, _, dW_plain = run(False)
    step, g, dW = run(True)
    for name, (buf, rows) in g.items():
        buf.check(name, rows)
    dW.check("dW")
    H.check("H (input)")
    # vectors: exactly T elements belong to the library
    for name in ("lp_train", "lse_train", "lp_roll", "lse_roll", "rho", "w_tilde"):
        tail = g[name][0].raw[GUARD + 4 * T:GUARD + 4 * (T + 5)].cpu().numpy()
        assert (tail == CANARY).all(), name + ": elements past T were written"
    # and the views changed nothing in the results
    for name in ("lp_train", "lse_train", "lp_roll", "lse_roll", "rho", "w_tilde"):
        assert torch.equal(getattr(step, name)[:T], getattr(plain, name)[:T]), name
    assert torch.equal(step.dH[:T], plain.dH[:T])
    assert torch.equal(dW.t, dW_plain.t)
    dg, dp = step.read_diag(), plain.read_diag()
    assert all(dg[k] == dp[k] or (dg[k] != dg[k] and dp[k] != dp[k]) for k in dp), (dg, dp)
    assert np.isfinite(step.dH[:T].float().cpu().numpy()).all()


@pytest.mark.parametrize("kind", ["block64", "tensor", "mx8", "mx4", "cols128"])
def test_quantisers_stay_inside_their_outputs(kind):
    import paper_2605_13907_b200 as ais
    g = torch.Generator().manual_seed(5)
    rows, cols = (384, 200) if kind == "cols128" else (203, 512)      # cols128: x is [K, N], blocks run down the columns
    ld = cols + 8
    x = Guarded((rows, cols), torch.bfloat16, ld=ld)
    x.t.copy_(torch.randn(rows, cols, generator=g).to(torch.bfloat16))
    if kind == "cols128":
        codes = Guarded((cols, rows), torch.uint8, ld=rows + 16)
        scales = Guarded((rows // 128, 208), torch.float32, ld=212)
        ais.quantize_fp8_cols(x.t, 128, codes.t, scales.t)
        ref_c, ref_s = ais.quantize_fp8_cols(x.t.contiguous(), 128)
        same_s = torch.equal(scales.t[:, :cols], ref_s[:, :cols])
    elif kind in ("mx8", "mx4"):
        fp4 = kind == "mx4"
        block = ais.FP4_MX32 if fp4 else ais.FP8_MX32
        cw = cols // 2 if fp4 else cols
        codes = Guarded((rows + 3, cw), torch.uint8, ld=cw + 32)
        scales = Guarded((ais.mx_scale_bytes(rows, cols),), torch.uint8)
        ais.quantize_fp8(x.t, block, codes.t[:rows], scales.t)
        ref_c, ref_s = ais.quantize_fp8(x.t.contiguous(), block)
        same_s = torch.equal(scales.t, ref_s)
    else:
        block = 0 if kind == "tensor" else 64
        codes = Guarded((rows + 3, cols), torch.uint8, ld=cols + 24)
        scales = Guarded((1, 4), torch.float32) if block == 0 else Guarded((cols // block, 204), torch.float32, ld=208)
        ais.quantize_fp8(x.t, block, codes.t[:rows], scales.t)
        ref_c, ref_s = ais.quantize_fp8(x.t.contiguous(), block)
        same_s = torch.equal(scales.t[:, :1], ref_s[:, :1]) if block == 0 else torch.equal(scales.t[:, :rows], ref_s[:, :rows])
    torch.cuda.synchronize()
    codes.check("codes", None if kind == "cols128" else rows)
    scales.check("scales")
    x.check("x (input)")
    assert same_s
    assert torch.equal(codes.t[:ref_c.shape[0]], ref_c)


def test_row_scatter_and_gather_stay_inside_their_outputs():
    import paper_2605_13907_b200 as ais
    g = torch.Generator().manual_seed(6)
    S, L, width = 5, 37, 96
    T = S * L
    mask = (torch.rand(T, generator=g) < 0.6).to(torch.uint8)
    offs = torch.arange(0, T + 1, L, dtype=torch.int32)
    comp = ais.RowCompaction(mask.cuda(), offs.cuda())
    n = int(mask.sum())
    assert comp.n == n
    src = torch.randn(T, width, generator=g).to(torch.bfloat16).cuda()
    packed = Guarded((n + 4, width), torch.bfloat16, ld=width + 8)
    comp.gather_rows(src, packed.t)
    torch.cuda.synchronize()
    packed.check("packed rows", n)
    assert torch.equal(packed.t[:n], src[mask.bool().cuda()])
    back = Guarded((T, width), torch.bfloat16, ld=width + 8)
    comp.scatter_rows(packed.t, back.t)
    torch.cuda.synchronize()
    back.check("scattered rows")
    m = mask.bool().cuda()
    assert torch.equal(back.t[m], src[m]) and torch.all(back.t[~m] == 0)
