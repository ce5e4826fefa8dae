"""Seeded synthetic GRPO batches shaped like the paper's workloads.

This module only manufactures inputs (hidden states, LM-head weights, sampled
tokens, masks, sequence offsets, rewards).  It contains none of the method's
arithmetic and is the one module shared by the CPU oracle's tests and the GPU
library's tests and benchmark.  The batches stand in for the paper's models and
datasets (Qwen3-8B and LLaDA-8B LM-head shapes, G responses per prompt, long
chain-of-thought length mixes); nothing is read from disk or network.

Token ids are drawn from the softmax of the bf16 logits at temperature 1 with
the Gumbel-max construction (argmax of logits plus Gumbel noise), computed with
plain torch ops in row chunks.
"""

from __future__ import annotations

from dataclasses import dataclass, replace
import math

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    d: int
    V: int
    P: int                 # prompts
    G: int                 # responses per prompt
    block: int             # FP8 block size along d
    lengths: str           # "const:L" | "uniform:lo:hi" | "geometric:mean:max"
    reward_p: float        # rewards ~ Bernoulli(reward_p) per response
    w_std: float           # std of the LM-head weights
    rmsnorm: bool          # hidden states normalised to unit RMS per row
    mask_mode: str = "none"   # "none" | "llada" (per-sequence mask ratio over response positions)
    vocab_chunk: int = 0
    seed: int = 0

    @property
    def S(self) -> int:
        return self.P * self.G


WORKLOADS = {
    # d=256, V=1024, 2 prompts x 4 responses x 64 tokens, no padding
    "tiny": Workload("tiny", d=256, V=1024, P=2, G=4, block=128, lengths="const:64", reward_p=0.5,
                     w_std=1.0 / 16.0, rmsnorm=False, seed=1001),
    # Qwen3-8B LM-head shape, 8 prompts x 8 responses, lengths uniform in [256, 2048]
    "qwen3_8b": Workload("qwen3_8b", d=4096, V=151936, P=8, G=8, block=128, lengths="uniform:256:2048",
                         reward_p=0.3, w_std=0.02, rmsnorm=True, seed=1002),
    # long chain-of-thought: 32 x 16, censored geometric lengths (mean 3000, max 8192), 16k vocab chunks
    "long_cot": Workload("long_cot", d=4096, V=151936, P=32, G=16, block=128, lengths="geometric:3000:8192",
                         reward_p=0.2, w_std=0.02, rmsnorm=True, vocab_chunk=16384, seed=1003),
    # large-vocabulary stress shape with FP8 block 32
    "large_vocab": Workload("large_vocab", d=5120, V=262144, P=16, G=8, block=32, lengths="uniform:1024:4096",
                            reward_p=0.3, w_std=0.02, rmsnorm=True, seed=1004),
    # LLaDA-8B shape: 512 response positions per sequence, a random subset of them masked (= valid)
    "llada_8b": Workload("llada_8b", d=4096, V=126464, P=16, G=8, block=128, lengths="const:512",
                         reward_p=0.4, w_std=0.02, rmsnorm=True, mask_mode="llada", seed=1005),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (reduced sizes for CPU tests)."""
    return replace(w, **kw)


def draw_lengths(w: Workload, rng: np.random.Generator) -> np.ndarray:
    kind, *args = w.lengths.split(":")
    S = w.S
    if kind == "const":
        return np.full(S, int(args[0]), dtype=np.int64)
    if kind == "uniform":
        lo, hi = int(args[0]), int(args[1])
        return rng.integers(lo, hi + 1, size=S, dtype=np.int64)
    if kind == "geometric":
        mean, mx = float(args[0]), int(args[1])
        return np.minimum(rng.geometric(1.0 / mean, size=S), mx).astype(np.int64)
    raise ValueError(w.lengths)


@dataclass
class Batch:
    workload: Workload
    H: torch.Tensor            # [T, d] bf16
    W: torch.Tensor            # [V, d] bf16 (one row per vocabulary entry)
    tokens: torch.Tensor       # [T] int32
    mask: torch.Tensor         # [T] uint8
    seq_offsets: torch.Tensor  # [S+1] int32 (host)
    rewards: torch.Tensor      # [S] float32 (host)

    @property
    def T(self) -> int:
        return self.H.shape[0]

    @property
    def n_valid(self) -> int:
        return int(self.mask.sum().item())


def sample_tokens(H: torch.Tensor, W: torch.Tensor, gen: torch.Generator, rows_per_chunk: int | None = None) -> torch.Tensor:
    """y_t ~ softmax(H_t W^T) via Gumbel-max, chunked over rows so the [rows, V] block stays small."""
    T, V = H.shape[0], W.shape[0]
    dev = H.device
    if rows_per_chunk is None:
        rows_per_chunk = max(1, min(T, (1 << 28) // max(V, 1)))
    out = torch.empty(T, dtype=torch.int32, device=dev)
    Wc = W if dev.type == "cuda" else W.float()
    for r0 in range(0, T, rows_per_chunk):
        h = H[r0:r0 + rows_per_chunk]
        z = (h @ Wc.T).float() if dev.type == "cuda" else h.float() @ Wc.T
        u = torch.rand(z.shape, generator=gen, device=dev, dtype=torch.float32)
        u.clamp_(min=1e-20, max=1.0 - 1e-7)
        z -= torch.log(-torch.log(u))
        out[r0:r0 + rows_per_chunk] = torch.argmax(z, dim=1).to(torch.int32)
    return out


def make_batch(w: Workload, device: str | torch.device = "cpu") -> Batch:
    """Build the batch for a workload.  Structure (lengths, masks, rewards) always comes from a numpy
    generator on the host; the dense tensors come from a torch generator on ``device``."""
    rng = np.random.default_rng(w.seed)
    lengths = draw_lengths(w, rng)
    offsets = np.zeros(w.S + 1, dtype=np.int64)
    np.cumsum(lengths, out=offsets[1:])
    T = int(offsets[-1])
    rewards = (rng.random(w.S) < w.reward_p).astype(np.float32)

    mask = np.ones(T, dtype=np.uint8)
    if w.mask_mode == "llada":
        mask[:] = 0
        for s in range(w.S):
            L = int(lengths[s])
            ratio = 1.0 - rng.random()                       # uniform on (0, 1]
            k = max(1, min(L, math.ceil(ratio * L)))
            pos = rng.choice(L, size=k, replace=False)
            mask[offsets[s] + pos] = 1

    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed)
    H = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
    rows = max(1, (1 << 26) // w.d)
    for r0 in range(0, T, rows):
        h = torch.randn(min(rows, T - r0), w.d, generator=gen, device=dev, dtype=torch.float32)
        if w.rmsnorm:
            h = h * torch.rsqrt(h.pow(2).mean(dim=1, keepdim=True) + 1e-6)
        H[r0:r0 + rows] = h.to(torch.bfloat16)
    W = torch.empty(w.V, w.d, dtype=torch.bfloat16, device=dev)
    for r0 in range(0, w.V, rows):
        x = torch.randn(min(rows, w.V - r0), w.d, generator=gen, device=dev, dtype=torch.float32)
        W[r0:r0 + rows] = (x * w.w_std).to(torch.bfloat16)
    tokens = sample_tokens(H, W, gen)
    return Batch(w, H, W, tokens, torch.from_numpy(mask).to(dev),
                 torch.from_numpy(offsets.astype(np.int32)), torch.from_numpy(rewards))


def to_numpy(b: Batch, rows=None) -> dict:
    """Host copies for the oracle: exact bf16 values as float64 arrays.  ``rows`` selects a subset of token rows."""
    if rows is None:
        H = b.H
        tok, msk = b.tokens, b.mask
    else:
        idx = torch.as_tensor(rows, device=b.H.device, dtype=torch.long)
        H = b.H[idx]
        tok, msk = b.tokens[idx], b.mask[idx]
    return dict(H=H.float().cpu().numpy().astype(np.float64),
                W=b.W.float().cpu().numpy(),
                tokens=tok.cpu().numpy().astype(np.int64),
                mask=msk.cpu().numpy().astype(np.uint8),
                seq_offsets=b.seq_offsets.numpy().astype(np.int64),
                rewards=b.rewards.numpy().astype(np.float64))
