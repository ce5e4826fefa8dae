#!/usr/bin/env python
"""Benchmark of the AIS-GRPO LM-head path on B200.

One step = one pass of the whole path over one synthetic batch: FP8 quantisation of H and W, trainer (bf16)
and rollout (FP8) log-probabilities, diagnostics / alpha / rectification weights, loss and dH.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload qwen3_8b] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is valid tokens per second over all ranks with inputs resident in HBM;
`e2e` is the same through host buffers (pinned host -> device copies of the step's inputs and a device -> host
read of loss, diagnostics and dH inside the timed region).  `--impl reference` times the float64 CPU oracle
on a bounded sample instead.

With --gpus N > 1 the script starts N ranks of itself, one per GPU (torch.distributed.run, NCCL); started under
torchrun already (RANK / WORLD_SIZE in the environment) it runs as the rank it is given.  Every rank owns its own
prompts (weak scaling), the LM head is replicated, and the only exchange is the all-reduce of the 12 moments behind
the mixing coefficient.
"""

from __future__ import annotations

import argparse
import importlib
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

# DRAM bytes (read + write) of one launch of each tensor-core kernel on a bench workload, from a one-pass profiler capture
# of the full-size step (the two DRAM byte counters alone need no replay): the two backward kernels are taken together
# because one call enqueues both.  None for workloads, variants and kernels that were not captured.
TRAFFIC = {
    "qwen3_8b": {"fwd_train_bf16": 19.28e9, "fwd_roll_fp8": 9.95e9, "bwd": (31.03e9 + 21.50e9) + (66.69e9 + 0.57e9)},
}
METRIC = "AIS-corrected fwd+bwd tokens/sec"
UNIT = "tokens/s"
NOMINAL = {"bf16_tflops": 2250.0, "fp8_tflops": 4500.0, "fp4_tflops": 9000.0, "hbm_gbs": 7700.0}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"], bf16_tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def _workload_text(w) -> str:
    return (f"{w.name}: d={w.d} V={w.V} P={w.P} G={w.G} block={w.block} lengths={w.lengths}, "
            "sequences packed back to back (T = sum of lengths)" + (", scattered per-sequence masks" if w.mask_mode != "none" else ""))


# ------------------------------------------------------------------------------------------ CPU oracle, stage by stage
def oracle_stages(H, W, tokens, mask, offs, rewards, P, G, block):
    """The oracle's stages as they stand, one after the other, each timed: quantiser emulation, trainer log-probs,
    rollout log-probs, ratios / diagnostics / rectification, loss and dH (no dW: the timed GPU step has none)."""
    from oracle import ais as oais
    from oracle import e4m3
    t = {}
    t0 = time.perf_counter()
    qH, sH = e4m3.quantize_blocks(H, block)
    qW, sW = e4m3.quantize_blocks(W, block)
    t["quantiser_emulation"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    lp_t, _ = oais.logprob_train(H, W, tokens, mask)
    t["trainer_logprob"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    Hq = e4m3.dequantize_blocks(qH, sH, block)
    Wq = e4m3.dequantize_blocks(qW, sW, block)
    lp_r, _ = oais.log_softmax_gather(oais.logits(Hq, Wq), tokens, mask)
    t["rollout_logprob"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    p = oais.Params()
    adv = oais.advantages(rewards, G)
    adv_tok = adv[oais.seq_ids(offs, len(mask))]
    _, _, wbar = oais.ratios(lp_t, lp_r, mask, p.C)
    diag = oais.diagnostics(lp_t, lp_r, mask, adv_tok, p)
    w_tilde = oais.rectify(wbar, diag["alpha"], mask)
    t["diagnostics"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    _, c = oais.loss_and_coeff(lp_t, lp_t, mask, offs, adv, w_tilde, P, G, p.clip_eps)
    oais.grad_hidden(H, W, tokens, c)
    t["loss_and_dH"] = time.perf_counter() - t0
    return t


def oracle_sample(w: workloads.Workload, tokens_n: int = 192, vocab_n: int = 32768):
    """Times the oracle on `tokens_n` rows against `vocab_n` vocabulary rows of the workload's shape and scales the
    rate to the full vocabulary (every stage of the path but the O(T) reductions costs O(V) per token)."""
    vocab_n = min(vocab_n, w.V)
    rng = np.random.default_rng(w.seed)
    G, P = w.G, 1
    S = P * G
    per = max(1, tokens_n // S)
    T = per * S
    H = torch.randn(T, w.d, generator=torch.Generator().manual_seed(w.seed))
    if w.rmsnorm:
        H = H * torch.rsqrt(H.pow(2).mean(dim=1, keepdim=True) + 1e-6)
    H = H.to(torch.bfloat16).float().numpy().astype(np.float64)
    W = (torch.randn(vocab_n, w.d, generator=torch.Generator().manual_seed(w.seed + 1)) * w.w_std)
    W = W.to(torch.bfloat16).float().numpy()
    tokens = rng.integers(0, vocab_n, T)
    mask = np.ones(T, np.uint8)
    offs = np.arange(S + 1) * per
    rewards = (rng.random(S) < w.reward_p).astype(np.float64)
    block = w.block if w.block > 0 else 128
    stages = oracle_stages(H, W, tokens, mask, offs, rewards, P, G, block)
    dt = sum(stages.values())
    scale = vocab_n / w.V
    return dict(rate=T / dt * scale, seconds=dt, stages_s=stages,
                rate_without_quantiser=T / (dt - stages["quantiser_emulation"]) * scale,
                sample=f"{T} tokens x d={w.d} x {vocab_n} of V={w.V} vocabulary rows, rate scaled by {vocab_n}/{w.V}")


def oracle_tiny_full():
    """The whole `tiny` workload through the oracle's stages (512 tokens, d=256, V=1024): no sampling, no scaling."""
    w = workloads.WORKLOADS["tiny"]
    a = workloads.to_numpy(workloads.make_batch(w, device="cpu"))
    stages = oracle_stages(a["H"], a["W"], a["tokens"], a["mask"], a["seq_offsets"], a["rewards"], w.P, w.G, w.block)
    dt = sum(stages.values())
    return dict(value=len(a["mask"]) / dt, unit=UNIT, seconds=dt, stages_s=stages, sample="tiny in full: 512 tokens, d=256, V=1024")


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def cpu_baseline_object(w) -> dict:
    s = oracle_sample(w)
    return {"value": s["rate"], "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": s["sample"],
            "seconds": s["seconds"], "stages_s": s["stages_s"], "value_without_quantiser_emulation": s["rate_without_quantiser"],
            "note": "float64 numpy oracle as it stands; stages timed one after the other; loss_and_dH forms no dW",
            "tiny_full": oracle_tiny_full()}


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))


def _ld_u(V: int) -> int:
    return (V + 63) // 64 * 64


# ------------------------------------------------------------------------------------------ ranks
def rank_env():
    """(rank, world, local rank) as torchrun gives them; (0, 1, 0) for a plain start."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def needs_launch(args) -> bool:
    """--gpus N > 1 without a torchrun environment: this process is the launcher, not a rank."""
    return args.gpus > 1 and "WORLD_SIZE" not in os.environ


def launch_ranks(args, argv) -> int:
    """Starts args.gpus ranks of this script on this node, one per GPU, and returns their exit code.  Rank 0's JSON
    line goes to this process's stdout unchanged."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--local-addr", "127.0.0.1", os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def reduce_over_ranks(local: dict, world: int, device) -> dict:
    """Whole-job figures from the per-rank ones: times are the MAX over ranks, token counts the SUM."""
    if world == 1:
        return dict(ms_per_step=local["ms_per_step"], e2e_ms=local["e2e_ms"], tokens_all=float(local["n_valid"]))
    import torch.distributed as dist
    stats = torch.tensor([local["ms_per_step"], local["e2e_ms"], float(local["n_valid"])], dtype=torch.float64, device=device)
    mx = stats.clone()
    dist.all_reduce(mx, op=dist.ReduceOp.MAX)
    sm = stats.clone()
    dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return dict(ms_per_step=float(mx[0]), e2e_ms=float(mx[1]), tokens_all=float(sm[2]))


def rank_workload(args, rank: int):
    """The workload of one rank: the named workload with the rank's own seed (its own prompts), plus the variant flags."""
    base = workloads.WORKLOADS[args.workload]
    w = workloads.scaled(base, seed=base.seed + 7919 * rank)
    if args.prompts:
        w = workloads.scaled(w, P=args.prompts)                       # reduced case for profiler captures
    if args.fp8_per_tensor:
        w = workloads.scaled(w, block=0)                              # variant: one FP8 scale per tensor
    if args.fp8_mx:
        w = workloads.scaled(w, block=-32)                            # variant: microscaling, E8M0 scale per 32 elements
    if args.fp4_mx:
        w = workloads.scaled(w, block=-4)                             # variant: microscaling FP4 (E2M1) rollout pass
    return w


# ------------------------------------------------------------------------------------------ one rank's measurement
def measure_rank(args, rank: int, world: int, local: int) -> dict:
    """Everything one rank measures on its GPU: the timed steps, the end-to-end steps, clocks, and (rank 0, one GPU) the
    streaming kernels alone.  Returns plain numbers; nothing here talks to other ranks except the step's own
    all-reduce of the moments."""
    import torch.distributed as dist
    import paper_2605_13907_b200 as ais

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    w = rank_workload(args, rank)
    batch = workloads.make_batch(w, device=dev)
    if args.compact:
        # scattered masks: pack the valid rows once per batch (inside the step for the end-to-end figure) and run on those
        rc0 = ais.RowCompaction(batch.mask, batch.seq_offsets.to(dev), n_packed=batch.n_valid)
        packed = workloads.Batch(w, rc0.gather_rows(batch.H), batch.W, rc0.gather(batch.tokens),
                                 torch.ones(rc0.n, dtype=torch.uint8, device=dev), rc0.packed_offsets.cpu(), batch.rewards)
        batch = packed
    T, n_valid = batch.T, batch.n_valid
    params = ais.default_params(vocab_chunk=w.vocab_chunk)
    if args.w_dv:
        batch.W = batch.W.t().contiguous()                             # the same head stored [d, V]
    step = ais.AisStep(T, w.d, w.V, w.P, w.G, w.block, device=dev, params=params, workspace_bytes_cap=args.workspace_gb << 30,
                       group=(dist.group.WORLD if world > 1 else None), P_total=w.P * world,
                       w_layout=ais.W_DV if args.w_dv else ais.W_VD)
    offs = batch.seq_offsets.to(dev)
    rew = batch.rewards.to(dev)
    stream = torch.cuda.current_stream(dev)

    # variant (not the headline step): also produce the LM-head weight gradient, one more T x d x V pass
    dW_buf = torch.empty((w.d, w.V) if args.w_dv else (w.V, w.d), dtype=torch.float32, device=dev) if args.with_dw else None

    def one_step(ev=None):
        marks = []

        def mark():
            if ev is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record(stream)
                marks.append(e)
        mark()
        ais.quantize_fp8(batch.H, w.block, step.qH, step.sH)
        mark()
        step.quantize_weights(batch.W)
        mark()
        ais.logprob_fwd(step.shape, step.params, batch.H, batch.W, None, None, None, None, batch.tokens, batch.mask,
                        step.lp_train, step.lse_train, None, None, step.status, step.workspace)
        mark()
        ais.logprob_fwd(step.shape, step.params, None, None, step.qH, step.sH, step.qW, step.sW, batch.tokens, batch.mask,
                        None, None, step.lp_roll, step.lse_roll, step.status, step.workspace)
        mark()
        step.diagnose(batch.mask, offs, rew)
        mark()
        step.backward(batch.H, batch.W, batch.tokens, batch.mask, offs, dW=dW_buf)
        mark()
        if ev is not None:
            ev.append(marks)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # the HBM-bound kernels timed alone, before the long power-capped loop (burst conditions, like the copy that
    # measured the bandwidth they are compared with); inside the step they are bound by launch latency
    streaming = None
    if rank == 0 and world == 1 and w.block > 0 and not args.prompts and not args.no_streaming and not args.w_dv:
        streaming = streaming_scale(dev, batch.W, w.block, args.streaming_rows, H=batch.H)
    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    events = []
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for _ in range(args.steps):
        one_step(events)
    t_end.record(stream)
    barrier()
    total_ms = t_start.elapsed_time(t_end)
    clocks = sampler.stop() if sampler else None
    status = int(step.status.item())
    if status != 0:
        raise RuntimeError(f"device status word {status}")
    diag = step.read_diag()

    names = ["quantize_H", "quantize_W", "fwd_train_bf16", "fwd_roll_fp8", "diagnostics", "loss_bwd"]
    seg = {n: 0.0 for n in names}
    for marks in events:
        for i, n in enumerate(names):
            seg[n] += marks[i].elapsed_time(marks[i + 1])
    seg = {n: v / args.steps for n, v in seg.items()}

    # ---- end to end through host buffers
    pin = dict(H=batch.H.cpu().pin_memory(), tokens=batch.tokens.cpu().pin_memory(), mask=batch.mask.cpu().pin_memory(),
               offs=batch.seq_offsets.pin_memory(), rew=batch.rewards.pin_memory())
    dH_host = torch.empty(step.dH.shape, dtype=step.dH.dtype).pin_memory()
    small_host = torch.empty(step.diag.numel() + 1, dtype=torch.float64).pin_memory()
    H2 = torch.empty_like(batch.H)
    tok2, msk2 = torch.empty_like(batch.tokens), torch.empty_like(batch.mask)
    offs2, rew2 = torch.empty_like(offs), torch.empty_like(rew)
    h2d = sum(t.numel() * t.element_size() for t in pin.values())
    d2h = dH_host.numel() * dH_host.element_size() + small_host.numel() * 8

    # Every step copies its inputs in from pinned host memory and its results (dH, diagnostics, loss) out.  The copies
    # run on two side streams so that a step's input copy and the previous step's result copy overlap the tensor-core
    # passes: two device buffers for H alternate, and the backward waits until the previous dH has left the device.
    in_s, out_s = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    Hbuf = [H2, torch.empty_like(batch.H)]
    ev_in = [torch.cuda.Event(), torch.cuda.Event()]
    ev_used = [torch.cuda.Event(), torch.cuda.Event()]      # the step that read Hbuf[i] has finished
    ev_bwd, ev_out = torch.cuda.Event(), torch.cuda.Event()

    def e2e_prefetch(i):
        with torch.cuda.stream(in_s):
            in_s.wait_event(ev_used[i % 2])
            Hbuf[i % 2].copy_(pin["H"], non_blocking=True)
            ev_in[i % 2].record(in_s)

    def e2e_step(i, last):
        stream.wait_event(ev_in[i % 2])
        if not last:
            e2e_prefetch(i + 1)
        tok2.copy_(pin["tokens"], non_blocking=True)
        msk2.copy_(pin["mask"], non_blocking=True)
        offs2.copy_(pin["offs"], non_blocking=True)
        rew2.copy_(pin["rew"], non_blocking=True)
        Hi = Hbuf[i % 2]
        step.forward(Hi, batch.W, tok2, msk2)
        step.diagnose(msk2, offs2, rew2)
        stream.wait_event(ev_out)                           # dH and the diagnostics of the previous step are on the host
        step.backward(Hi, batch.W, tok2, msk2, offs2)
        ev_bwd.record(stream)
        ev_used[i % 2].record(stream)
        with torch.cuda.stream(out_s):
            out_s.wait_event(ev_bwd)
            dH_host.copy_(step.dH, non_blocking=True)
            small_host[:-1].copy_(step.diag, non_blocking=True)
            small_host[-1:].copy_(step.loss.double(), non_blocking=True)
            ev_out.record(out_s)

    e2e_steps = max(1, min(args.steps, 5))
    ev_used[0].record(stream)
    ev_used[1].record(stream)
    ev_out.record(stream)
    e2e_prefetch(0)
    e2e_step(0, True)                                       # warm-up
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    e2e_prefetch(0)
    for i in range(e2e_steps):
        e2e_step(i, i == e2e_steps - 1)
    stream.wait_event(ev_out)                               # the last results have reached the host
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps

    # rows the backward passes really work on: a 128-row tile is skipped when every gradient factor in it is zero
    # (masked rows; rows of a prompt whose responses all got the same reward), the dH pass works on pairs of tiles
    adv_tok = np.repeat(step.adv.cpu().numpy(), np.diff(batch.seq_offsets.numpy()))
    live = (batch.mask.cpu().numpy() != 0) & (adv_tok != 0)
    pad = (-T) % 256
    live_tiles = np.concatenate([live, np.zeros(pad, bool)]).reshape(-1, 128).any(axis=1)
    rows_in_tile = np.minimum(128, T - 128 * np.arange(len(live_tiles))).clip(min=0)
    rows_recompute = int(rows_in_tile[live_tiles].sum())
    live_pairs = np.repeat(live_tiles.reshape(-1, 2).any(axis=1), 2)
    rows_dh = int(rows_in_tile[live_pairs].sum())

    fixed = ais.workspace_min_bytes(step.shape, step.params) - 128 * _ld_u(w.V) * 2
    blk_rows = (step.workspace.numel() - fixed) // (_ld_u(w.V) * 2) // 128 * 128
    blk_rows = max(128, min(blk_rows, (T + 127) // 128 * 128))
    chunks = -(-T // blk_rows)
    launches = (6 if w.block == 0 else 4 if w.block < 0 else 2) + 3 + 3 + (4 if world == 1 else 5) + 4 + (3 if args.with_dw else 2) * chunks
    return dict(ms_per_step=total_ms / args.steps, e2e_ms=e2e_ms, n_valid=n_valid, T=T, seg=seg, clocks=clocks, diag=diag,
                h2d=h2d, d2h=d2h, streaming=streaming, zero_rows=int(T - live.sum() - (batch.mask.cpu().numpy() == 0).sum()),
                rows_recompute=rows_recompute, rows_dh=rows_dh, bwd_row_chunks=chunks, launches_per_step=launches,
                workload=w)


# ------------------------------------------------------------------------------------------ the JSON line
def assemble_line(args, world: int, local: dict, glob: dict) -> dict:
    """Rank 0's JSON line from its own measurement and the whole-job figures."""
    peaks = _peaks()
    w = local["workload"]
    T, seg = local["T"], local["seg"]
    clocks = local["clocks"] or {}
    mhz = clocks.get("sm_mhz")
    flops_pass = 2.0 * T * w.d * w.V                      # algorithmic FLOPs of one T x d x V contraction over all rows
    sus, burst = peaks["bf16_tflops_sustained"], peaks["bf16_tflops"]
    roll_ratio = 4 if w.block == -4 else 2
    roll_nominal = NOMINAL["fp4_tflops"] if w.block == -4 else NOMINAL["fp8_tflops"]
    traffic = (TRAFFIC.get(args.workload, {}) if not args.prompts and world == 1 else {})

    def pass_entry(ms, flops, ratio, nominal, name, extra=None):
        tf = flops / (ms * 1e-3) / 1e12
        e = {"ms": ms, "tflops": tf, "peak": ratio * sus, "frac": tf / (ratio * sus), "frac_of_burst": tf / (ratio * burst),
             "frac_nominal": tf / nominal, "gcycles": (ms * 1e-3 * mhz * 1e-3 if mhz else None),
             "traffic": traffic.get(name) if w.block > 0 or name != "fwd_roll_fp8" else None}
        if extra:
            e.update(extra)
        return e

    passes = {
        "fwd_train_bf16": pass_entry(seg["fwd_train_bf16"], flops_pass, 1, NOMINAL["bf16_tflops"], "fwd_train_bf16"),
        "fwd_roll_fp8": pass_entry(seg["fwd_roll_fp8"], flops_pass, roll_ratio, roll_nominal, "fwd_roll_fp8"),
    }
    if w.block > 0:
        # fp32 scales per block of both operands send every block's partial sums out of tensor memory and through the CUDA
        # cores.  Tensor memory holds two 128 x 256 partial tiles; with promotion warps that neither load nor compute the
        # round trip MMA -> commit -> hand-over -> next MMA still takes 805 clocks per block against 542 tensor-pipe clocks
        # (timing-only measurement), so the formulation cannot exceed 542 / 805 of the FP8 tensor rate on this kernel structure
        passes["fwd_roll_fp8"]["ceiling"] = {"frac_of_fp8_tensor_rate": 542.0 / 805.0,
                                             "why": "fp32 block scales: one tensor-memory round trip per K block, two partial tiles in flight"}
    n_bwd = 3 if args.with_dw else 2
    flops_bwd = 2.0 * w.d * w.V * (local["rows_recompute"] + local["rows_dh"] + (T if args.with_dw else 0))
    passes["bwd"] = pass_entry(seg["loss_bwd"], flops_bwd, 1, NOMINAL["bf16_tflops"], "bwd", {
        "kernels": n_bwd, "rows_recompute": local["rows_recompute"], "rows_dH": local["rows_dh"],
        "note": "recompute + dH%s; FLOPs of the rows in 128-row tiles that hold a non-zero gradient factor "
                "(the other tiles are skipped)" % (" + dW over all rows" if args.with_dw else "")})
    # the kernel with the largest share of this run's step: the two forward kernels as timed, the backward kernels as
    # the average of their segment (they are enqueued by one call)
    per_kernel = {"fwd_train_bf16": seg["fwd_train_bf16"], "fwd_roll_fp8": seg["fwd_roll_fp8"], "bwd": seg["loss_bwd"] / n_bwd}
    top = max(per_kernel, key=per_kernel.get)
    kernel_names = {
        "fwd_train_bf16": "lmhead_kernel<bf16 forward> (trainer log-probs)",
        "fwd_roll_fp8": {0: "lmhead_kernel<per-tensor FP8 forward>", -32: "lmhead_kernel<microscaling FP8 forward>",
                         -4: "lmhead_kernel<microscaling FP4 forward>"}.get(
            w.block, "lmhead_fp8_block_kernel (rollout log-probs, E4M3 with fp32 scales per %d elements)" % w.block),
        "bwd": "lmhead_kernel<recompute> and lmhead_kernel<dH> (average of the two launches)",
    }
    tp = passes[top]
    roofline = {"bound": "tensor", "kernel": kernel_names[top], "achieved": tp["tflops"], "peak": tp["peak"], "unit": "TFLOP/s",
                "frac": tp["frac"], "frac_of_burst": tp["frac_of_burst"], "frac_nominal": tp["frac_nominal"], "traffic": tp["traffic"],
                "peak_source": peaks["source"] + " bf16 sustained (kernel timed inside a long step)" +
                               (" x %d (nominal FP8 : bf16 ratio)" % roll_ratio if top == "fwd_roll_fp8" else ""),
                "chosen_by": "largest per-kernel time of this run: " + ", ".join("%s %.1f ms" % kv for kv in per_kernel.items()),
                "passes": passes}
    if "ceiling" in tp:
        roofline["ceiling"] = tp["ceiling"]
    bytes_per_elem = 3.0 + 4.0 / w.block if w.block > 0 else 2.53 if w.block == -4 else 3.03 if w.block < 0 else 5.0
    qh = T * w.d * bytes_per_elem / (seg["quantize_H"] * 1e-3) / 1e9
    qw = w.V * w.d * bytes_per_elem / (seg["quantize_W"] * 1e-3) / 1e9
    roofline["quantize_in_step"] = {"H_gbs": qh, "W_gbs": qw, "H_frac": qh / peaks["hbm_gbs"], "W_frac": qw / peaks["hbm_gbs"],
                                    "H_frac_nominal": qh / NOMINAL["hbm_gbs"], "W_frac_nominal": qw / NOMINAL["hbm_gbs"],
                                    "note": "inside the power-capped step; timed alone under `streaming`"}
    out = {
        "metric": METRIC, "value": glob["tokens_all"] / (glob["ms_per_step"] * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": glob["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16+fp8_e4m3", "data": "synthetic",
        "config": {"workload": _workload_text(w), "rows": T, "valid_tokens_per_gpu": local["n_valid"],
                   "l2": "inputs larger than L2 (H %.2f GB, W %.2f GB)" % (T * w.d * 2 / 1e9, w.V * w.d * 2 / 1e9),
                   "zero_gradient_rows": local["zero_rows"],
                   "parallelism": f"dp{world} (whole prompts per GPU, LM head replicated, one all-reduce of 12 moments for alpha)",
                   "bwd_row_chunks": local["bwd_row_chunks"], "alpha": local["diag"]["alpha"], "d_bar": local["diag"]["d_bar"]},
        "segments_ms": seg,
        "roofline": roofline,
        "e2e": {"value": glob["tokens_all"] / (glob["e2e_ms"] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": local["h2d"],
                "d2h_bytes_per_step": local["d2h"],
                "note": "per step: H, tokens, mask, offsets and rewards in from pinned host memory, dH, diagnostics and loss out; "
                        "W (%.2f GB) stays resident on the device and is re-quantised every step; copies on side streams overlap "
                        "the passes, so this is pipelined throughput" % (w.V * w.d * 2 / 1e9)},
        "gpu_launches": local["launches_per_step"] * args.steps,
        "clocks": local["clocks"],
    }
    st = local.get("streaming")
    if st is not None:
        keys = ("moments_gbs", "rectify_gbs", "quantize_W_gbs", "quantize_H_gbs")
        st.update({"peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                   "frac": {k[:-4]: st[k] / peaks["hbm_gbs"] for k in keys if k in st},
                   "frac_nominal": {k[:-4]: st[k] / NOMINAL["hbm_gbs"] for k in keys if k in st}})
        out["streaming"] = st
    return out


def resolve(spec: str):
    mod, _, fn = spec.partition(":")
    return getattr(importlib.import_module(mod), fn)


def run_ours(args) -> None:
    import torch.distributed as dist
    rank, world, local = rank_env()
    cpu_ranks = args.dist_backend == "gloo"
    dev = torch.device("cpu") if cpu_ranks else torch.device("cuda", local)
    if world > 1:
        if cpu_ranks:
            dist.init_process_group("gloo")
        else:
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=dev)
    measure = resolve(args.measure) if args.measure else measure_rank
    res = measure(args, rank, world, local)
    glob = reduce_over_ranks(res, world, dev)
    if rank == 0:
        out = assemble_line(args, world, res, glob)
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline_object(res["workload"])
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------ streaming kernels at scale
def streaming_scale(dev, W: torch.Tensor, block: int, rows: int = 1 << 26, H: torch.Tensor | None = None):
    """HBM-bound kernels timed alone (CUDA events, 10 launches after 3 warm-ups, operands larger than L2): the batch
    reductions on a synthetic batch of `rows` rows (at the workloads' own sizes they move about 1 MB and are bound by
    launch latency), and the quantiser on the workload's W and H.  Bytes are the algorithmic ones: ais_diag_moments reads
    lp_train, lp_roll (4 B each) and the mask (1 B) per row; ais_diag_finalize reads the same 9 B and writes rho and
    w_tilde (8 B); the quantiser moves 2 + 1 + 4/block B per element."""
    import paper_2605_13907_b200 as ais
    G, L = 8, 1024
    S = rows // L
    g = torch.Generator(device=dev).manual_seed(7)
    lp_t = -5.0 * torch.rand(rows, generator=g, device=dev)
    lp_r = lp_t + 0.05 * torch.randn(rows, generator=g, device=dev)
    mask = (torch.rand(rows, generator=g, device=dev) < 0.9).to(torch.uint8)
    offs = torch.arange(0, rows + 1, L, dtype=torch.int32, device=dev)
    rew = (torch.rand(S, generator=g, device=dev) < 0.3).float()
    shape = ais.make_shape(rows, 128, 1024, S // G, G, 128)
    params = ais.default_params(vocab_chunk=1024)
    ws = torch.empty(ais.workspace_min_bytes(shape, params), dtype=torch.uint8, device=dev)
    adv = torch.empty(S, device=dev)
    nseq = torch.empty(S, dtype=torch.int32, device=dev)
    moments = torch.empty(16, dtype=torch.float64, device=dev)
    rho, wt = torch.empty(rows, device=dev), torch.empty(rows, device=dev)
    diag = torch.empty(32, dtype=torch.float64, device=dev)          # an ais_diag struct (19 doubles + flags)

    def timed(fn, n=10, warm=3):
        for _ in range(warm):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / n * 1e-3

    t_mom = timed(lambda: ais.diag_moments(shape, params, lp_t, lp_r, mask, offs, rew, adv, nseq, moments, ws))
    t_fin = timed(lambda: ais.diag_finalize(shape, params, moments, lp_t, lp_r, mask, rho, wt, diag))
    qW, sW = ais.quantize_fp8(W, block)
    t_q = timed(lambda: ais.quantize_fp8(W, block, qW, sW))
    out = {"rows": rows, "moments_gbs": rows * 9 / t_mom / 1e9, "rectify_gbs": rows * 17 / t_fin / 1e9,
           "quantize_W_gbs": W.numel() * (3.0 + 4.0 / block) / t_q / 1e9}
    if H is not None and H.numel() > 0:
        qH, sH = ais.quantize_fp8(H, block)
        t_h = timed(lambda: ais.quantize_fp8(H, block, qH, sH))
        out["quantize_H_gbs"] = H.numel() * (3.0 + 4.0 / block) / t_h / 1e9
    return out


# ------------------------------------------------------------------------------------------ reference arm (CPU oracle)
def run_reference(args) -> None:
    rank, world, _ = rank_env()
    if rank != 0:
        return
    w = workloads.WORKLOADS[args.workload]
    steps, warm = max(1, min(args.steps, 3)), min(args.warmup, 1)
    for _ in range(warm):
        oracle_sample(w, tokens_n=64, vocab_n=2048)
    runs = [oracle_sample(w) for _ in range(steps)]
    value = len(runs) / sum(1.0 / r["rate"] for r in runs)
    stages = {k: sum(r["stages_s"][k] for r in runs) / len(runs) for k in runs[0]["stages_s"]}
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warm,
           "ms_per_step": 1e3 * sum(r["seconds"] for r in runs) / len(runs), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": _workload_text(w)},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": runs[0]["sample"],
                            "stages_s": stages},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


def build_parser() -> argparse.ArgumentParser:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="qwen3_8b", choices=sorted(workloads.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workspace-gb", type=int, default=48)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-streaming", action="store_true", help="skip the HBM-bound kernels timed alone at 2^26 rows")
    ap.add_argument("--streaming-only", action="store_true",
                    help="only time the HBM-bound kernels alone (batch reductions at --streaming-rows rows, quantiser on W)")
    ap.add_argument("--streaming-rows", type=int, default=1 << 26)
    ap.add_argument("--prompts", type=int, default=0, help="override the number of prompts (small profiling case)")
    ap.add_argument("--compact", action="store_true",
                    help="pack the valid rows first (for workloads with scattered masks, e.g. llada_8b)")
    ap.add_argument("--with-dw", action="store_true", help="variant: ais_loss_bwd also writes dW (a fifth tensor-core pass)")
    ap.add_argument("--fp4-mx", action="store_true",
                    help="variant (not the headline workload): microscaling FP4 rollout pass (E2M1, scale per 32 elements)")
    ap.add_argument("--fp8-mx", action="store_true",
                    help="variant (not the headline workload): microscaling FP8, power-of-two scale per 32 elements")
    ap.add_argument("--fp8-per-tensor", action="store_true",
                    help="variant (not the headline workload): per-tensor dynamic FP8 scaling instead of per-block scales")
    ap.add_argument("--w-dv", action="store_true",
                    help="variant (not the headline layout): the LM head stored [d, V] instead of [V, d]")
    ap.add_argument("--dist-backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend of the ranks; gloo only together with --measure (tests of the rank logic on CPU)")
    ap.add_argument("--measure", default="",
                    help="module:function replacing the per-rank GPU measurement (tests of the launcher, the reduction over "
                         "ranks and the JSON line without a GPU); the default measures on the rank's GPU")
    return ap


def main(argv=None) -> int:
    argv = list(sys.argv[1:] if argv is None else argv)
    args = build_parser().parse_args(argv)
    if args.dist_backend == "gloo" and not args.measure:
        raise SystemExit("--dist-backend gloo has no measurement of its own: the path runs on GPUs only")
    if args.impl == "reference":
        run_reference(args)
    elif args.streaming_only:
        w = workloads.WORKLOADS[args.workload]
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        W = (torch.randn(w.V, w.d, device=dev) * w.w_std).to(torch.bfloat16)
        out = streaming_scale(dev, W, w.block if w.block > 0 else 128, args.streaming_rows)
        out["peak_gbs"] = _peaks()["hbm_gbs"]
        print(json.dumps({"streaming": out}), flush=True)
    elif needs_launch(args):
        return launch_ranks(args, argv)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)
    return 0


if __name__ == "__main__":
    sys.exit(main())
