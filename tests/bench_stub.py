"""Stand-in for bench.measure_rank in the CPU test of the benchmark's rank logic: no GPU work, fixed numbers that
depend on the rank, so that the reduction over ranks (MAX of the times, SUM of the tokens) shows in rank 0's line."""

import bench


def measure_rank(args, rank: int, world: int, local: int) -> dict:
    import torch
    import torch.distributed as dist
    w = bench.rank_workload(args, rank)
    # the one exchange of a step, on CPU tensors: every rank contributes its own 12 sums
    from paper_2605_13907_b200 import dist as ais_dist
    moments = torch.full((12,), float(rank + 1), dtype=torch.float64)
    ais_dist.allreduce_moments(moments, dist.group.WORLD if world > 1 else None)
    assert float(moments[0]) == world * (world + 1) / 2
    T = 1000 * (rank + 1)
    seg = {"quantize_H": 0.1, "quantize_W": 0.9, "fwd_train_bf16": 80.0, "fwd_roll_fp8": 70.0 + rank, "diagnostics": 0.03,
           "loss_bwd": 120.0}
    return dict(ms_per_step=100.0 + 10.0 * rank, e2e_ms=110.0 + 10.0 * rank, n_valid=T - 7, T=T, seg=seg,
                clocks={"sm_mhz": 1300.0, "sm_max_mhz": 1965.0, "reasons": []}, diag={"alpha": 0.5, "d_bar": 0.03},
                h2d=10, d2h=20, streaming=None, zero_rows=0, rows_recompute=T, rows_dh=T, bwd_row_chunks=1,
                launches_per_step=18, workload=w, seed=w.seed)
