"""bench.py's multi-rank logic without a GPU: `bench.py --gpus 2` must start two ranks (one per GPU on a GPU machine),
form the process group, reduce the per-rank figures (MAX of the times, SUM of the tokens) and print ONE JSON line
with n_gpus = 2 from rank 0.  The per-rank GPU measurement is replaced by tests/bench_stub.py through --measure and
the ranks talk over gloo, so the launcher, the rank environment, the all-reduces and the line assembly are the ones
a GPU run uses."""

import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra, env_extra=None, timeout=300):
    env = dict(os.environ)
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    env["PYTHONPATH"] = os.pathsep.join([ROOT, os.path.join(ROOT, "tests"), env.get("PYTHONPATH", "")])
    env.update(env_extra or {})
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "4", "--warmup", "3", "--no-cpu-baseline",
           "--dist-backend", "gloo", "--measure", "bench_stub:measure_rank"] + extra
    return subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=timeout, cwd=ROOT)


def _json_lines(text):
    out = []
    for line in text.splitlines():
        line = line.strip()
        if line.startswith("{"):
            out.append(json.loads(line))
    return out


def test_gpus_2_starts_two_ranks_and_rank_0_prints_one_line():
    res = _run(["--gpus", "2"])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = _json_lines(res.stdout)
    assert len(lines) == 1, res.stdout
    line = lines[0]
    assert line["n_gpus"] == 2 and line["steps"] == 4 and line["scaling"] == "weak"
    # times: the slower rank (110 ms, 120 ms end to end); tokens: both ranks (993 + 1993)
    assert line["ms_per_step"] == 110.0
    assert abs(line["value"] - (993 + 1993) / 0.110) < 1e-6
    assert abs(line["e2e"]["value"] - (993 + 1993) / 0.120) < 1e-6
    assert line["config"]["parallelism"].startswith("dp2")
    assert line["metric"].startswith("AIS-corrected") and line["unit"] == "tokens/s" and line["vs_baseline"] is None
    assert "cpu_baseline" not in line                       # reported at one GPU only
    r = line["roofline"]
    assert r["bound"] == "tensor" and 0 < r["frac"] and "frac_nominal" in r and "passes" in r
    assert r["kernel"].startswith("lmhead_kernel<bf16 forward>")      # 80 ms against 70 and 120 / 2 in the stub's segments


def test_plain_start_is_one_rank_and_torchrun_environment_is_respected():
    one = _run([])
    assert one.returncode == 0, one.stderr[-2000:]
    line = _json_lines(one.stdout)[0]
    assert line["n_gpus"] == 1 and line["ms_per_step"] == 100.0 and abs(line["value"] - 993 / 0.100) < 1e-6
    # started by a launcher that already set the rank variables (the way the two-GPU bench is driven): no second launch
    env = {"RANK": "0", "WORLD_SIZE": "1", "LOCAL_RANK": "0", "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": "29571"}
    again = _run(["--gpus", "1"], env_extra=env)
    assert again.returncode == 0 and _json_lines(again.stdout)[0]["n_gpus"] == 1


def test_backward_fraction_counts_only_rows_in_live_tiles():
    """assemble_line charges the backward passes with the rows they process, never with skipped tiles."""
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import bench
    import bench_stub
    args = bench.build_parser().parse_args(["--no-cpu-baseline"])
    local = bench_stub.measure_rank(args, 0, 1, 0)
    local["rows_recompute"], local["rows_dh"] = 600, 512
    glob = bench.reduce_over_ranks(local, 1, None)
    line = bench.assemble_line(args, 1, local, glob)
    w = local["workload"]
    want = 2.0 * w.d * w.V * (600 + 512) / 0.120 / 1e12
    assert abs(line["roofline"]["passes"]["bwd"]["tflops"] - want) < 1e-9 * want
    assert 0.5 < line["roofline"]["passes"]["fwd_roll_fp8"]["ceiling"]["frac_of_fp8_tensor_rate"] < 0.7
