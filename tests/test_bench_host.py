"""Host logic of the multi-rank bench path, on CPU with the gloo backend (world size 2):
every rank takes its own seeded batch of the same shape (replicas, no data-path
collective), the elapsed time reported is the slowest rank's, the value is the whole job's.
Also: the reference arm of bench.py runs the CPU oracle and prints the agreed JSON line,
and only rank 0 does so; and `bench.py --gpus N` without a launcher starts its own N ranks."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2401_06706_b200 import synth  # noqa: E402


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.shard_for_rank(synth.named_workloads()["cfg1_tiny"], rank, world)
    inp = synth.make_inputs(w, "cpu")
    elapsed = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    dist.barrier()
    worst = bench.max_over_ranks(dist, elapsed, "cpu")
    nodes = w.batch * inp.stats["n_draft"]
    rec = {"seed": w.seed, "worst": worst, "value": bench.whole_job_value(world, nodes, worst),
           "first_logit": float(inp.target.flatten()[0])}
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump(rec, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_replica_and_report_the_slowest(tmp_path):
    port = 29500 + os.getpid() % 500
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (json.load(open(tmp_path / f"rank{r}.json")) for r in (0, 1))
    assert r0["seed"] != r1["seed"] and r0["first_logit"] != r1["first_logit"]   # own batch per rank
    assert r0["worst"] == r1["worst"] == 15.0                                     # max over ranks
    assert r0["value"] == r1["value"] == pytest.approx(2 * 1 * 2 / 15e-3)         # whole job


def test_single_rank_keeps_the_workload_unchanged():
    w = synth.named_workloads()["cfg2_b8_with"]
    assert bench.shard_for_rank(w, 0, 1) is w
    assert bench.max_over_ranks(None, 3.5, "cpu") == 3.5


def _run_reference(env_extra):
    env = dict(os.environ, **env_extra)
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1_tiny",
           "--steps", "2", "--warmup", "1"]
    return subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=300)


def test_reference_arm_prints_the_contract_line_on_rank_zero_only():
    out = _run_reference({"RANK": "0", "WORLD_SIZE": "1"})
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "cfg1_tiny"
    other = _run_reference({"RANK": "1", "WORLD_SIZE": "2"})
    assert other.returncode == 0 and other.stdout.strip() == ""


def test_gpus_n_without_a_launcher_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no WORLD_SIZE around it: the script starts two ranks itself
    (shown on the reference arm, which needs no GPU); stdout is still the one JSON line of rank 0."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1_tiny",
           "--steps", "1", "--warmup", "1", "--gpus", "2"]
    out = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=600)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    cmd = bench.spawn_command(["--gpus", "2"], 2, 29999)
    assert "torch.distributed.run" in cmd and "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd


def test_sweep_resume_reads_the_points_a_cut_off_file_holds(tmp_path):
    import bench
    path = tmp_path / "sweep.jsonl"
    path.write_text('{"workload": "a", "us_median": 1.0}\n{"workload": "b"}\n{"workload": "c", "us_med')   # cut off in the third line
    assert bench.sweep_points_done(str(path)) == {"a", "b"}
