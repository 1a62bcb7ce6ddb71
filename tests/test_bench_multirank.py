"""bench.py's replica aggregation with two gloo ranks on CPU (no GPU): slowest rank decides the time."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 * (rank + 1), dist, torch.device("cpu"))
    out.put((rank, ms, bench.whole_job_rate(20, world, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_work():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, rate in got:
        assert ms == 20.0                       # max over ranks of 10, 20
        assert rate == pytest.approx(2 * 20 / 0.020)


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.whole_job_rate(20, 1, 100.0) == pytest.approx(200.0)


def test_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher around it: bench.py starts two ranks under torch.distributed.run
    and rank 0 prints one line for the whole job.  Rehearsed on CPU (gloo) with pretended times of 10 and 20 ms."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--steps", "4",
                          "--n-cg", "10"], capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["value"] is None
    assert line["dry_run"]["ms"] == 20.0                     # the slower rank
    assert line["dry_run"]["rate_from_pretended_times"] == pytest.approx(2 * 10 * 4 * 2 / 0.020)


def test_reference_arm_prints_the_contract_line():
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "mid",
                          "--steps", "1", "--warmup", "0", "--ref-rows", "64"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    # the same config keys as the GPU arm prints, and a step time that is the time this run spent per step
    assert set(line["config"]) == {"workload", "widths", "l", "S", "C", "n_cg", "step", "l2", "parallelism"}
    assert line["ms_per_step"] * line["steps"] <= 1e3 * 300
    assert line["full_step_ms_extrapolated"] >= line["ms_per_step"] * 0.5
    assert line["cpu_baseline"]["one_core"]["cores"] == 1
