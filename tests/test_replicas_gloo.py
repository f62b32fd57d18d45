"""The N > 1 path on CPU: replicas only (no data-path collective), so what is distributed is the measurement.
Two gloo ranks check the aggregation bench.py uses, and the launch contract of the reference arm under torchrun
(rank 0 alone runs and prints, the other ranks exit 0 without work)."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2601_20357_b200.replicas import whole_job
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms, units, value = whole_job(10.0 * (rank + 1), 5 + rank, dist, torch.device("cpu"))
        out.put((rank, ms, units, value))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_whole_job_is_slowest_rank_time_and_summed_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for rank, ms, units, value in got:
        assert ms == 20.0 and units == 11 and value == pytest.approx(11 / 0.020)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2601_20357_b200.replicas import whole_job
    assert whole_job(4.0, 2) == (4.0, 2, 500.0)
    with pytest.raises(ValueError):
        whole_job(0.0, 2)


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "1", "--config", "tiny"]
    r = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
