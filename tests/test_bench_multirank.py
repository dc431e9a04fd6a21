"""The N > 1 logic of bench.py on CPU: two gloo ranks.

The path shards by sequence with no exchange, so N GPUs run N independent replicas; what the ranks share is the
barrier and the max-over-ranks reduction of the timings, and rank 0 alone prints.  These tests run that logic with
world size 2 over gloo, and launch the reference arm under torch.distributed.run the way the benchmark is launched.
"""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    # rank r measured (10 + r) ms for the steps, (3 - r) ms for attention alone
    got = bench.max_over_ranks([10.0 + rank, 3.0 - rank, 0.5], dist, torch.device("cpu"))
    dist.barrier()
    out.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_gloo_world2():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # every rank sees the slowest rank's time for each entry
    assert res[0] == res[1] == [11.0, 3.0, 0.5]


def test_whole_job_rate_is_aggregate():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_rate(16, 8, 1, 0.032)
    assert one == pytest.approx(16 * 8 / 0.032)
    # weak scaling: N replicas in the same time decode N times the tokens
    assert bench.whole_job_rate(16, 8, 4, 0.032) == pytest.approx(4 * one)


def test_reference_arm_two_ranks_prints_once():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl",
           "reference", "--config", "cfg1_tiny", "--steps", "1", "--warmup", "0", "--ref-budget", "0.2"]
    r = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                      # rank 0 alone prints
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
    assert rec["value"] > 0
