"""The multi-GPU path of bench.py is "replicas only": every rank runs the same workload on its own GPU, the
timed region is the maximum over ranks, and the reported value is world x one rank's units over that time.
This runs the rank-combining code on two CPU processes with the gloo backend (no GPU), and checks that the
reference arm prints on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 0 is the faster replica on the first number and the slower one on the second
    mine = [10.0 + rank, 7.0 - rank, 3.0]
    combined = bench.max_over_ranks(mine, world)
    spec = bench.WORKLOADS["decode7b"]
    value = bench.whole_job_value(spec, world, step_bytes=4_000_000_000, step_flops=0, steps=5, slowest_ms=combined[0])
    dist.barrier()
    if rank == 0:
        out.put((combined, value))
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_sum_the_units():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    combined, value = out.get()
    assert combined == [11.0, 7.0, 3.0]
    # 2 replicas x 5 steps x 4 GB in 11 ms
    assert value == pytest.approx(2 * 5 * 4.0 / 11e-3)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    spec = bench.WORKLOADS["prefill7b"]
    assert bench.whole_job_value(spec, 1, 0, 2e12, 10, 20.0) == pytest.approx(10 * 2e12 / 20e-3 / 1e12)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "2", "--warmup", "0", "--ref-budget", "2"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
