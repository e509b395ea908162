"""The N > 1 path of the benchmark on CPU: two gloo ranks stand in for two GPUs.

The BitLinear path does not shard ("replicas only"): every rank runs the whole workload on its own GPU
and the only exchange is the maximum of the device-side timings, from which rank 0 reports the
whole-job throughput.  These tests run that exchange with world_size 2 over gloo.
"""
import os
import socket
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, str(ROOT))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [0.150 + 0.010 * rank, 0.140 - 0.005 * rank, 0.300 + 0.020 * rank]  # step, kernel, e2e in ms
    got = bench.max_over_ranks(dist, mine, "cpu")
    # the ranks go on with their timed rounds until ALL have measured enough: rank 1 is not done in the first poll
    polls = [bench.all_ranks_agree(dist, rank == 0, "cpu"), bench.all_ranks_agree(dist, True, "cpu")]
    dist.barrier()
    if rank == 0:
        out.put(got + polls)
    dist.destroy_process_group()


def test_timings_are_reduced_with_max_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    got = out.get()
    assert got[3:] == [False, True]
    got = got[:3]
    assert got == [0.160, 0.140, 0.320]
    sys.path.insert(0, str(ROOT))
    import bench
    # two replicas of 805,376,000 bytes in 0.160 ms: the slower rank sets the time, the bytes add up
    assert abs(bench.aggregate_throughput(805_376_000, 2, got[0]) - 2 * 805_376_000 / 0.160e-3 / 1e9) < 1e-6
    assert bench.max_over_ranks(None, [1.0, 2.0], "cpu") == [1.0, 2.0]
    assert bench.all_ranks_agree(None, True, "cpu") and not bench.all_ranks_agree(None, False, "cpu")


def test_reference_arm_prints_nothing_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
