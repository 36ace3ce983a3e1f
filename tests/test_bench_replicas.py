"""The multi-GPU path of bench.py is "replicas only": ranks share nothing but the barrier and the
max-over-ranks time.  That host logic is covered here with two gloo ranks on CPU."""
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    job_ms = bench.reduce_max_ms(local_ms, world, torch.device("cpu"))
    dist.barrier()
    out[rank] = (job_ms, bench.job_value(world, 1_000_000_000, 4, job_ms))
    dist.destroy_process_group()


def test_job_time_is_max_over_ranks_and_value_is_aggregate():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0            # every rank sees the slowest rank's time
    # 2 ranks x 1 GB x 4 steps in 15 ms
    assert res[0][1] == pytest.approx(2 * 4 * 1e9 / 15e-3 / 1e9)
    import bench
    assert bench.reduce_max_ms(7.5, 1, torch.device("cpu")) == 7.5
    assert bench.job_value(1, 2 << 30, 10, 20.0) == pytest.approx((2 << 30) * 10 / 0.02 / 1e9)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_in_flight_slowdown_factor():
    """The overlap arithmetic of the interference study: a loop that outlasts the transfer does transfer_ms / f of
    its work while the transfer runs and the rest at full speed."""
    import bench
    # 20 ms of work, transfer 10 ms, everything 2x slower while it runs: 5 ms of work done in 10 ms, 15 ms left
    assert bench.in_flight_factor(20.0, 25.0, 10.0) == pytest.approx(2.0)
    # no disturbance at all
    assert bench.in_flight_factor(20.0, 20.0, 10.0) == pytest.approx(1.0)
    # the loop ends before the transfer does: plain ratio
    assert bench.in_flight_factor(5.0, 12.0, 16.0) == pytest.approx(2.4)
    # nothing got done while the transfer ran
    assert bench.in_flight_factor(20.0, 30.0, 10.0) == float("inf")
