"""World-size-2 check (gloo, CPU) of the host logic that bench.py uses when it runs N replicas:
every rank times its own replica, the slowest rank decides, and the reported value is N times the
per-replica work divided by that time.  The two functions of bench.py that do this (reduce_max_ms,
aggregate_value) are called here as they stand.  No data-path collective exists, so this is all there
is to cover."""

import os
import socket
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if root not in sys.path:
        sys.path.insert(0, root)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank "measures" a different time for the same per-replica work
    dist.barrier()
    elapsed_ms = bench.reduce_max_ms(10.0 + 5.0 * rank, world, dist, torch, torch.device("cpu"))
    value = bench.aggregate_value(6_000_000_000, world, elapsed_ms)
    if rank == 0:
        out.put((elapsed_ms, value))
    dist.destroy_process_group()


PORT = _free_port()


def test_replica_timing_takes_the_slowest_rank():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, PORT, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    elapsed, value = out.get(timeout=10)
    assert elapsed == 15.0
    assert value == pytest.approx(2 * 6.0 / 0.015)


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    """bench.py --impl reference under a 2-rank launch: rank 1 exits without printing."""
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
