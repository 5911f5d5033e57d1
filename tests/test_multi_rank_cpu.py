"""The N > 1 path of bench.py is N independent replicas with a barrier and a max-over-ranks reduction of
the timed region.  That host logic is exercised here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    import bench

    w, r, local = bench.dist_setup(world)          # picks gloo when no GPU is present
    assert (w, r, local) == (world, rank, rank)
    bench.barrier(w)
    mine = 10.0 + 5.0 * rank                        # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine, w, torch.device("cpu"))
    # whole-job value of N replicas: N steps per slowest-rank step time
    value = w * 1e3 / slowest
    out[rank] = (slowest, value)
    bench.barrier(w)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time():
    if torch.cuda.is_available():
        import pytest

        pytest.skip("the CPU/gloo variant of the check")
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1]
    slowest, value = out[0]
    assert slowest == 15.0
    assert abs(value - 2 * 1e3 / 15.0) < 1e-9


def test_reference_arm_is_rank0_only(tmp_path):
    """Under torchrun the reference (oracle) arm runs on rank 0 alone; other ranks leave without work."""
    import subprocess

    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
