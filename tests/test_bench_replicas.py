"""The multi-GPU rule of bench.py on CPU: replicas only, no data-path collective.  Two gloo ranks
report different times and unit counts; the job's rate must be the sum of the units over the ranks
divided by the slowest rank's time (the only communication is that reduction)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    units = [1000.0, 3000.0][rank]
    ms = [2.0, 5.0][rank]
    rate, slowest = bench.job_throughput(units, ms, dist, torch.device("cpu"))
    dist.barrier()
    if rank == 0:
        torch.save({"rate": rate, "slowest": slowest}, out)
    dist.destroy_process_group()


def test_two_replicas_sum_units_over_slowest_time(tmp_path):
    out = str(tmp_path / "r.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["slowest"] == pytest.approx(5.0)
    assert r["rate"] == pytest.approx(4000.0 / 5e-3)


def test_single_process_needs_no_process_group():
    import bench
    rate, ms = bench.job_throughput(10.0, 4.0)
    assert ms == 4.0 and rate == pytest.approx(2500.0)
