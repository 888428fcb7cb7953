"""bench.py's multi-rank bookkeeping ("replicas only"): max over ranks of the step time and the
whole-job throughput, exercised with two gloo ranks on CPU."""
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
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 1 is slower on the first, faster on the second
    red = bench.max_over_ranks(local)
    dist.barrier()
    if rank == 0:
        value = bench.whole_job_throughput(1000.0, world, red[0])
        torch.save({"red": red, "value": value}, out)
    dist.destroy_process_group()


def test_two_rank_max_and_throughput(tmp_path):
    out = str(tmp_path / "r.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["red"] == [15.0, 3.0]
    assert abs(r["value"] - 2 * 1000.0 / 15e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_throughput(10.0, 1, 2.0) == 5000.0
