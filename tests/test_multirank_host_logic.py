"""The N > 1 path of bench.py on CPU: two gloo ranks, replicas only (the hot path has no exchange step), so
the only cross-rank logic is the barrier, the max-over-ranks time and the whole-job throughput."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank "measured" a different time for the same per-rank work
    ms = 2.0 + rank
    worst = bench.max_over_ranks(ms, dist, device="cpu")
    value = bench.whole_job_throughput(world, bytes_per_rank=10 ** 9, ms=worst)
    dist.barrier()
    if rank == 0:
        torch.save({"worst": worst, "value": value}, out)
    dist.destroy_process_group()


def test_two_rank_aggregation(tmp_path):
    world, port = 2, _free_port()
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    got = torch.load(out)
    assert got["worst"] == 3.0                       # the slowest rank sets the time
    assert abs(got["value"] - 2 * 1e9 / 3e-3 / 1e9) < 1e-6   # both ranks' bytes over that time, in GB/s
