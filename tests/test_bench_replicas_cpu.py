"""The multi-GPU mode of bench.py runs independent replicas (sequences are independent units; the path has no
collective).  Its only cross-rank step is the aggregation of the per-rank step times: the job is as slow as its
slowest rank and processes every rank's tokens.  Checked here with two gloo ranks on the CPU."""
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


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 100.0 if rank == 0 else 250.0            # rank 1 is the slow one
    value, ms = bench.replicas_throughput(local_ms, 256, world, torch.device("cpu"))
    out[rank] = (value, ms)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_all_tokens_over_the_slowest_rank():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        results = dict(out)
    for rank in range(world):
        value, ms = results[rank]
        assert ms == 250.0
        assert abs(value - 2 * 256 / 0.250) < 1e-9


def test_single_replica_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.replicas_throughput(125.0, 256, 1)
    assert ms == 125.0 and abs(value - 2048.0) < 1e-9
