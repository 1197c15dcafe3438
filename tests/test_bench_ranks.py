"""The benchmark's multi-rank bookkeeping (replicas: one context per rank, no data-path collective) on
two gloo ranks on the CPU: barrier, max-over-ranks time, whole-job throughput."""
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
    p = s.getsockname()[1]
    s.close()
    return p


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"), world)      # rank 1 is slower
    value = bench.job_throughput(world, k=3, steps=9, ms=ms)
    prefix = bench.si.make_prefix("zipf", 15, 32000, 1.1, seed=2, tensor_id=rank)
    gathered = [None] * world
    dist.all_gather_object(gathered, prefix)
    if rank == 0:
        torch.save({"ms": ms, "value": value, "prefixes": gathered}, out)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_rank, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["ms"] == 15.0                                     # the slowest rank sets the time
    assert abs(r["value"] - 2 * 3 * 9 / 15e-3) < 1e-6          # all ranks' drafts over that time
    assert r["prefixes"][0] != r["prefixes"][1]                # each replica serves its own request


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, torch.device("cpu"), 1) == 7.5
    assert abs(bench.job_throughput(1, 3, 9, 9.0) - 3000.0) < 1e-6
