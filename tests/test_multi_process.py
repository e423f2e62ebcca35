"""Replica aggregation of the benchmark over two processes (gloo, CPU): tokens add up, the time is the
slowest rank's.  The verification path itself shards by request with no collective."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    args = bench.parse_args(["--batch", "8", "--shape", "llama8b"])
    shape, ks, ctx, seed = bench.workload(args, rank)
    tok, ms = bench.aggregate(100.0 * (rank + 1), 5.0 + rank, world)
    out.put((rank, tok, ms, ks, ctx))
    dist.destroy_process_group()


def test_two_rank_aggregation():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(r[1] == 300.0 and r[2] == 6.0 for r in res)       # sum of tokens, max of times, same on every rank
    assert (res[0][3], res[0][4]) != (res[1][3], res[1][4])     # each rank draws its own requests
