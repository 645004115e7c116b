"""Multi-GPU mode is replicas only (sequences are independent, weights replicated, no data-path
collective): the bench aggregates per-rank results as max of times and sum of tokens.  This checks that
aggregation with two gloo ranks on CPU."""
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


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, toks = bench.aggregate_replicas([10.0 + rank, 20.0 - rank], [5.0 + rank, 7.0], world, device="cpu")
    if rank == 0:
        out.put((ms, toks))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    ms, toks = q.get()
    assert ms == [11.0, 20.0]        # max over ranks of each timing
    assert toks == [11.0, 14.0]      # sum over ranks of each token count
