"""World-size-2 gloo run of the benchmark's replica aggregation (job time = max over ranks, job work =
sum over ranks): the only multi-rank logic of this library, which has no exchange step."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    ms, flops = bench.aggregate(3.0 + rank, 100.0 * (rank + 1))
    out.put((rank, ms, flops))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_world_size_2():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, flops in res:
        assert ms == 4.0 and flops == 300.0


def test_aggregate_without_process_group_is_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.aggregate(1.5, 7.0) == (1.5, 7.0)
