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


def test_kv_head_shards_partition_the_heads():
    """Every KV head and its query heads land on exactly one rank; sizes differ by at most one."""
    sys.path.insert(0, ROOT)
    import importlib.util

    spec = importlib.util.spec_from_file_location(
        "_sharding", os.path.join(ROOT, "paper_2503_03588_b200", "sharding.py"))
    sh = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(sh)
    for (hq, hkv) in [(28, 4), (8, 8), (16, 2), (7, 1)]:
        for world in (1, 2, 3, 4, 8):
            seen_q, seen_k, sizes = [], [], []
            for rank in range(world):
                qs, ks = sh.kv_head_shard(hq, hkv, world, rank)
                assert (qs.stop - qs.start) == (ks.stop - ks.start) * (hq // hkv)
                assert qs.start == ks.start * (hq // hkv)
                seen_q += list(range(qs.start, qs.stop))
                seen_k += list(range(ks.start, ks.stop))
                sizes.append(ks.stop - ks.start)
            assert seen_q == list(range(hq)) and seen_k == list(range(hkv))
            assert max(sizes) - min(sizes) <= 1


def _shard_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import importlib.util

    spec = importlib.util.spec_from_file_location(
        "_sharding", os.path.join(ROOT, "paper_2503_03588_b200", "sharding.py"))
    sh = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(sh)
    # Each rank marks the heads it owns in a head-indexed vector; the sum over ranks must be all ones
    # (this all-reduce is the test's bookkeeping: the operator itself exchanges nothing).
    qs, ks = sh.kv_head_shard(28, 4, world, rank)
    mark = torch.zeros(28 + 4)
    mark[qs] += 1
    mark[28 + ks.start:28 + ks.stop] += 1
    dist.all_reduce(mark)
    out.put((rank, mark.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_kv_head_sharding_world_size_2():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = [out.get(timeout=120) for _ in range(2)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, mark in res:
        assert mark == [1.0] * 32
