"""Host logic of bench.py: layer sharding and the max-over-ranks reduction, on 2 gloo ranks."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_shard_layers_partition():
    for world in (1, 2, 4, 8):
        got = sorted(sum((bench.shard_layers(28, world, r) for r in range(world)), []))
        assert got == list(range(28))
        sizes = [len(bench.shard_layers(28, world, r)) for r in range(world)]
        assert max(sizes) - min(sizes) <= 1


def _worker(rank, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE="2")
    dist.init_process_group("gloo", rank=rank, world_size=2)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
    layers = bench.shard_layers(28, 2, rank)
    out.put((rank, ms, layers))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert sorted(res[0][2] + res[1][2]) == list(range(28))


def test_max_over_ranks_single_process():
    assert bench.max_over_ranks(3.5, None) == 3.5
