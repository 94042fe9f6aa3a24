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


def test_shard_tokens_partition():
    for n, world in ((262144, 8), (1001, 4), (5, 8), (0, 2)):
        spans = [bench.shard_tokens(n, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == n
        assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
        sizes = [b - a for a, b in spans]
        assert max(sizes) - min(sizes) <= 1


def _shard_worker(rank, port, out):
    """Two ranks score halves of the tokens with the CPU oracle; after the exchange both hold the components of
    the whole set."""
    import numpy as np
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle as O
    from _util import random_layer
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE="2")
    dist.init_process_group("gloo", rank=rank, world_size=2)
    r = np.random.default_rng(7)
    layer = random_layer(r, d=6, d_ff=(4, 5, 3), n_shared=1, top_k=1, shared_gate=True)
    X = r.standard_normal((41, 6))
    t0, t1 = bench.shard_tokens(41, 2, rank)
    p2, pinf, w2 = O.camera_components(layer, X[t0:t1])
    a, b = torch.from_numpy(p2.copy()), torch.from_numpy(pinf.copy())
    bench.reduce_components(a, b, dist)
    full = O.camera_components(layer, X)
    out.put((rank, float(np.abs(a.numpy() - full[0]).max()), float(np.abs(b.numpy() - full[1]).max()),
             float(np.abs(O.energy(a.numpy(), b.numpy(), w2, 0.95) - O.energy(*full, 0.95)).max())))
    dist.barrier()
    dist.destroy_process_group()


def test_token_sharded_components_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_shard_worker, args=(r, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, e2, einf, ee in res:
        assert e2 < 1e-12 and einf == 0.0 and ee < 1e-12
