"""The one exchange step of the head-sharded multi-GPU forward, on CPU ranks (gloo, world
size 2 and 3): token shards of the routing results are all-gathered into the same [B, N, k]
tensors on every rank, ragged shard sizes included."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _expected(B, N, k):
    g = torch.Generator().manual_seed(5)
    gid = torch.randint(0, 7, (B, N, k), generator=g, dtype=torch.int32)
    gate = torch.rand(B, N, k, generator=g)
    return gid, gate


def _worker(rank, world, port, N, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2510_18692_b200.sharded import gather_routing, shard_bounds
    gid, gate = _expected(2, N, 2)
    lo, hi = shard_bounds(N, world, rank)
    got_gid, got_gate = gather_routing(gid[:, lo:hi].contiguous(), gate[:, lo:hi].contiguous(), N)
    out.put((rank, bool(torch.equal(got_gid, gid)), bool(torch.equal(got_gate, gate)), (lo, hi)))
    dist.barrier()
    dist.destroy_process_group()


def _run(world, N):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() + world * 37 + N) % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, N, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return res


def test_routing_all_gather_world2():
    res = _run(2, 1001)                                  # shards of 501 and 500 tokens
    assert [r[1:3] for r in res] == [(True, True)] * 2
    assert [r[3] for r in res] == [(0, 501), (501, 1001)]


def test_routing_all_gather_world3_ragged():
    res = _run(3, 100)                                   # 34 + 33 + 33
    assert [r[1:3] for r in res] == [(True, True)] * 3
    assert [r[3] for r in res] == [(0, 34), (34, 67), (67, 100)]


def test_shard_bounds_cover_everything_once():
    sys.path.insert(0, ROOT)
    from paper_2510_18692_b200.sharded import shard_bounds
    for n in (0, 1, 7, 40, 561600):
        for parts in (1, 2, 3, 8):
            b = [shard_bounds(n, parts, i) for i in range(parts)]
            assert b[0][0] == 0 and b[-1][1] == n
            assert all(b[i][1] == b[i + 1][0] for i in range(parts - 1))
            assert max(h - l for l, h in b) - min(h - l for l, h in b) <= 1
