"""N > 1 plumbing of the benchmark on CPU (gloo, world size 2): per-rank workloads and the
max-over-ranks / sum-over-ranks reduction.  The data path itself has no collective."""
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
    from workloads import generate, get_config
    w = bench.rank_workload(get_config("c0"), rank)
    x = generate(w)
    times, flops = bench.reduce_over_ranks([10.0 + rank, 5.0 - rank], 100.0 * (rank + 1), "cpu", dist)
    gathered = [None] * world
    dist.all_gather_object(gathered, (w.seed, float(x["q"].double().sum())))
    # strong scaling: this rank's heads of the ONE workload, generated locally
    w1 = get_config("c0")
    h0, h1 = bench.head_shard(w1.H, rank, world)
    shard = generate(w1, heads=(h0, h1))
    shards = [None] * world
    dist.all_gather_object(shards, (h0, h1, {n: shard[n].clone() for n in ("q", "k", "v")}))
    dist.barrier()
    if rank == 0:
        torch.save({"times": times, "flops": flops, "gathered": gathered, "shards": shards}, out)
    dist.destroy_process_group()


def test_two_ranks_reduce_and_shard(tmp_path):
    out = str(tmp_path / "r.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["times"] == [11.0, 5.0]                 # maximum over ranks, element-wise
    assert r["flops"] == 300.0                        # work adds up
    (s0, q0), (s1, q1) = r["gathered"]
    assert s0 == 0 and s1 == 1000 and q0 != q1        # same shape, different data per rank
    # head shards: the ranges tile 0..H-1 in rank order and hold the single-GPU workload's bits
    from workloads import generate, get_config
    w = get_config("c0")
    full = generate(w)
    pos = 0
    for (h0, h1, x) in r["shards"]:
        assert h0 == pos and h1 > h0
        for n in ("q", "k", "v"):
            assert torch.equal(x[n], full[n][:, h0:h1])
        pos = h1
    assert pos == w.H


def test_head_shards_tile_the_heads():
    sys.path.insert(0, ROOT)
    import bench
    for H in (1, 2, 5, 32, 33):
        for world in (1, 2, 3, 4, 8):
            if world > H:
                continue
            r = [bench.head_shard(H, i, world) for i in range(world)]
            assert r[0][0] == 0 and r[-1][1] == H
            assert all(a[1] == b[0] for a, b in zip(r, r[1:]))
            sizes = [b - a for a, b in r]
            assert max(sizes) - min(sizes) <= 1 and min(sizes) >= 1


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks([1.0, 2.0], 7.0, "cpu", None) == ([1.0, 2.0], 7.0)
