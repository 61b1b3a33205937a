"""Multi-rank host logic on CPU (gloo, world size 2): batch shards, per-shard routing equals the global
routing restricted to the shard, histogram and step-time reductions."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import dsn_oracle as O
    from paper_2109_10060_b200.sharding import max_over_ranks, reduce_histogram, shard_range
    B, T, R, C = 37, 5, 3, 16
    g = np.random.default_rng(123)                      # same draw on every rank
    idx = g.integers(0, T, size=B).astype(np.int32)
    x = g.standard_normal((B, R, C))
    W = g.standard_normal((C, C))
    k_in, k_out = [4, 8, 12, 16, 16], [16, 12, 8, 4, 16]
    lo, hi = shard_range(B, rank, world)
    counts, offsets, perm, inv = O.route(idx[lo:hi], T)   # per-shard routing
    y_shard = O.sliced_linear(x[lo:hi], W, idx[lo:hi], k_in, k_out, fill=0.0)
    # histogram over all ranks equals the global histogram
    hist = reduce_histogram(torch.from_numpy(counts.astype(np.int64)), dist)
    assert hist.tolist() == np.bincount(idx, minlength=T).tolist() and int(hist.sum()) == B
    # outputs gathered in rank order equal the unsharded result
    parts = [None] * world
    dist.all_gather_object(parts, (lo, hi, y_shard))
    y = np.concatenate([p[2] for p in sorted(parts, key=lambda p: p[0])], axis=0)
    np.testing.assert_array_equal(y, O.sliced_linear(x, W, idx, k_in, k_out, fill=0.0))
    # per-shard grouping is the global stable grouping restricted to the shard
    gperm = O.route(idx, T)[2]
    mine = [int(i) - lo for i in gperm if lo <= i < hi]
    by_group = [i for t in range(T) for i in mine if idx[lo + i] == t]
    assert perm.tolist() == by_group
    t = max_over_ranks(torch.tensor([1.0 + rank], dtype=torch.float64), dist)
    assert float(t) == float(world)
    out.put((rank, lo, hi))
    dist.destroy_process_group()


def test_two_rank_batch_sharding_on_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    got = sorted(out.get(timeout=10) for _ in range(2))
    assert got == [(0, 0, 19), (1, 19, 37)]


def test_shard_ranges_cover_the_batch():
    from paper_2109_10060_b200.sharding import shard_range
    for B in (0, 1, 7, 128, 1025):
        for world in (1, 2, 3, 8):
            spans = [shard_range(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
