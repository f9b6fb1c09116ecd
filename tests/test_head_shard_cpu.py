"""Head-sharded runs on CPU: the split of the heads over ranks, and two gloo ranks that each run the oracle's step on
their own heads of a seeded workload; gathered, the shards reproduce the un-sharded result head for head (Eq. 1 is per
head: no exchange between ranks exists on the data path)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2602_01801_b200 import synth                      # noqa: E402
from paper_2602_01801_b200.fastar import head_shard          # noqa: E402


def test_head_shard_covers_every_head_once():
    for H in (1, 3, 12, 40):
        for world in (1, 2, 3, 8):
            ranges = [head_shard(H, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == H
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))         # contiguous, no gap, no overlap
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    assert head_shard(12, 8, 0) == (0, 2) and head_shard(12, 8, 4) == (8, 9) and head_shard(40, 8, 7) == (35, 40)
    with pytest.raises(ValueError):
        head_shard(4, 2, 2)


def _step_on_heads(cfg, w):
    """The oracle's update + AnnSA on every head `w` holds; returns [heads][n][d] outputs and the cache lengths."""
    from oracle import fastar_oracle as O
    R = w.lsh_projection().astype(np.float64)
    outs, lens = [], []
    Q, K, V = w.chunk(0)
    for h in range(K.shape[0]):
        cache = O.HeadCache(cfg.capacity, cfg.head_dim)
        O.tempcache_update(cache, K[h], V[h], cfg.frame_len, 2.0)
        Q1, K1, V1 = (x[h] for x in w.chunk(1))
        O.tempcache_update(cache, K1, V1, cfg.frame_len, cfg.tau)
        outs.append(O.annsa(Q1, cache, R, cfg.lsh_tables, cfg.lsh_bits, cfg.block, cfg.block, cfg.keep_blocks)["out"])
        lens.append(cache.L)
    return np.stack(outs), lens


def _config():
    return synth.small_config(num_heads=3, grid_h=6, grid_w=10, frames_per_chunk=2, capacity=512, block=64, keep_blocks=3,
                              head_dim=64)


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = _config()
    h0, h1 = head_shard(cfg.num_heads, world, rank)
    out, lens = _step_on_heads(cfg, bench.HeadSlice(synth.Workload(cfg), h0, h1))
    gathered = [None] * world
    dist.all_gather_object(gathered, (h0, h1, out, lens))
    if rank == 0:
        q.put(gathered)
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_step():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    gathered = q.get(timeout=300)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = _config()
    want, want_lens = _step_on_heads(cfg, synth.Workload(cfg))
    assert [(a, b) for a, b, _, _ in gathered] == [(0, 2), (2, 3)]               # 3 heads over 2 ranks: 2 + 1
    got = np.concatenate([o for _, _, o, _ in gathered])
    assert got.shape == want.shape and np.array_equal(got, want)
    assert sum((l for _, _, _, l in gathered), []) == want_lens
