"""Multi-rank host logic on CPU (gloo, world size 2): context shards are disjoint and cover
the batch, per-shard results concatenate to the unsharded result, timing is the max over ranks."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2311_08252_b200.sharding import max_over_ranks, shard_bounds, whole_job_throughput


def test_shard_bounds_cover_and_are_disjoint():
    for n in (0, 1, 7, 256, 257):
        for world in (1, 2, 3, 8):
            cuts = [shard_bounds(n, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            for a, b in zip(cuts, cuts[1:]):
                assert a[1] == b[0]
            sizes = [e - s for s, e in cuts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_bounds(4, 2, 2)
    assert whole_job_throughput(4, 10, 2, 0.5) == 160.0


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import datagen
    import oracle
    w = datagen.WORKLOADS["tiny"].scaled(n_tokens=100_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    ctx = datagen.make_contexts(w, T, B=37, Lc=32)          # the global batch, same on all ranks
    s, e = shard_bounds(37, rank, world)
    mine = oracle.draft(T, sa, w.vocab, ctx[s:e], np.full(e - s, 32), K=w.K, m=w.m, N=w.N)
    gathered = [None] * world
    dist.all_gather_object(gathered, (s, e, mine["tokens"], mine["n_nodes"]))
    t = max_over_ranks(1.0 + rank, dist)
    if rank == 0:
        full = oracle.draft(T, sa, w.vocab, ctx, np.full(37, 32), K=w.K, m=w.m, N=w.N)
        tok = np.concatenate([g[2] for g in gathered])
        nn = np.concatenate([g[3] for g in gathered])
        ok = np.array_equal(tok, full["tokens"]) and np.array_equal(nn, full["n_nodes"])
        ok = ok and [g[:2] for g in gathered] == [shard_bounds(37, r, world) for r in range(world)]
        ok = ok and t == float(world)
        open(os.path.join(out_dir, "ok"), "w").write("1" if ok else "0")
    dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert open(tmp_path / "ok").read() == "1"
