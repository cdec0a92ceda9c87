"""The draft over a datastore cut into shards (rest_retrieve, rest_gather_rows,
rest_draft_from_runs and the exchange logic between them), several shards on one GPU: bit-exact
against the oracle over the whole datastore wherever the candidate cap does not bind, against
the sharded definition computed by scanning where it does, and against plain rest_draft for a
single shard."""
import threading

import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2311_08252_b200 as rest
import sharded_util as su
from gpu_util import to_dev
from paper_2311_08252_b200.sharding import (SHARD_HALO, ThreadComm, shard_suffix_array, shard_tokens,
                                            sharded_draft_cuda)

pytestmark = pytest.mark.gpu

TREE_KEYS = ("tokens", "parents", "depth", "pos_ids", "node_count", "n_nodes")


def run_sharded(T, vocab, world, ctx, ctx_len, sa_bytes=4, **kw):
    """Cuts T into `world` shards (own suffix array each, built on the device), runs one
    sharded draft with one host thread per shard, returns every shard's (trees, info)."""
    stores = []
    for r in range(world):
        ext, owned = shard_tokens(T, r, world)
        d_ext = to_dev(ext)
        sa = shard_suffix_array(rest.rest_suffix_array_build(d_ext, sa_bytes), owned)
        stores.append(rest.Datastore(d_ext, sa.contiguous(), vocab, validate=True))
    comm = ThreadComm(world)
    d_ctx, d_len = to_dev(ctx), to_dev(np.asarray(ctx_len, np.int32))
    results, errors = [None] * world, []

    def work(r):
        try:
            results[r] = sharded_draft_cuda(comm.view(r), stores[r], d_ctx, d_len, **kw)
        except Exception as e:          # a failed thread must not leave the others at the barrier
            errors.append(e)
            comm._barrier.abort()

    threads = [threading.Thread(target=work, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for s in stores:
        s.close()
    return results


def tree_dict(trees):
    d = {k: getattr(trees, k).cpu().numpy() for k in TREE_KEYS + ("match_n", "match_range", "status")}
    d["mask"] = trees.mask.cpu().numpy().view(np.uint32)
    return d


def test_one_shard_is_rest_draft():
    """With a single shard every piece of the sharded draft must reproduce rest_draft, the
    candidate cap included (the allocation rule reduces to rest_draft's sampling)."""
    w = datagen.WORKLOADS["batched"].scaled(n_tokens=2_000_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    B = 160
    ctx = datagen.make_contexts(w, T, B=B, Lc=48)
    ctx_len = np.full(B, 48, np.int32)
    ctx_len[::9] = np.arange(len(ctx_len[::9])) % 5
    for K, m, N in ((300, 10, 64), (20000, 16, 128), (7, 3, 256)):
        ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, K=K, m=m, N=N)
        trees, info = run_sharded(T, w.vocab, 1, ctx, ctx_len, K=K, m=m, N=N)[0]
        got = tree_dict(trees)
        for key in TREE_KEYS + ("mask", "match_n", "status"):
            assert np.array_equal(got[key], ref[key]), (K, key)
        assert np.array_equal(got["match_range"][:, 1], ref["match_range"][:, 1] - ref["match_range"][:, 0])
        assert (ref["match_range"][:, 1] - ref["match_range"][:, 0] > K).sum() > (8 if K <= 300 else 0)


@pytest.mark.parametrize("world,sa_bytes", [(2, 4), (3, 8)])
def test_shards_reproduce_the_whole_datastore_where_the_cap_does_not_bind(world, sa_bytes):
    w = datagen.WORKLOADS["single_stream"].scaled(n_tokens=3_000_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    B, K = 128, 32768 // world
    ctx = datagen.make_contexts(w, T, B=B, Lc=40)
    # contexts cut out around the shard boundaries: their matches straddle two shards
    cut = len(T) // world
    for i in range(8):
        ctx[i] = T[cut - 30 + 3 * i:cut + 10 + 3 * i]
    ctx_len = np.full(B, 40, np.int32)
    ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, K=K, m=w.m, N=w.N)
    hits = ref["match_range"][:, 1] - ref["match_range"][:, 0]
    results = run_sharded(T, w.vocab, world, ctx, ctx_len, sa_bytes=sa_bytes, K=K, m=w.m, N=w.N)
    free = hits <= K
    assert free.sum() > B // 2
    for trees, info in results:                      # every shard holds the same, complete result
        got = tree_dict(trees)
        assert np.array_equal(got["match_n"], ref["match_n"])
        assert np.array_equal(got["match_range"][:, 1], hits)
        for key in TREE_KEYS + ("mask",):
            assert np.array_equal(got[key][free], ref[key][free]), key
        assert (info["taken"].sum(dim=0).cpu().numpy() == np.minimum(hits, K)).all()


def test_cap_binding_across_shards_follows_the_sharded_definition():
    rng = np.random.default_rng(9)
    vocab, n_tok, B, Lc = 3, 5000, 20, 10
    T = rng.integers(0, vocab, n_tok).astype(np.int32)
    ctx = rng.integers(0, vocab, (B, Lc)).astype(np.int32)
    ctx_len = np.full(B, Lc, np.int32)
    kw = dict(n_max=4, n_min=2, K=50, m=6, N=40)
    want, want_info = su.sharded_reference(T, 2, SHARD_HALO, ctx, ctx_len, kw["n_max"], kw["n_min"],
                                           kw["K"], kw["m"], kw["N"])
    assert sum(i[1] > kw["K"] for i in want_info) > B // 2
    trees, info = run_sharded(T, vocab, 2, ctx, ctx_len, **kw)[1]
    got = tree_dict(trees)
    for b in range(B):
        assert int(got["match_n"][b]) == want_info[b][0] and int(got["match_range"][b, 1]) == want_info[b][1]
        assert info["taken"][:, b].tolist() == want_info[b][2]
        for key in TREE_KEYS + ("mask",):
            assert np.array_equal(got[key][b], want[b][key]), (b, key)


def test_runs_out_of_order_are_reported():
    B, R, Kr, m, N = 2, 2, 8, 4, 16
    rows = np.zeros((B, R, Kr, m), np.int32)
    lens = np.full((B, R, Kr), m, np.int32)
    for b in range(B):
        for r in range(R):
            rows[b, r, :, 0] = np.arange(Kr) * 2 + r      # sorted runs, interleaving when merged
    rows[1, 0, 3, 0] = 0                                   # context 1: run 0 is not in order
    runs = np.full((B, R), Kr, np.int32)
    out = rest.rest_draft_from_runs(to_dev(rows), to_dev(lens), to_dev(runs), to_dev(np.array([5, 5], np.int32)),
                                    N=N)
    torch.cuda.synchronize()
    assert out.status.tolist() == [0, 2] and out.n_nodes.tolist() == [N, 0]
    assert out.tokens[0].tolist() == list(range(16)) and (out.tokens[1] == -1).all()
    assert (out.depth[0] == 1).all() and (out.node_count[0] == 1).all()
