"""Plain stand-ins and brute-force references for the sharded-datastore tests: one shard's
retrieval and row gathering by scanning, and the tree that Algorithm 2 and the breadth-first
emission give for an explicit list of candidate rows (Counter of prefixes, full sort).  Written
from the definitions; shares nothing with the CUDA library or the oracle."""
from collections import Counter

import numpy as np


def shard_order(ext, owned):
    """Positions [0, owned) of a shard ordered by their suffixes in the shard's slice `ext`
    (first 32 tokens, a suffix that ends early first, ties by position)."""
    ext = [int(x) for x in ext]
    return sorted(range(owned), key=lambda p: (ext[p:p + 32], p))


def shard_retrieve(ext, order, q_ctx, n_max, n_min):
    """Longest suffix of the context (length n_min..n_max) that occurs at an owned position:
    (n, lo, hi) with [lo, hi) the range of `order` whose suffixes start with it; (0, 0, 0) if none."""
    ext = [int(x) for x in ext]
    ctx = [int(x) for x in q_ctx]
    for n in range(min(n_max, len(ctx)), n_min - 1, -1):
        q = ctx[len(ctx) - n:]
        hits = [i for i, p in enumerate(order) if ext[p:p + n] == q]
        if hits:
            assert hits == list(range(hits[0], hits[-1] + 1))
            return n, hits[0], hits[-1] + 1
    return 0, 0, 0


def shard_rows(ext, order, n, lo, hi, take, m, first_k=False):
    """The `take` sampled candidate rows of a shard's range [lo, hi) for a match of length n."""
    ext = [int(x) for x in ext]
    cnt = hi - lo
    rows = []
    for j in range(take):
        slot = lo + j if (first_k or take >= cnt) else lo + (j * cnt) // take
        p = order[slot]
        rows.append(ext[p + n:p + n + m])
    return rows


def allocation(cnts, K):
    """Rows per shard by the rule of the sharded draft (plain integers)."""
    total = sum(cnts)
    if total <= K:
        return list(cnts)
    out, run = [], 0
    for c in cnts:
        out.append((K * (run + c)) // total - (K * run) // total)
        run += c
    return out


def tree_from_rows(rows, N, ctx_len):
    """Algorithm 2 on an explicit candidate list, then the breadth-first emission: weight of a
    prefix = number of rows that have it; keep the N best by (weight desc, depth asc, path asc);
    order them by (depth, path); parents, ancestor masks, position ids."""
    w = Counter()
    for r in rows:
        for d in range(1, len(r) + 1):
            w[tuple(r[:d])] += 1
    kept = sorted(w, key=lambda p: (-w[p], len(p), p))[:N]
    kept.sort(key=lambda p: (len(p), p))
    index = {p: i for i, p in enumerate(kept)}
    Wm = (N + 31) // 32
    out = {"tokens": np.full(N, -1, np.int32), "parents": np.full(N, -1, np.int32),
           "depth": np.zeros(N, np.int32), "pos_ids": np.full(N, ctx_len, np.int32),
           "node_count": np.zeros(N, np.int32), "mask": np.zeros((N, Wm), np.uint32),
           "n_nodes": len(kept)}
    for i in range(N):
        out["mask"][i, i >> 5] = np.uint32(1 << (i & 31))
    for i, p in enumerate(kept):
        out["tokens"][i] = p[-1]
        out["depth"][i] = len(p)
        out["pos_ids"][i] = ctx_len + len(p) - 1
        out["node_count"][i] = w[p]
        if len(p) > 1:
            par = index[p[:-1]]
            out["parents"][i] = par
            out["mask"][i] |= out["mask"][par]
    return out


def sharded_reference(tokens, world, halo, ctxs, ctx_lens, n_max, n_min, K, m, N):
    """The sharded draft computed directly from its definition, context by context."""
    from paper_2311_08252_b200.sharding import shard_bounds
    shards = []
    for r in range(world):
        b, e = shard_bounds(len(tokens), r, world)
        ext = tokens[b:min(len(tokens), e + halo)]
        shards.append((ext, shard_order(ext, e - b)))
    trees, info = [], []
    for ctx, cl in zip(ctxs, ctx_lens):
        found = [shard_retrieve(ext, order, ctx[:cl], n_max, n_min) for ext, order in shards]
        n_star = max(f[0] for f in found)
        cnts = [(f[2] - f[1]) if (f[0] == n_star and n_star > 0) else 0 for f in found]
        take = allocation(cnts, K)
        rows = []
        for (ext, order), f, t in zip(shards, found, take):
            if t:
                rows += shard_rows(ext, order, n_star, f[1], f[2], t, m)
        trees.append(tree_from_rows(rows, N, cl))
        info.append((n_star, sum(cnts), take))
    return trees, info
