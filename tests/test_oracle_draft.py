"""Pins for the draft side of the CPU oracle (Algorithm 1, Algorithm 2, BFS + mask).

The oracle is checked against things other than itself: a hand-worked example, brute-force
substring scans written directly from the definitions, and structural invariants of a Trie.
"""
import os
from collections import Counter

import numpy as np
import pytest

import datagen
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def read_golden():
    rec = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        rec[key] = vals
    return rec


def ints(v):
    return [int(x, 0) for x in v]


def test_worked_example_draft():
    g = read_golden()
    T = np.array(ints(g["T"]), np.int32)
    sa = oracle.suffix_array(T)
    assert sa.tolist() == ints(g["SA"])
    prm = dict(kv.split("=") for kv in g["PARAMS"])
    ctx = np.array(ints(g["CTX"]), np.int32)
    out = oracle.draft(T, sa, 10, ctx[None], [ctx.size], n_max=int(prm["n_max"]),
                       n_min=int(prm["n_min"]), K=int(prm["K"]), m=int(prm["m"]), N=int(prm["N"]))
    assert out["match_n"][0] == int(g["MATCH_N"][0])
    assert out["match_range"][0].tolist() == ints(g["RANGE"])
    assert out["tokens"][0].tolist() == ints(g["TOKENS"])
    assert out["parents"][0].tolist() == ints(g["PARENTS"])
    assert out["depth"][0].tolist() == ints(g["DEPTH"])
    assert out["pos_ids"][0].tolist() == ints(g["POS_IDS"])
    assert out["mask"][0, :, 0].tolist() == ints(g["MASK"])
    assert out["node_count"][0].tolist() == ints(g["COUNTS"])
    assert out["n_nodes"][0] == int(g["N_NODES"][0])
    assert out["status"][0] == 0


def test_worked_example_accept():
    g = read_golden()
    tokens = np.array([ints(g["TOKENS"])], np.int32)
    parents = np.array([ints(g["PARENTS"])], np.int32)
    for tag in ("A", "B"):
        ver = np.array([ints(g["VERIFIER_" + tag])], np.int32)
        al, an, ot = oracle.accept(tokens, parents, [4], ver, max_depth=3)
        want_nodes = ints(g["ACCEPT_NODES_" + tag])
        want_out = ints(g["OUT_TOKENS_" + tag])
        assert al[0] == len(want_nodes)
        assert an[0, :al[0]].tolist() == want_nodes
        assert (an[0, al[0]:] == -1).all()
        assert ot[0, :al[0] + 1].tolist() == want_out
        assert (ot[0, al[0] + 1:] == -1).all()


# ---------------------------------------------------------------------------------------
# Brute force, straight from the definitions: substring scans, Counter of prefixes.
# ---------------------------------------------------------------------------------------
def brute_sorted_suffixes(T):
    T = list(T)
    return sorted(range(len(T)), key=lambda p: T[p:])   # shorter list sorts first on ties


def brute_draft(T, ctx, n_max, n_min, K, m, N, sample_mode=0):
    T = list(map(int, T))
    ctx = list(map(int, ctx))
    n_tok = len(T)
    for n in range(min(n_max, len(ctx)), n_min - 1, -1):
        if n < 1:
            break
        q = ctx[len(ctx) - n:]
        occ = [p for p in range(n_tok) if T[p:p + n] == q]
        if occ:
            break
    else:
        return None
    if not occ:
        return None
    occ.sort(key=lambda p: T[p:])          # suffix-array order of the matches
    cnt = len(occ)
    if cnt > K:
        occ = [occ[(j * cnt) // K] if sample_mode == 0 else occ[j] for j in range(K)]
    weights = Counter()
    for p in occ:
        cont = T[p + n:p + n + m]
        for d in range(1, len(cont) + 1):
            weights[tuple(cont[:d])] += 1
    ranked = sorted(weights.items(), key=lambda kv: (-kv[1], len(kv[0]), kv[0]))[:N]
    kept = sorted((path for path, _ in ranked), key=lambda p: (len(p), p))
    index = {p: i for i, p in enumerate(kept)}
    res = dict(n=n, cnt=cnt, tokens=[p[-1] for p in kept],
               parents=[index.get(p[:-1], -2) if len(p) > 1 else -1 for p in kept],
               depth=[len(p) for p in kept], counts=[weights[p] for p in kept], paths=kept)
    masks = []
    for p in kept:
        bits = 0
        for d in range(1, len(p) + 1):
            bits |= 1 << index[p[:d]]
        masks.append(bits)
    res["mask"] = masks
    return res


def mask_as_int(row):
    v = 0
    for w, word in enumerate(row.tolist()):
        v |= int(word) << (32 * w)
    return v


@pytest.mark.parametrize("seed,vocab,n_tok,K,m,N", [
    (1, 3, 400, 5000, 4, 16),
    (2, 4, 1500, 5000, 6, 40),
    (3, 2, 300, 5000, 10, 64),
    (4, 5, 2500, 7, 5, 24),        # K binds: strided sampling
    (5, 3, 900, 20, 8, 70),        # K binds, N spans three mask words
    (6, 8, 4096, 5000, 10, 64),
])
def test_draft_matches_brute_force(seed, vocab, n_tok, K, m, N):
    rng = np.random.default_rng(seed)
    T = rng.integers(0, vocab, n_tok).astype(np.int32)
    sa = oracle.suffix_array(T)
    assert sa.tolist() == brute_sorted_suffixes(T)
    B, Lc = 12, 24
    ctx = rng.integers(0, vocab, (B, Lc)).astype(np.int32)
    # a few contexts copied from the datastore so that long matches occur, one near the end
    for b in range(0, B, 3):
        p = int(rng.integers(0, n_tok - Lc))
        ctx[b] = T[p:p + Lc]
    ctx[1] = T[n_tok - Lc - 2:n_tok - 2]
    ctx_len = np.full(B, Lc, np.int32)
    ctx_len[2] = 5
    ctx_len[3] = 1                          # shorter than n_min -> empty tree
    for mode in (0, 1):
        out = oracle.draft(T, sa, vocab, ctx, ctx_len, n_max=16, n_min=2, K=K, m=m, N=N,
                           sample_mode=mode)
        for b in range(B):
            ref = brute_draft(T, ctx[b, :ctx_len[b]], 16, 2, K, m, N, mode)
            if ref is None:
                assert out["n_nodes"][b] == 0 and out["match_n"][b] == 0
                assert (out["tokens"][b] == -1).all()
                continue
            nn = len(ref["tokens"])
            assert out["match_n"][b] == ref["n"]
            assert out["match_range"][b, 1] - out["match_range"][b, 0] == ref["cnt"]
            assert out["n_nodes"][b] == nn
            assert out["tokens"][b, :nn].tolist() == ref["tokens"]
            assert out["parents"][b, :nn].tolist() == ref["parents"]
            assert out["depth"][b, :nn].tolist() == ref["depth"]
            assert out["node_count"][b, :nn].tolist() == ref["counts"]
            assert [mask_as_int(r) for r in out["mask"][b, :nn]] == ref["mask"]
            assert (out["pos_ids"][b, :nn] == ctx_len[b] + out["depth"][b, :nn] - 1).all()
            # padding slots
            assert (out["tokens"][b, nn:] == -1).all() and (out["parents"][b, nn:] == -1).all()
            assert (out["depth"][b, nn:] == 0).all() and (out["pos_ids"][b, nn:] == ctx_len[b]).all()
            for i in range(nn, N):
                assert mask_as_int(out["mask"][b, i]) == 1 << i


def test_retrieve_is_longest_match_with_occurrence_count():
    rng = np.random.default_rng(11)
    T = rng.integers(0, 3, 2000).astype(np.int32)
    Tl = T.tolist()
    sa = oracle.suffix_array(T)
    for trial in range(200):
        ctx = rng.integers(0, 3, 20).astype(np.int32)
        n, lo, hi = oracle.retrieve(T, sa, ctx, 16, 2)
        best = 0
        for k in range(16, 1, -1):
            q = ctx[-k:].tolist()
            c = sum(1 for p in range(len(Tl)) if Tl[p:p + k] == q)
            if c:
                best, bc = k, c
                break
        assert n == best
        if best:
            assert hi - lo == bc
            for slot in range(lo, hi):
                p = int(sa[slot])
                assert Tl[p:p + n] == ctx[-n:].tolist()


def test_trie_invariants_on_synthetic_workload():
    w = datagen.WORKLOADS["tiny"].scaled(n_tokens=200_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab, W=32)
    ctx = datagen.make_contexts(w, T, B=64, Lc=64)
    out = oracle.draft(T, sa, w.vocab, ctx, np.full(64, 64), K=w.K, m=w.m, N=w.N)
    assert (out["status"] == 0).all()
    assert (out["n_nodes"] > 0).sum() > 16
    for b in range(64):
        nn = int(out["n_nodes"][b])
        par, dep, cnt, tok = (out[k][b] for k in ("parents", "depth", "node_count", "tokens"))
        lo, hi = out["match_range"][b]
        Kp = min(hi - lo, w.K)
        if nn:
            # depth-1 weights add up to the number of candidates that have a first token
            d1 = cnt[:nn][dep[:nn] == 1].sum()
            assert d1 <= Kp
            if nn < w.N:       # whole trie kept: every candidate with a first token is counted
                p = sa[lo:hi]
                assert d1 == (p + out["match_n"][b] < T.size).sum()
        seen = set()
        for i in range(nn):
            assert par[i] < i
            if par[i] >= 0:
                assert dep[i] == dep[par[i]] + 1
                assert cnt[par[i]] >= cnt[i]                       # ancestor-closed selection
                assert mask_as_int(out["mask"][b, i]) == mask_as_int(out["mask"][b, par[i]]) | (1 << i)
            else:
                assert dep[i] == 1 and mask_as_int(out["mask"][b, i]) == 1 << i
            assert bin(mask_as_int(out["mask"][b, i])).count("1") == dep[i]
            assert (par[i], tok[i]) not in seen                     # siblings are distinct
            seen.add((par[i], tok[i]))
        # children of one parent are contiguous-in-order and ascend by token
        for i in range(1, nn):
            if dep[i] == dep[i - 1]:
                assert (par[i - 1], tok[i - 1]) < (par[i], tok[i])
            else:
                assert dep[i] == dep[i - 1] + 1
        # a parent's weight is at least the sum of its kept children
        for i in range(nn):
            kids = [j for j in range(nn) if par[j] == i]
            assert cnt[i] >= sum(cnt[j] for j in kids)


def test_results_depend_only_on_the_first_32_tokens_of_each_suffix():
    # A suffix array ordered on 32-token windows (ties by position) drafts the same trees
    # as the true suffix array: tied entries have identical n+m-token windows.
    rng = np.random.default_rng(5)
    T = (rng.integers(0, 2, 6000) * rng.integers(0, 2, 6000)).astype(np.int32)   # long repeats
    T[1000:1400] = 0
    sa_true = oracle.suffix_array(T)
    sa_w = datagen.build_suffix_array(T, 2, W=32)
    sa_full = datagen.build_suffix_array(T, 2, W=0)
    assert sa_full.tolist() == sa_true.tolist()
    assert datagen.verify_suffix_array(T, sa_w, 32) == 0
    assert sa_w.tolist() != sa_true.tolist()
    ctx = rng.integers(0, 2, (32, 40)).astype(np.int32)
    ctx[0] = 0
    for K in (5000, 50):
        a = oracle.draft(T, sa_true, 2, ctx, np.full(32, 40), K=K, m=10, N=64)
        b = oracle.draft(T, sa_w, 2, ctx, np.full(32, 40), K=K, m=10, N=64)
        for key in a:
            assert np.array_equal(a[key], b[key]), key


def test_prepending_context_only_shifts_position_ids():
    rng = np.random.default_rng(7)
    T = rng.integers(0, 4, 3000).astype(np.int32)
    sa = oracle.suffix_array(T)
    ctx = rng.integers(0, 4, (8, 48)).astype(np.int32)
    a = oracle.draft(T, sa, 4, ctx[:, 16:], np.full(8, 32), m=6, N=32)
    b = oracle.draft(T, sa, 4, ctx, np.full(8, 48), m=6, N=32)
    for key in a:
        if key == "pos_ids":
            assert np.array_equal(a[key] + 16, b[key])
        else:
            assert np.array_equal(a[key], b[key]), key


def test_bad_inputs_set_status():
    T = np.array([1, 2, 3, 1, 2, 4, 1, 2, 3, 5], np.int32)
    sa = oracle.suffix_array(T)
    ctx = np.array([[9, 7, 1, 2], [9, 7, 1, 99], [9, 7, -1, 2]], np.int32)
    out = oracle.draft(T, sa, 10, ctx, [4, 4, 4], m=3, N=4)
    assert out["status"].tolist() == [0, 1, 1]
    assert out["n_nodes"].tolist() == [4, 0, 0]
    # an out-of-range suffix-array entry met while gathering candidates is reported
    Z = np.zeros(64, np.int32)
    saz = oracle.suffix_array(Z)
    assert saz.tolist() == list(range(63, -1, -1))
    ok = oracle.draft(Z, saz, 1, np.zeros((1, 20), np.int32), [20], m=3, N=4)
    assert ok["status"].tolist() == [0] and ok["match_range"][0].tolist() == [15, 64]
    bad = saz.copy()
    bad[40] = 1000          # interior of the match range, not touched by the bisection
    out = oracle.draft(Z, bad, 1, np.zeros((1, 20), np.int32), [20], m=3, N=4)
    assert out["status"].tolist() == [2] and out["n_nodes"].tolist() == [0]
