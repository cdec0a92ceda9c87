"""Parity of rest_draft (CUDA, through the C ABI) with the CPU oracle: bit-exact match
lengths, ranges, tokens, parents, depths, position ids, masks, weights and status."""
import numpy as np
import pytest

import datagen
import oracle
import paper_2311_08252_b200 as rest
from gpu_util import assert_draft_equal, gpu_draft

pytestmark = pytest.mark.gpu

# the single-context and the batched suffix-array search must give the same trees
SEARCHES = (rest.REST_SEARCH_SINGLE, rest.REST_SEARCH_BATCHED)


def test_worked_example():
    T = np.array([1, 2, 3, 1, 2, 4, 1, 2, 3, 5], np.int32)
    sa = oracle.suffix_array(T).astype(np.int32)
    ctx = np.array([[9, 7, 1, 2]], np.int32)
    got, _ = gpu_draft(T, sa, 10, ctx, [4], validate=True, m=3, N=4)
    assert got["tokens"][0].tolist() == [3, 4, 1, 5]
    assert got["parents"][0].tolist() == [-1, -1, 0, 0]
    assert got["mask"][0, :, 0].tolist() == [1, 2, 5, 9]
    assert got["node_count"][0].tolist() == [2, 1, 1, 1]
    assert got["match_n"][0] == 2 and got["match_range"][0].tolist() == [0, 3]


@pytest.mark.parametrize("seed,vocab,n_tok,K,m,N,sa_bytes", [
    (1, 3, 400, 5000, 4, 16, 4),
    (2, 4, 1500, 5000, 6, 40, 8),
    (3, 2, 3000, 5000, 10, 64, 4),      # binary alphabet: thousands of matches, deep shared prefixes
    (4, 5, 2500, 7, 5, 24, 4),          # K binds
    (5, 3, 9000, 600, 16, 128, 8),      # K binds, rows span two gather iterations, N = 128, m = 16
    (6, 8, 4096, 5000, 10, 64, 4),
    (7, 2, 40000, 20000, 16, 128, 4),   # stress shape: K = 20000, m = 16
    (8, 3, 70000, 32768, 1, 1, 4),      # extremes: K max, m = 1, N = 1
    (9, 3, 30000, 20000, 16, 256, 4),   # N = 256: the largest tree
    (10, 4, 9000, 5000, 12, 200, 8),    # N = 200, not a multiple of 32
])
def test_small_alphabets_match_oracle(seed, vocab, n_tok, K, m, N, sa_bytes):
    rng = np.random.default_rng(seed)
    T = rng.integers(0, vocab, n_tok).astype(np.int32)
    sa = datagen.build_suffix_array(T, vocab, W=32, sa_bytes=sa_bytes)
    B, Lc = 40, 24
    ctx = rng.integers(0, vocab, (B, Lc)).astype(np.int32)
    for b in range(0, B, 3):
        p = int(rng.integers(0, n_tok - Lc))
        ctx[b] = T[p:p + Lc]
    ctx[1] = T[n_tok - Lc - 2:n_tok - 2]          # continuations cut by the end of the stream
    ctx[4] = T[n_tok - Lc:]                        # match ends exactly at the end
    ctx_len = rng.integers(0, Lc + 1, B).astype(np.int32)
    ctx_len[:8] = Lc
    for mode in (0, 1):
        kw = dict(K=K, m=m, N=N, sample_mode=mode)
        ref = oracle.draft(T, sa, vocab, ctx, ctx_len, **kw)
        for search in SEARCHES:
            for index in (True, False):
                got, _ = gpu_draft(T, sa, vocab, ctx, ctx_len, validate=True, index=index, search=search, **kw)
                assert_draft_equal(got, ref, f"mode {mode}, search {search:#x}, index {index}")
        got, _ = gpu_draft(T, sa, vocab, ctx, ctx_len, search=rest.REST_SEARCH_BATCHED, workspace=False, **kw)
        assert_draft_equal(got, ref, f"mode {mode}, batched in one launch")


@pytest.mark.parametrize("name,n_tok,B", [
    ("tiny", 1_000_000, 256), ("single_stream", 3_000_000, 128), ("batched", 2_000_000, 256),
    ("large", 2_000_000, 64), ("stress", 2_000_000, 128)])
def test_workload_recipes_match_oracle(name, n_tok, B):
    w = datagen.WORKLOADS[name].scaled(n_tokens=n_tok)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab, W=32, sa_bytes=w.sa_bytes)
    ctx = datagen.make_contexts(w, T, B=B, Lc=min(w.Lc, 512))
    ctx_len = np.full(B, ctx.shape[1], np.int32)
    kw = dict(K=w.K, m=w.m, N=w.N, n_max=w.n_max, n_min=w.n_min)
    ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, **kw)
    for search in SEARCHES:
        for index in (True, False):
            got, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, validate=True, index=index, search=search, **kw)
            assert_draft_equal(got, ref, f"{name}, search {search:#x}, index {index}")
    assert (ref["n_nodes"] > 0).sum() > B // 2


def test_more_contexts_than_the_gpu_holds_at_once():
    """B = 2500 contexts (more than 16 per SM): the call picks the batched path by itself, with
    and without scratch; every setting agrees with the oracle."""
    w = datagen.WORKLOADS["batched"].scaled(n_tokens=3_000_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab, W=32, sa_bytes=w.sa_bytes)
    B = 2500
    ctx = datagen.make_contexts(w, T, B=B, Lc=48)
    ctx_len = np.full(B, 48, np.int32)
    ctx_len[::7] = np.arange(len(ctx_len[::7])) % 20      # short contexts: fewer lengths to search
    kw = dict(K=w.K, m=w.m, N=w.N)
    ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, **kw)
    for search in (rest.REST_SEARCH_AUTO,) + SEARCHES:
        got, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, search=search, **kw)
        assert_draft_equal(got, ref, f"search {search:#x}")
    # without scratch for the context lists the batched path runs as one launch
    for search in (rest.REST_SEARCH_AUTO, rest.REST_SEARCH_BATCHED):
        got, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, search=search, workspace=False, **kw)
        assert_draft_equal(got, ref, f"one launch, search {search:#x}")
    assert rest.draft_workspace_bytes(B, **kw) >= 8 * B
    # fewer contexts: scratch only where sharing the gather of long candidate lists pays
    assert rest.draft_workspace_bytes(64, **kw) > 0 and rest.draft_workspace_bytes(8, **kw) == 0
    assert rest.draft_workspace_bytes(8, K=20000, m=w.m, N=w.N) > 0
    assert rest.draft_workspace_bytes(64, K=512, m=w.m, N=w.N) == 0 and rest.draft_workspace_bytes(1, K=20000) == 0
    assert len(set(ref["match_n"].tolist())) > 8          # matched lengths all over 2 ... 16
    with pytest.raises(rest.RestError):
        gpu_draft(T, sa, w.vocab, ctx[:2], ctx_len[:2], search=0x400, **kw)


def test_largest_trees_on_the_stress_recipe():
    w = datagen.WORKLOADS["stress"].scaled(n_tokens=2_000_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    B = 96
    ctx = datagen.make_contexts(w, T, B=B, Lc=64)
    ctx_len = np.full(B, 64, np.int32)
    for N in (256, 176):
        kw = dict(K=w.K, m=w.m, N=N)
        ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, **kw)
        got, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, **kw)
        assert_draft_equal(got, ref, f"N={N}")
        assert ref["n_nodes"].max() > 128


def test_other_suffix_limits_and_repeatability():
    w = datagen.WORKLOADS["tiny"].scaled(n_tokens=300_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    ctx = datagen.make_contexts(w, T, B=96, Lc=40)
    ctx_len = np.full(96, 40, np.int32)
    for n_max, n_min in ((16, 1), (8, 3), (4, 4), (1, 1)):
        kw = dict(K=300, m=7, N=48, n_max=n_max, n_min=n_min)
        ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, **kw)
        for search in SEARCHES:
            got, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, search=search, **kw)
            assert_draft_equal(got, ref, f"n_max={n_max} n_min={n_min} search {search:#x}")
            again, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, search=search, **kw)
            assert_draft_equal(again, got, "second run")
            plain, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, search=search, index=False, **kw)
            assert_draft_equal(plain, ref, f"n_max={n_max} n_min={n_min} search {search:#x}, no index")


def test_bad_context_tokens_and_corrupt_datastore():
    import paper_2311_08252_b200 as rest
    import torch
    T = np.array([1, 2, 3, 1, 2, 4, 1, 2, 3, 5], np.int32)
    sa = oracle.suffix_array(T).astype(np.int32)
    ctx = np.array([[9, 7, 1, 2], [9, 7, 1, 99], [9, 7, -1, 2]], np.int32)
    ref = oracle.draft(T, sa, 10, ctx, [4, 4, 4], m=3, N=4)
    got, _ = gpu_draft(T, sa, 10, ctx, [4, 4, 4], m=3, N=4)
    assert_draft_equal(got, ref)
    assert got["status"].tolist() == [0, 1, 1]
    # validation refuses a non-permutation, an unsorted array and an out-of-range token
    dev = torch.device("cuda:0")
    for mutate in ("dup", "swap", "range", "token"):
        s2, t2 = sa.copy(), T.copy()
        if mutate == "dup":
            s2[3] = s2[4]
        elif mutate == "swap":
            s2[[0, 5]] = s2[[5, 0]]
        elif mutate == "range":
            s2[2] = 1000
        else:
            t2[3] = 10
        with pytest.raises(rest.RestError, match="validation"):
            rest.Datastore(torch.from_numpy(t2).to(dev), torch.from_numpy(s2).to(dev), 10, validate=True)
    # without validation an out-of-range entry met while gathering is reported, never dereferenced
    Z = np.zeros(64, np.int32)
    saz = oracle.suffix_array(Z).astype(np.int32)
    bad = saz.copy()
    bad[40] = 1000
    got, _ = gpu_draft(Z, bad, 1, np.zeros((1, 20), np.int32), [20], m=3, N=4)
    assert got["status"].tolist() == [2] and got["n_nodes"].tolist() == [0]
    assert (got["tokens"] == -1).all()


def test_random_parameters_against_the_oracle():
    """Seeded sweep: random / periodic / self-repeating streams of 1 to 200 k tokens over alphabets
    of 2 to 32000 symbols, both suffix-array widths, every suffix-length window, K from 1 to the
    maximum, m and N over their whole ranges, both sampling modes, ragged context lengths."""
    rng = np.random.default_rng(20231108)
    for case in range(400):
        vocab = int(rng.choice([2, 3, 4, 8, 50, 32000]))
        n_tok = int(rng.choice([1, 2, 5, 33, 100, 1000, 5000, 40000, 200000]))
        kind = int(rng.integers(0, 3))
        if kind == 0:
            T = rng.integers(0, vocab, n_tok)
        elif kind == 1:
            T = np.tile(rng.integers(0, vocab, int(rng.integers(1, 7))), n_tok)[:n_tok]
        else:
            T = rng.integers(0, vocab, n_tok)
            if n_tok > 50:
                T[n_tok // 2:] = T[:n_tok - n_tok // 2]
        T = T.astype(np.int32)
        sa = datagen.build_suffix_array(T, vocab, W=32, sa_bytes=int(rng.choice([4, 8])))
        B, Lc = int(rng.integers(1, 50)), int(rng.integers(1, 40))
        ctx = rng.integers(0, vocab, (B, Lc)).astype(np.int32)
        for b in range(0, B, 2):
            if n_tok > Lc:
                p = int(rng.integers(0, n_tok - Lc + 1))
                ctx[b] = T[p:p + Lc]
        ctx_len = rng.integers(0, Lc + 1, B).astype(np.int32)
        n_max = int(rng.integers(1, 17))
        kw = dict(K=int(rng.choice([1, 7, 100, 5000, 32768])), m=int(rng.integers(1, 17)),
                  N=int(rng.choice([1, 16, 64, 100, 128, 256])), n_max=n_max,
                  n_min=int(rng.integers(1, n_max + 1)), sample_mode=int(rng.integers(0, 2)))
        ref = oracle.draft(T, sa, vocab, ctx, ctx_len, **kw)
        search = SEARCHES[case % 2]
        index = (case // 2) % 2 == 0
        got, _ = gpu_draft(T, sa, vocab, ctx, ctx_len, search=search, index=index, **kw)
        assert_draft_equal(got, ref, f"case {case}: vocab {vocab}, {n_tok} tokens, {kw}, search {search:#x}, "
                                     f"index {index}")


@pytest.mark.parametrize("B", [2, 40, 200])
def test_long_candidate_lists_shared_between_blocks(B):
    """Contexts whose candidate lists run into the thousands hand part of their rows to idle
    blocks through the caller's scratch (fewer contexts than SMs: blocks that only help; more:
    blocks that help once their own context is done).  Same trees as the oracle, with the scratch
    the library asks for, with a scratch full of ones from an earlier use, and without one."""
    import torch
    from gpu_util import to_dev
    rng = np.random.default_rng(100 + B)
    vocab, n_tok, Lc = 2, 60000, 24
    T = rng.integers(0, vocab, n_tok).astype(np.int32)
    sa = datagen.build_suffix_array(T, vocab, W=32, sa_bytes=4)
    ctx = rng.integers(0, vocab, (B, Lc)).astype(np.int32)
    # short contexts: their longest matching suffix is the whole context, with thousands of matches
    ctx_len = np.resize(np.array([3, 4, 2, 9, Lc, 5, 12, 3, 7, Lc], np.int32), B)
    ctx[1, :4] = T[n_tok - 6:n_tok - 2]                     # one of its rows is cut short by the end of the stream
    for K, m, N, mode in ((20000, 16, 128, 0), (8192, 10, 64, 1), (3000, 5, 256, 0)):
        kw = dict(K=K, m=m, N=N, sample_mode=mode)
        ref = oracle.draft(T, sa, vocab, ctx, ctx_len, **kw)
        hits = ref["match_range"][:, 1] - ref["match_range"][:, 0]
        assert (hits > 2048).sum() >= min(B, 2) and (hits < 512).sum() >= (1 if B > 3 else 0)
        need = rest.draft_workspace_bytes(B, **{k: v for k, v in kw.items() if k != "sample_mode"})
        assert (need > 0) == (K >= 8192 or B >= 48)      # where the library expects sharing to pay
        dirty = torch.full((max(need, 16),), 0xFF, dtype=torch.uint8, device="cuda:0")
        for workspace in (None, dirty, False):
            got, _ = gpu_draft(T, sa, vocab, ctx, ctx_len, validate=True, search=rest.REST_SEARCH_SINGLE,
                               workspace=workspace, **kw)
            assert_draft_equal(got, ref, f"B {B}, K {K}, workspace {type(workspace).__name__}")
        # the same scratch again, straight after a call that used it
        got, _ = gpu_draft(T, sa, vocab, ctx, ctx_len, search=rest.REST_SEARCH_SINGLE, workspace=dirty, **kw)
        assert_draft_equal(got, ref, f"B {B}, K {K}, scratch reused")
