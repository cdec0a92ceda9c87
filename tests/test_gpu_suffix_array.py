"""rest_suffix_array_build against the oracle's comparison sort (where the 32-token order is the
full order), against the order's definition checked entry by entry, and through rest_draft."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2311_08252_b200 as rest
from gpu_util import assert_draft_equal, gpu_draft, to_dev

pytestmark = pytest.mark.gpu


def gpu_sa(T, sa_bytes=4):
    sa = rest.rest_suffix_array_build(to_dev(np.asarray(T, np.int32)), sa_bytes=sa_bytes)
    torch.cuda.synchronize()
    return sa.cpu().numpy()


def bounded_order_reference(T, W=32):
    """The order's definition, by brute force: sort positions by (first W tokens, padded with -1
    past the end, then position)."""
    n = len(T)
    keys = [(tuple(int(x) for x in T[p:p + W]) , p) for p in range(n)]
    # a suffix that ends early is smaller: tuple comparison already puts a proper prefix first
    return np.array([p for _, p in sorted(keys)], np.int64)


@pytest.mark.parametrize("seed,vocab,n", [(1, 32000, 5000), (2, 50, 20000), (3, 2**31 - 2, 3000)])
def test_equals_the_full_suffix_order_when_no_two_suffixes_share_32_tokens(seed, vocab, n):
    rng = np.random.default_rng(seed)
    T = rng.integers(0, vocab, n).astype(np.int32)
    T[-1] = vocab - 1
    want = oracle.suffix_array(T)
    assert np.array_equal(gpu_sa(T), want)
    assert np.array_equal(gpu_sa(T, 8), want.astype(np.int64))


@pytest.mark.parametrize("name", ["binary", "constant", "period3", "two_runs", "single", "pair"])
def test_repetitive_streams_follow_the_bounded_order(name):
    rng = np.random.default_rng(5)
    T = {"binary": rng.integers(0, 2, 3000), "constant": np.full(500, 7),
         "period3": np.tile([4, 1, 9], 400), "two_runs": np.r_[np.full(300, 3), np.full(300, 2)],
         "single": np.array([11]), "pair": np.array([5, 5])}[name].astype(np.int32)
    got = gpu_sa(T)
    assert np.array_equal(got, bounded_order_reference(T))
    assert got.dtype == np.int32


@pytest.mark.parametrize("name", ["single_stream", "stress", "large"])
def test_workload_recipes_and_drafts_on_the_device_built_array(name):
    w = datagen.WORKLOADS[name].scaled(n_tokens=1_500_000)
    T = datagen.make_tokens(w)
    sa = gpu_sa(T, w.sa_bytes)
    assert datagen.verify_suffix_array(T, sa, W=32) == 0          # permutation, ordered, ties by position
    B = 64
    ctx = datagen.make_contexts(w, T, B=B, Lc=64)
    ctx_len = np.full(B, 64, np.int32)
    kw = dict(K=w.K, m=w.m, N=w.N)
    ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, **kw)
    got, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, validate=True, **kw)
    assert_draft_equal(got, ref, name)
    assert (ref["n_nodes"] > 0).mean() > 0.5


def largest_first_token_bucket(T):
    return int(np.unique(T, return_counts=True)[1].max())


@pytest.mark.parametrize("case", ["single_stream", "large", "vocab50", "tokens_up_to_2^31", "constant", "binary"])
def test_bucket_method_gives_the_same_array_as_prefix_doubling(case):
    """The builder's second method (groups of first-token buckets sorted on their packed
    32-token keys; what streams beyond 2^31 - 1 tokens get) must give the very same array."""
    rng = np.random.default_rng(11)
    sa_bytes = 4
    if case in ("single_stream", "large"):
        w = datagen.WORKLOADS[case].scaled(n_tokens=1_200_000)
        T, sa_bytes = datagen.make_tokens(w), w.sa_bytes
    elif case == "vocab50":
        T = rng.integers(0, 50, 300_000).astype(np.int32)
    elif case == "tokens_up_to_2^31":
        T = rng.integers(0, 2**31 - 2, 40_000).astype(np.int32)      # 31-bit tokens: two per key word
        T[::7] = T[3]                                                 # and some repetition
    elif case == "constant":
        T = np.full(5000, 3, np.int32)
    else:
        T = rng.integers(0, 2, 50_000).astype(np.int32)
    d_T = to_dev(T)
    want = rest.rest_suffix_array_build(d_T, sa_bytes)
    biggest = largest_first_token_bucket(T)
    got = rest.rest_suffix_array_build(d_T, sa_bytes, max_group=max(biggest, 1024))
    assert got.dtype == want.dtype and torch.equal(got, want)
    if case in ("single_stream", "vocab50"):
        assert len(T) > 4 * max(biggest, 1024)        # several groups were sorted
    if case == "vocab50":
        # groups too small for the most frequent first token are refused
        with pytest.raises(rest.RestError, match="unsupported"):
            rest.rest_suffix_array_build(d_T, sa_bytes, max_group=1024)


@pytest.mark.parametrize("name", ["binary", "constant", "period3", "long_repeat", "recipe"])
def test_full_order_equals_the_oracle_suffix_array(name):
    """Streams whose suffixes share far more than 32 tokens: the full-order build must give the
    true suffix array (the oracle's comparison sort of whole suffixes)."""
    rng = np.random.default_rng(6)
    if name == "recipe":
        T = datagen.make_tokens(datagen.WORKLOADS["single_stream"].scaled(n_tokens=60_000))
    else:
        block = rng.integers(0, 9, 700)
        T = {"binary": rng.integers(0, 2, 4000), "constant": np.full(900, 7),
             "period3": np.tile([4, 1, 9], 500), "long_repeat": np.r_[block, block, [8], block]}[name]
    T = T.astype(np.int32)
    want = oracle.suffix_array(T)
    for sa_bytes in (4, 8):
        got = rest.rest_suffix_array_build(to_dev(T), sa_bytes, full=True).cpu().numpy()
        assert np.array_equal(got, want)
    if name in ("constant", "period3", "long_repeat"):
        assert not np.array_equal(gpu_sa(T), want)      # the 32-token order differs on these streams


@pytest.mark.parametrize("kind", ["recipe", "binary", "constant", "period3"])
def test_append_equals_a_build_from_scratch(kind):
    """Tokens appended to a stream: the merged array must be the one a build of the whole stream
    gives, for tails shorter and longer than the 32-token window and for both entry widths."""
    rng = np.random.default_rng(8)
    if kind == "recipe":
        T = datagen.make_tokens(datagen.WORKLOADS["single_stream"].scaled(n_tokens=400_000))
    elif kind == "binary":
        T = rng.integers(0, 2, 30_000)
    elif kind == "constant":
        T = np.full(3000, 5)
    else:
        T = np.tile([4, 1, 9], 1000)
    d_T = to_dev(T.astype(np.int32))
    n = len(T)
    for sa_bytes in (4, 8):
        want = rest.rest_suffix_array_build(d_T, sa_bytes)
        for n_old in (1, 7, 31, 32, 33, n // 3, n - 40, n - 1):
            old = rest.rest_suffix_array_build(d_T[:n_old].contiguous(), sa_bytes)
            got = rest.rest_suffix_array_append(d_T, old)
            assert got.dtype == want.dtype and torch.equal(got, want), (kind, sa_bytes, n_old)
    # in steps: three appends in a row
    sa = rest.rest_suffix_array_build(d_T[:1000].contiguous(), 4)
    for upto in (1010, n // 2, n):
        sa = rest.rest_suffix_array_append(d_T[:upto].contiguous(), sa)
    assert torch.equal(sa, rest.rest_suffix_array_build(d_T, 4))


def test_argument_checks():
    L = rest.lib()
    assert L.rest_suffix_array_workspace_bytes(0) == 0
    assert L.rest_suffix_array_workspace_bytes((1 << 40) + 1) == 0
    # beyond 2^31 - 1 tokens the recommended scratch is that of groups of 2^30 positions
    assert 32 << 30 < L.rest_suffix_array_workspace_bytes(1 << 32) < 33 << 30
    assert L.rest_suffix_array_build(256, 10, 5, 256, 256, 1 << 30, None) == 1
    assert L.rest_suffix_array_build(256, 10, 4, 256, 256, 16, None) == 3
    assert L.rest_suffix_array_build(256, 1 << 31, 4, 256, 256, 1 << 30, None) == 1     # needs 64-bit entries
    assert L.rest_suffix_array_build(256, (1 << 40) + 1, 8, 256, 256, 1 << 30, None) == 2
