"""Input generators: determinism, value ranges, and the host suffix-array builder checked
against the oracle's comparison sort."""
import numpy as np

import datagen
import oracle


def test_tokens_are_deterministic_and_in_range():
    w = datagen.WORKLOADS["single_stream"].scaled(n_tokens=300_000)
    a = datagen.make_tokens(w)
    b = datagen.make_tokens(w)
    assert np.array_equal(a, b)
    assert a.min() >= 0 and a.max() < w.vocab
    c = datagen.make_tokens(datagen.WORKLOADS["large"].scaled(n_tokens=300_000))
    assert c.min() >= 0 and c.max() < w.vocab and not np.array_equal(a, c)


def test_builder_equals_comparison_sort_and_verifier_rejects_errors():
    for name, n in (("tiny", 50_000), ("stress", 30_000), ("single_stream", 70_000)):
        w = datagen.WORKLOADS[name].scaled(n_tokens=n)
        T = datagen.make_tokens(w)
        full = datagen.build_suffix_array(T, w.vocab, W=0)
        assert np.array_equal(full, oracle.suffix_array(T))
        sa = datagen.build_suffix_array(T, w.vocab, W=32)
        assert datagen.verify_suffix_array(T, sa, 32) == 0
        assert datagen.verify_suffix_array(T, full, 0) == 0
        sa64 = datagen.build_suffix_array(T, w.vocab, W=32, sa_bytes=8)
        assert sa64.dtype == np.int64 and np.array_equal(sa64, sa)
        bad = sa.copy()
        bad[[10, 11]] = bad[[11, 10]]
        assert datagen.verify_suffix_array(T, bad, 32) in (4, 5)
        bad = sa.copy()
        bad[5] = bad[6]
        assert datagen.verify_suffix_array(T, bad, 32) == 3


def test_contexts_mix_gives_a_spread_of_match_lengths():
    w = datagen.WORKLOADS["tiny"].scaled(n_tokens=400_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    ctx = datagen.make_contexts(w, T, B=200, Lc=64)
    assert np.array_equal(ctx, datagen.make_contexts(w, T, B=200, Lc=64))
    ns = np.array([oracle.retrieve(T, sa, c)[0] for c in ctx])
    assert (ns == 0).sum() >= 1 and (ns == 16).sum() >= 1
    assert ((ns >= 2) & (ns <= 9)).sum() > 100


def test_random_tree_is_breadth_first():
    for seed in range(5):
        par, dep, mask = datagen.make_random_tree(seed, 64, 10, n_nodes=50)
        for i in range(50):
            assert par[i] < i
            if par[i] >= 0:
                assert dep[i] == dep[par[i]] + 1
        assert (np.diff(dep[:50]) >= 0).all()
        assert (dep[50:] == 0).all()
