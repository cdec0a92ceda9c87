"""Parity of rest_accept with the oracle, and the closed draft -> accept loop against plain
token-by-token decoding."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2311_08252_b200 as rest
from gpu_util import gpu_draft, to_dev

pytestmark = pytest.mark.gpu


def gpu_accept(tokens, parents, n_nodes, ver, max_depth):
    out = rest.rest_accept(to_dev(tokens), to_dev(parents), to_dev(n_nodes), to_dev(ver), max_depth)
    torch.cuda.synchronize()
    return [o.cpu().numpy() for o in out]


@pytest.mark.parametrize("name,N", [("tiny", 64), ("stress", 128), ("stress", 256)])
def test_accept_matches_oracle_on_drafted_trees(name, N):
    w = datagen.WORKLOADS[name].scaled(n_tokens=500_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    B = 333
    ctx = datagen.make_contexts(w, T, B=B, Lc=32)
    ref = oracle.draft(T, sa, w.vocab, ctx, np.full(B, 32), K=w.K, m=w.m, N=N)
    for seed in (1, 2):
        ver = datagen.make_verifier_tokens(seed, ref["tokens"], ref["parents"], ref["n_nodes"], w.vocab)
        for max_depth in (w.m, 3, 1, 0):
            want = oracle.accept(ref["tokens"], ref["parents"], ref["n_nodes"], ver, max_depth)
            got = gpu_accept(ref["tokens"], ref["parents"], ref["n_nodes"], ver, max_depth)
            for g, r in zip(got, want):
                assert np.array_equal(g, r)
        assert want[0].max() >= 0
    assert oracle.accept(ref["tokens"], ref["parents"], ref["n_nodes"], ver, w.m)[0].max() >= 2


def test_edge_cases():
    tok = np.full((2, 4), -1, np.int32)
    par = np.full((2, 4), -1, np.int32)
    tok[1] = [5, 6, 7, 8]
    par[1] = [-1, 0, 1, 2]
    ver = np.array([[-1, 1, 2, 3, 4], [5, 6, 7, 8, 9]], np.int32)
    nn = np.array([0, 4], np.int32)
    for md in (4, 2):
        want = oracle.accept(tok, par, nn, ver, md)
        got = gpu_accept(tok, par, nn, ver, md)
        for g, r in zip(got, want):
            assert np.array_equal(g, r)
    assert got[0].tolist() == [0, 2]


def test_closed_loop_is_lossless():
    vocab, m, N = 11, 6, 32

    def toy_next(prefix):
        return (int(prefix[-2]) * 7 + int(prefix[-1]) * 3 + 1) % vocab

    rng = np.random.default_rng(0)
    T = [3, 5]
    for _ in range(6000):
        T.append(toy_next(T) if rng.random() < 0.85 else int(rng.integers(0, vocab)))
    T = np.array(T, np.int32)
    sa = oracle.suffix_array(T).astype(np.int32)
    ds = rest.Datastore(to_dev(T), to_dev(sa), vocab)
    plain = [1, 4, 2, 8]
    while len(plain) < 150:
        plain.append(toy_next(plain))
    seq, steps, acc = [1, 4, 2, 8], 0, 0
    while len(seq) < 150:
        ctx = to_dev(np.array([seq], np.int32))
        d = rest.rest_draft(ds, ctx, to_dev(np.array([len(seq)], np.int32)), m=m, N=N)
        tok, par, nn = d.tokens.cpu().numpy(), d.parents.cpu().numpy(), d.n_nodes.cpu().numpy()
        ver = np.zeros((1, N + 1), np.int32)
        ver[0, 0] = toy_next(seq)
        for i in range(int(nn[0])):
            path, j = [], i
            while j >= 0:
                path.append(int(tok[0, j]))
                j = int(par[0, j])
            ver[0, i + 1] = toy_next(seq + path[::-1])
        al, an, ot = rest.rest_accept(d.tokens, d.parents, d.n_nodes, to_dev(ver), m)
        seq += ot[0, :int(al[0]) + 1].cpu().tolist()
        acc += int(al[0])
        steps += 1
    assert seq[:150] == plain[:150]
    assert acc / steps > 0.5
