"""Parity of rest_kv_commit with the oracle (bit-exact), and the closed
draft -> accept -> commit loop against the cache of plain token-by-token decoding."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_08252_b200 as rest
from gpu_util import to_dev
from test_oracle_kv_commit import enc, toy_next

pytestmark = pytest.mark.gpu


def bf16_from_bits(a):
    return to_dev(a.view(np.int16)).view(torch.bfloat16)


def bits_of(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def random_paths(rng, B, N, max_depth):
    """Strictly increasing node lists with nodes[i] >= i, lengths from 0 to max_depth."""
    nodes = np.full((B, max_depth), -1, np.int32)
    lens = rng.integers(0, max_depth + 1, size=B).astype(np.int32)
    if B > 1:
        lens[0], lens[1] = 0, max_depth
    for b in range(B):
        nodes[b, :lens[b]] = np.sort(rng.choice(N, size=lens[b], replace=False))
    return nodes, lens


@pytest.mark.parametrize("B,H,N,max_depth", [(37, 3, 64, 16), (5, 32, 128, 16), (300, 1, 64, 3),
                                             (2, 2, 16, 1)])
def test_commit_matches_oracle(B, H, N, max_depth):
    rng = np.random.default_rng(B * 1000 + H)
    D, Lmax = 128, 300
    Lcap = Lmax + N
    kv_len = rng.integers(0, Lmax + 1, size=B).astype(np.int32)
    kb = rng.integers(0, 65536, size=(B, H, Lcap, D)).astype(np.uint16)
    vb = rng.integers(0, 65536, size=(B, H, Lcap, D)).astype(np.uint16)
    nodes, lens = random_paths(rng, B, N, max_depth)
    want_k, want_v, want_len = oracle.kv_commit(kb, vb, kv_len, nodes, lens)
    k, v = bf16_from_bits(kb), bf16_from_bits(vb)
    d_len = to_dev(kv_len)
    new_len = torch.empty_like(d_len)
    rest.rest_kv_commit(k, v, d_len, to_dev(nodes), to_dev(lens), N, new_kv_len=new_len)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(k), want_k)
    assert np.array_equal(bits_of(v), want_v)
    assert np.array_equal(new_len.cpu().numpy(), want_len)


def test_strided_cache_and_aliased_length():
    # [B, Lcap, H, D] storage viewed as [B, H, Lcap, D]; new length written over the old one
    rng = np.random.default_rng(7)
    B, H, N, D, Lcap, md = 9, 4, 64, 128, 200, 16
    store = rng.integers(0, 65536, size=(2, B, Lcap, H, D)).astype(np.uint16)
    kb, vb = store[0].transpose(0, 2, 1, 3), store[1].transpose(0, 2, 1, 3)
    kv_len = rng.integers(0, Lcap - N, size=B).astype(np.int32)
    nodes, lens = random_paths(rng, B, N, md)
    want_k, want_v, want_len = oracle.kv_commit(kb, vb, kv_len, nodes, lens)
    dstore = bf16_from_bits(store)
    k, v = dstore[0].permute(0, 2, 1, 3), dstore[1].permute(0, 2, 1, 3)
    d_len = to_dev(kv_len)
    rest.rest_kv_commit(k, v, d_len, to_dev(nodes), to_dev(lens), N, new_kv_len=d_len)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(k), want_k)
    assert np.array_equal(bits_of(v), want_v)
    assert np.array_equal(d_len.cpu().numpy(), want_len)


def test_aliased_length_with_a_grid_far_beyond_one_wave():
    """Thousands of blocks with the new length written over the old one: no block of a context
    may see the updated length (which would move the wrong rows)."""
    rng = np.random.default_rng(11)
    B, H, N, D, Lcap, md = 2048, 8, 16, 128, 40, 16
    kb = rng.integers(0, 65536, size=(B, H, Lcap, D)).astype(np.uint16)
    vb = rng.integers(0, 65536, size=(B, H, Lcap, D)).astype(np.uint16)
    kv_len = rng.integers(0, Lcap - N - md, size=B).astype(np.int32)
    lens = rng.integers(1, md + 1, size=B).astype(np.int32)
    nodes = np.full((B, md), -1, np.int32)
    for b in range(B):
        nodes[b, :lens[b]] = np.sort(rng.choice(N, size=lens[b], replace=False))
    want_k, want_v, want_len = oracle.kv_commit(kb, vb, kv_len, nodes, lens)
    k, v = bf16_from_bits(kb), bf16_from_bits(vb)
    d_len = to_dev(kv_len)
    rest.rest_kv_commit(k, v, d_len, to_dev(nodes), to_dev(lens), N, new_kv_len=d_len)
    torch.cuda.synchronize()
    assert np.array_equal(d_len.cpu().numpy(), want_len)
    assert np.array_equal(bits_of(k), want_k)
    assert np.array_equal(bits_of(v), want_v)


def test_empty_batch_and_zero_depth():
    k = torch.zeros((0, 2, 64, 128), dtype=torch.bfloat16, device="cuda")
    e = torch.zeros((0,), dtype=torch.int32, device="cuda")
    rest.rest_kv_commit(k, k.clone(), e, torch.zeros((0, 4), dtype=torch.int32, device="cuda"), e, 16)
    k = torch.ones((2, 2, 64, 128), dtype=torch.bfloat16, device="cuda")
    v = k.clone()
    kv_len = to_dev(np.array([3, 9], np.int32))
    new_len = torch.zeros_like(kv_len)
    rest.rest_kv_commit(k, v, kv_len, torch.zeros((2, 0), dtype=torch.int32, device="cuda"),
                        torch.zeros_like(kv_len), 16, new_kv_len=new_len)
    torch.cuda.synchronize()
    assert new_len.tolist() == [3, 9]
    assert bool((k == 1).all())


def test_closed_loop_cache_equals_plain_decoding():
    vocab, m, N, H, D, Lcap = 11, 6, 32, 2, 128, 260
    rng = np.random.default_rng(0)
    T = [3, 5]
    for _ in range(6000):
        T.append(toy_next(T, vocab) if rng.random() < 0.85 else int(rng.integers(0, vocab)))
    T = np.array(T, np.int32)
    sa = oracle.suffix_array(T).astype(np.int32)
    ds = rest.Datastore(to_dev(T), to_dev(sa), vocab)
    seq = [1, 4, 2, 8]
    kb = np.zeros((1, H, Lcap, D), np.uint16)
    vb = np.zeros((1, H, Lcap, D), np.uint16)
    for p, x in enumerate(seq):
        kb[0, :, p], vb[0, :, p] = enc(x, p, H, D, 0), enc(x, p, H, D, 1)
    k, v = bf16_from_bits(kb), bf16_from_bits(vb)
    kv_len = to_dev(np.array([len(seq)], np.int32))
    while len(seq) < 200:
        L = len(seq)
        d = rest.rest_draft(ds, to_dev(np.array([seq], np.int32)), kv_len, m=m, N=N)
        tok, par, dep, nn = (x.cpu().numpy() for x in (d.tokens, d.parents, d.depth, d.n_nodes))
        ver = np.zeros((1, N + 1), np.int32)
        ver[0, 0] = toy_next(seq, vocab)
        rows_k = np.zeros((H, N, D), np.uint16)
        rows_v = np.zeros((H, N, D), np.uint16)
        for i in range(int(nn[0])):
            path, j = [], i
            while j >= 0:
                path.append(int(tok[0, j]))
                j = int(par[0, j])
            ver[0, i + 1] = toy_next(seq + path[::-1], vocab)
            rows_k[:, i] = enc(int(tok[0, i]), L + int(dep[0, i]) - 1, H, D, 0)
            rows_v[:, i] = enc(int(tok[0, i]), L + int(dep[0, i]) - 1, H, D, 1)
        k[0, :, L:L + N] = bf16_from_bits(rows_k)          # the model's K/V for the tree slots
        v[0, :, L:L + N] = bf16_from_bits(rows_v)
        al, an, ot = rest.rest_accept(d.tokens, d.parents, d.n_nodes, to_dev(ver), m)
        rest.rest_kv_commit(k, v, kv_len, an, al, N, new_kv_len=kv_len)
        a = int(al[0])
        seq += ot[0, :a + 1].cpu().tolist()
        p = len(seq) - 1                                   # the stop token's row: next forward pass
        k[0, :, p] = bf16_from_bits(enc(seq[p], p, H, D, 0))
        v[0, :, p] = bf16_from_bits(enc(seq[p], p, H, D, 1))
        assert int(kv_len[0]) == p
        kv_len += 1
    plain = [1, 4, 2, 8]
    while len(plain) < len(seq):
        plain.append(toy_next(plain, vocab))
    assert seq == plain
    got_k, got_v = bits_of(k), bits_of(v)
    for p, x in enumerate(plain):
        assert np.array_equal(got_k[0, :, p], enc(x, p, H, D, 0)), p
        assert np.array_equal(got_v[0, :, p], enc(x, p, H, D, 1)), p
    ds.close()
