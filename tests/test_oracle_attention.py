"""Pins for the oracle's tree attention (Sec. 3.2 "Draft verification").

The oracle's fp64 loop is compared with things it does not compute itself: torch's own
causal scaled-dot-product attention over the sequence "prefix followed by the root-to-node
path", chain and star trees that reduce to textbook cases, and closed forms.
"""
import math

import numpy as np
import torch
import torch.nn.functional as F

import datagen
import oracle


def bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def setup(seed, B, H, N, D, L, Lcap=None, n_nodes=None, max_depth=6):
    Lcap = L + N if Lcap is None else Lcap
    q, k, v = datagen.make_qkv(seed, B, H, N, D, Lcap)
    par, dep, mask = datagen.make_random_tree(seed + 1, N, max_depth, n_nodes)
    mask = np.broadcast_to(mask, (B,) + mask.shape).copy()
    return q, k, v, par, dep, mask


def path_of(par, i):
    p = []
    while i >= 0:
        p.append(i)
        i = int(par[i])
    return p[::-1]


def test_each_node_equals_causal_attention_over_prefix_plus_path():
    B, H, N, D, L = 2, 3, 40, 32, 37
    q, k, v, par, dep, mask = setup(3, B, H, N, D, L, Lcap=L + N + 5, n_nodes=33)
    kv_len = np.array([L, L - 9], np.int32)
    scale = 1.0 / math.sqrt(D)
    out, lse = oracle.tree_attention(bits(q), bits(k), bits(v), kv_len, mask, scale, want_lse=True)
    qd, kd, vd = q.double(), k.double(), v.double()
    for b in range(B):
        Lb = int(kv_len[b])
        for i in range(N):
            path = path_of(par, i) if i < 33 else [i]
            rows = list(range(Lb)) + [Lb + j for j in path]
            ks = kd[b][:, rows]                                   # [H, S, D]
            vs = vd[b][:, rows]
            qs = torch.zeros(H, len(rows), D, dtype=torch.float64)
            qs[:, Lb:] = qd[b, path].transpose(0, 1)              # queries of the path nodes
            ref = F.scaled_dot_product_attention(qs[None], ks[None], vs[None], is_causal=True,
                                                 scale=scale)[0]
            got = torch.from_numpy(out[b, i])                     # [H, D]
            assert torch.allclose(got, ref[:, -1], rtol=1e-10, atol=1e-12), (b, i)
            s = (qd[b, i][:, None, :] * ks).sum(-1) * scale       # [H, S]
            assert torch.allclose(torch.from_numpy(lse[b, :, i]), torch.logsumexp(s, -1),
                                  rtol=1e-10, atol=1e-12)


def test_chain_tree_is_plain_causal_attention_of_new_tokens():
    B, H, N, D, L = 1, 2, 16, 16, 21
    q, k, v = datagen.make_qkv(5, B, H, N, D, L + N)
    mask = np.zeros((B, N, 1), np.uint32)
    for i in range(N):
        mask[0, i, 0] = (1 << (i + 1)) - 1
    out = oracle.tree_attention(bits(q), bits(k), bits(v), [L], mask, 0.25)
    qs = torch.zeros(B, H, L + N, D, dtype=torch.float64)
    qs[:, :, L:] = q.double().permute(0, 2, 1, 3)
    ref = F.scaled_dot_product_attention(qs, k.double(), v.double(), is_causal=True, scale=0.25)
    got = torch.from_numpy(out).permute(0, 2, 1, 3)
    assert torch.allclose(got, ref[:, :, L:], rtol=1e-10, atol=1e-12)


def test_star_tree_is_independent_single_token_decodes():
    B, H, N, D, L = 1, 2, 8, 16, 30
    q, k, v = datagen.make_qkv(6, B, H, N, D, L + N)
    mask = np.zeros((B, N, 1), np.uint32)
    for i in range(N):
        mask[0, i, 0] = 1 << i
    out = oracle.tree_attention(bits(q), bits(k), bits(v), [L], mask, 0.3)
    for i in range(N):
        rows = list(range(L)) + [L + i]
        kk, vv = k.double()[:, :, rows], v.double()[:, :, rows]
        qq = q.double()[:, i][:, :, None, :]
        ref = F.scaled_dot_product_attention(qq, kk, vv, scale=0.3)[:, :, 0]
        assert torch.allclose(torch.from_numpy(out[:, i]), ref, rtol=1e-10, atol=1e-12)


def test_closed_forms_and_prefix_permutation():
    B, H, N, D, L = 1, 2, 24, 16, 19
    q, k, v, par, dep, mask = setup(8, B, H, N, D, L)
    # zero keys -> uniform weights -> mean of the allowed value rows; lse = log(#keys)
    out, lse = oracle.tree_attention(bits(q), bits(torch.zeros_like(k)), bits(v), [L], mask, 1.0,
                                     want_lse=True)
    for i in range(N):
        rows = list(range(L)) + [L + j for j in path_of(par, i)]
        ref = v.double()[0][:, rows].mean(1)
        assert torch.allclose(torch.from_numpy(out[0, i]), ref, rtol=1e-12, atol=1e-13)
        assert np.allclose(lse[0, :, i], math.log(len(rows)))
    # constant values -> that constant
    vc = torch.full_like(v, 1.5)
    out = oracle.tree_attention(bits(q), bits(k), bits(vc), [L], mask, 0.2)
    assert np.allclose(out, 1.5, rtol=1e-12)
    # permuting prefix rows of K and V together changes nothing
    base = oracle.tree_attention(bits(q), bits(k), bits(v), [L], mask, 0.2)
    perm = torch.cat([torch.randperm(L, generator=torch.Generator().manual_seed(1)),
                      torch.arange(L, L + N)])
    out = oracle.tree_attention(bits(q), bits(k[:, :, perm]), bits(v[:, :, perm]), [L], mask, 0.2)
    assert np.allclose(out, base, rtol=1e-11, atol=1e-13)


def test_grouped_kv_heads_and_strides():
    B, H, Hkv, N, D, L = 2, 4, 2, 8, 16, 12
    q, k, v = datagen.make_qkv(9, B, H, N, D, L + N, H_kv=Hkv)
    _, _, mask = datagen.make_random_tree(4, N, 4)
    mask = np.broadcast_to(mask, (B,) + mask.shape).copy()
    out = oracle.tree_attention(bits(q), bits(k), bits(v), [L, L], mask, 0.25, H_kv=Hkv)
    k2 = k.repeat_interleave(2, dim=1)
    v2 = v.repeat_interleave(2, dim=1)
    ref = oracle.tree_attention(bits(q), bits(k2), bits(v2), [L, L], mask, 0.25)
    assert np.array_equal(out, ref)
    # a strided (non-dense) KV view gives the same numbers
    big = torch.zeros(B, Hkv, L + N + 7, D, dtype=torch.bfloat16)
    big[:, :, :L + N] = k
    kb = big.view(torch.int16).numpy().view(np.uint16)[:, :, :L + N]
    big2 = torch.zeros(B, Hkv, L + N + 7, D, dtype=torch.bfloat16)
    big2[:, :, :L + N] = v
    vb = big2.view(torch.int16).numpy().view(np.uint16)[:, :, :L + N]
    out2 = oracle.tree_attention(bits(q), kb, vb, [L, L], mask, 0.25, H_kv=Hkv)
    assert np.array_equal(out, out2)
