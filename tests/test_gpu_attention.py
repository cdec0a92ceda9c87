"""Parity of rest_tree_attention with the fp64 oracle.

Tolerance (from the arithmetic: bf16 inputs, bf16-rounded probabilities, fp32 accumulation,
bf16 output, values ~N(0,1)): every element within 1e-2 absolute of the fp64 result, and every
(context, node, head) output row within 2e-2 relative L2 error."""
import math

import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2311_08252_b200 as rest
from gpu_util import attention_errors, bits, to_dev

pytestmark = pytest.mark.gpu

MAX_ABS = 1e-2
MAX_REL = 2e-2


def abs_bound(ref):
    """The flat 1e-2 wherever the reference is an ordinary value (|ref| <= 2: bf16 spacing is at
    most 2^-7 there, so rounding the output costs at most 3.9e-3); from 2 on, where the spacing
    is 2^-6 and more and rounding alone costs up to 2^-8 |x|, 1e-2 + 2^-8 |ref|."""
    a = np.abs(ref)
    return np.where(a <= 2.0, MAX_ABS, MAX_ABS + a / 256.0)


def run_case(seed, B, H, N, L, Lcap=None, H_kv=None, kv_len=None, n_nodes=None, max_depth=8,
             want_lse=True, scale=None):
    D = 128
    Lcap = (L + N) if Lcap is None else Lcap
    q, k, v = datagen.make_qkv(seed, B, H, N, D, Lcap, H_kv=H_kv)
    masks = []
    for b in range(B):
        _, _, mk = datagen.make_random_tree(seed * 100 + b, N, max_depth, n_nodes)
        masks.append(mk)
    mask = np.stack(masks)
    kv_len = np.full(B, L, np.int32) if kv_len is None else np.asarray(kv_len, np.int32)
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    ref, ref_lse = oracle.tree_attention(bits(q), bits(k), bits(v), kv_len, mask, scale,
                                         H_kv=H_kv, want_lse=True)
    lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda:0") if want_lse else None
    out = rest.rest_tree_attention(q.cuda(), k.cuda(), v.cuda(), to_dev(kv_len), to_dev(mask),
                                   scale, lse=lse)
    torch.cuda.synchronize()
    max_abs, max_rel = attention_errors(out, ref)
    assert max_abs <= MAX_ABS and max_rel <= MAX_REL, (max_abs, max_rel)
    if want_lse:
        assert np.abs(lse.cpu().numpy().astype(np.float64) - ref_lse).max() <= 2e-3
    return out, ref


@pytest.mark.parametrize("B,H,N,L", [
    (1, 32, 64, 256),        # tiny workload shape: split keys
    (2, 4, 64, 37),          # prefix shorter than one tile, tree keys straddle tiles
    (1, 2, 16, 0),           # no prefix at all
    (3, 5, 128, 1000),       # N = 128, ragged tail
    (2, 3, 48, 200),         # N not a multiple of 32
    (1, 1, 64, 4096 + 17),   # many splits for one head
    (20, 16, 64, 513),       # enough units for a single split: direct output path
    (7, 14, 64, 700),        # 3 splits: a cluster of three
    (1, 59, 64, 700),        # 5 splits
    (7, 7, 64, 1000),        # 6 splits
    (6, 7, 48, 900),         # 7 splits, N = 48: owners get uneven row counts
    (40, 8, 128, 700),       # N = 128, one split per (context, head): direct output path
    (2, 3, 96, 300),         # 64 < N < 128: rows past N are padding of the 128-row block
    (1, 2, 80, 64),          # N = 80, prefix of exactly one tile
    (1, 1, 128, 0),          # N = 128, no prefix: only tree keys
    (1, 1, 128, 8192 + 5),   # N = 128, one head cut into many splits
    (1, 3, 112, 130),
    (2, 3, 256, 500),        # N = 256: two 128-row blocks per head
    (1, 2, 192, 100),        # second row block half empty
    (1, 1, 144, 0),          # N = 144, no prefix
    (1, 1, 256, 4096 + 9),   # N = 256, many splits
    (24, 8, 256, 700),       # N = 256, one split: direct output path
    (2, 3, 1, 100),          # any tree size the draft can write: a single draft token
    (1, 32, 7, 300),         # N = 7, key splits merged in a cluster (owners without rows)
    (3, 4, 40, 513),         # N = 40
    (50, 8, 61, 200),        # N = 61, one split
    (2, 2, 100, 700),        # N = 100: 128-row block, 28 rows of padding
    (1, 2, 129, 300),        # N = 129: the second row block holds one row
    (30, 12, 200, 150),      # N = 200, one split
    (1, 1, 255, 2048 + 3),   # N = 255, many splits
])
def test_matches_fp64_oracle(B, H, N, L):
    run_case(7, B, H, N, L)


def test_ragged_batch_grouped_heads_padding_nodes_and_strides():
    # different prefix lengths per context (some splits end up empty), grouped KV heads,
    # trees with unused slots, KV buffer longer than needed
    run_case(11, 4, 8, 64, 700, Lcap=900, H_kv=2, kv_len=[700, 1, 333, 64], n_nodes=41)
    run_case(12, 2, 6, 32, 90, H_kv=3, kv_len=[90, 31], n_nodes=1, scale=0.2)


def test_grouped_heads_large_batch_two_query_heads_per_block():
    # N = 64, heads in groups, batch large enough that no key split is needed: pairs of query
    # heads of a group are computed by one block
    rng = np.random.default_rng(3)
    run_case(16, 40, 16, 64, 513, H_kv=4, kv_len=rng.integers(0, 514, 40), n_nodes=50)
    run_case(17, 20, 32, 64, 300, H_kv=16, kv_len=rng.integers(1, 301, 20))
    run_case(18, 75, 8, 64, 130, H_kv=1, Lcap=300)


def test_partial_last_wave_goes_into_a_second_launch_with_key_splits():
    # slightly more (context, head) units than fit at once, caches of 16+ tiles: the units of
    # the partial last wave run as a second launch whose key range is cut over a cluster
    rng = np.random.default_rng(4)
    run_case(19, 10, 32, 64, 1100, kv_len=rng.integers(0, 1101, 10))
    run_case(20, 5, 62, 128, 1300, kv_len=rng.integers(900, 1301, 5), max_depth=16)
    run_case(21, 38, 8, 32, 1024)


def test_wide_rows_ragged_batch_and_grouped_heads():
    # N > 64 with contexts far shorter than the longest one: some key splits get no tile at all
    run_case(13, 4, 8, 128, 900, Lcap=1100, H_kv=2, kv_len=[900, 1, 333, 64], n_nodes=77, max_depth=16)
    run_case(14, 3, 6, 96, 200, H_kv=3, kv_len=[200, 31, 0], n_nodes=1, scale=0.2)
    run_case(15, 3, 4, 256, 600, Lcap=900, H_kv=2, kv_len=[600, 2, 129], n_nodes=201, max_depth=16)


@pytest.mark.parametrize("B,H,N,L", [(1, 2, 128, 1500), (30, 10, 128, 1500), (2, 2, 64, 1500)])
def test_scores_whose_maximum_keeps_growing(B, H, N, L):
    # Keys grow with their position, so the running maximum of every row rises again and again,
    # tile after tile, by far more than any lazy-rescale threshold; every fifth tile jumps.
    # Rows become so peaked that an output is nearly a single V row, with magnitudes up to 4-5,
    # where rounding the output to bf16 alone costs up to 2^-8 |x| (0.0156 at 4): the absolute
    # bound is therefore 1e-2 + 2^-8 |reference| for |reference| > 2 (the flat 1e-2 below that);
    # the row-wise bound is unchanged.
    D = 128
    q, k, v = datagen.make_qkv(31, B, H, N, D, L + N)
    pos = torch.arange(L + N, dtype=torch.float32)
    factor = 1.0 + 7.0 * pos / (L + N)
    factor[(pos.long() // 64) % 5 == 3] *= 2.5
    k = (k.float() * factor[None, None, :, None]).to(torch.bfloat16)
    masks = np.stack([datagen.make_random_tree(3100 + b, N, 12)[2] for b in range(B)])
    kv_len = np.full(B, L, np.int32)
    scale = 1.0 / math.sqrt(D)
    ref = oracle.tree_attention(bits(q), bits(k), bits(v), kv_len, masks, scale)
    out = rest.rest_tree_attention(q.cuda(), k.cuda(), v.cuda(), to_dev(kv_len), to_dev(masks), scale)
    torch.cuda.synchronize()
    err = np.abs(out.float().cpu().numpy().astype(np.float64) - ref)
    assert (err <= abs_bound(ref)).all(), float((err - abs_bound(ref)).max())
    _, max_rel = attention_errors(out, ref)
    assert max_rel <= MAX_REL, max_rel


def test_invariants_on_the_gpu_output():
    B, H, N, L, D = 1, 2, 64, 130, 128
    q, k, v = datagen.make_qkv(3, B, H, N, D, L + N)
    par, dep, mask = datagen.make_random_tree(5, N, 8)
    mask = mask[None].copy()
    kv_len = to_dev(np.array([L], np.int32))
    # constant V -> exactly that constant
    vc = torch.full_like(v, 1.5)
    out = rest.rest_tree_attention(q.cuda(), k.cuda(), vc.cuda(), kv_len, to_dev(mask), 0.1)
    assert torch.allclose(out.float().cpu(), torch.full((B, N, H, D), 1.5), atol=8e-3)
    # zero K -> mean of the allowed V rows
    out = rest.rest_tree_attention(q.cuda(), torch.zeros_like(k).cuda(), v.cuda(), kv_len,
                                   to_dev(mask), 0.1).float().cpu()
    for i in (0, 17, 63):
        rows, j = list(range(L)), i
        while j >= 0:
            rows.append(L + j)
            j = int(par[j])
        want = v[0][:, rows].float().mean(1)
        assert torch.allclose(out[0, i], want, atol=1e-2)
    # permuting the prefix rows of K and V together changes (almost) nothing
    base = rest.rest_tree_attention(q.cuda(), k.cuda(), v.cuda(), kv_len, to_dev(mask), 0.1).float().cpu()
    perm = torch.cat([torch.randperm(L, generator=torch.Generator().manual_seed(1)),
                      torch.arange(L, L + N)])
    out = rest.rest_tree_attention(q.cuda(), k[:, :, perm].contiguous().cuda(),
                                   v[:, :, perm].contiguous().cuda(), kv_len, to_dev(mask), 0.1).float().cpu()
    assert (out - base).abs().max() <= 1e-2


def test_attention_on_drafted_masks_full_head_count():
    # masks produced by rest_draft, 32 heads x 128, KV prefix 2048: the single-stream shape
    from gpu_util import gpu_draft
    w = datagen.WORKLOADS["single_stream"].scaled(n_tokens=1_000_000)
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    ctx = datagen.make_contexts(w, T, B=2, Lc=256)
    ref_d = oracle.draft(T, sa, w.vocab, ctx, [256, 256], K=w.K, m=w.m, N=w.N)
    got_d, out_d = gpu_draft(T, sa, w.vocab, ctx, [256, 256], K=w.K, m=w.m, N=w.N)
    assert np.array_equal(got_d["mask"], ref_d["mask"])
    L = 2048
    q, k, v = datagen.make_qkv(21, 2, 32, w.N, 128, L + w.N)
    scale = 1.0 / math.sqrt(128)
    out = rest.rest_tree_attention(q.cuda(), k.cuda(), v.cuda(), to_dev(np.array([L, L], np.int32)),
                                   out_d.mask, scale)
    torch.cuda.synchronize()
    # the oracle on a sample of heads (all nodes): fp64 over 2 x 4 heads
    hs = [0, 13, 31, 7]
    ref = oracle.tree_attention(bits(q[:, :, hs]), bits(k[:, hs]), bits(v[:, hs]), [L, L],
                                ref_d["mask"], scale)
    max_abs, max_rel = attention_errors(out[:, :, hs], ref)
    assert max_abs <= MAX_ABS and max_rel <= MAX_REL, (max_abs, max_rel)


def test_random_shapes_against_the_oracle():
    """Seeded sweep over batch sizes (also just around whole waves of blocks), head groupings,
    tree sizes, ragged prefixes and scales.  Outputs may reach magnitudes where rounding to bf16
    alone costs 2^-8 |x|, so the absolute bound is 1e-2 + 2^-8 |reference| where |reference| > 2
    and the flat 1e-2 everywhere else; the log-sum-exp bound
    is 5e-3 (with more than 64 draft rows the denominator sums bf16-rounded probabilities)."""
    rng = np.random.default_rng(20231108)
    done = 0
    while done < 60:
        N = int(rng.choice([16, 32, 48, 64, 64, 64, 80, 128, 128, 192, 256, 5, 37, 99, 150, 233]))
        H_kv = int(rng.integers(1, 9))
        H = H_kv * int(rng.choice([1, 1, 1, 2, 4]))
        mode = int(rng.integers(0, 3))
        if mode == 0:
            B = int(rng.integers(1, 4))
        elif mode == 1:
            B = max(1, int(rng.choice([148, 296, 300, 320, 600])) // H + int(rng.integers(0, 2)))
        else:
            B = int(rng.integers(1, 40))
        L = int(rng.choice([0, 1, 63, 64, 65, 200, 513, 1024, 1100, 2048]))
        if B * H * (L + N) * N > 2e8:
            continue
        kv_len = rng.integers(0, L + 1, B).astype(np.int32)
        if rng.random() < 0.5:
            kv_len[:] = L
        Lcap = L + N + int(rng.choice([0, 0, 7, 64]))
        q, k, v = datagen.make_qkv(int(rng.integers(1, 1 << 30)), B, H, N, 128, Lcap, H_kv=H_kv)
        masks = np.stack([datagen.make_random_tree(int(rng.integers(1, 1 << 30)), N, int(rng.integers(1, 17)),
                                                   int(rng.integers(1, N + 1)))[2] for _ in range(B)])
        scale = float(rng.choice([1 / math.sqrt(128), 0.05, 0.2]))
        ref, ref_lse = oracle.tree_attention(bits(q), bits(k), bits(v), kv_len, masks, scale, H_kv=H_kv,
                                             want_lse=True)
        lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda:0")
        out = rest.rest_tree_attention(q.cuda(), k.cuda(), v.cuda(), to_dev(kv_len), to_dev(masks), scale,
                                       lse=lse)
        torch.cuda.synchronize()
        what = dict(B=B, H=H, H_kv=H_kv, N=N, L=L, Lcap=Lcap, scale=scale)
        err = np.abs(out.float().cpu().numpy().astype(np.float64) - ref)
        assert (err <= abs_bound(ref)).all(), what
        assert attention_errors(out, ref)[1] <= MAX_REL, what
        assert np.abs(lse.cpu().numpy().astype(np.float64) - ref_lse).max() <= 5e-3, what
        done += 1


def test_split_plans_fit_the_device():
    for B, H, N, L in [(1, 32, 64, 2048), (1, 37, 64, 8192), (3, 32, 64, 4096), (1, 1, 64, 16384),
                       (1, 32, 128, 2048), (1, 4, 256, 8192), (256, 32, 64, 4096), (1, 2, 64, 100)]:
        p = rest.tree_attention_plan(B, H, N, 128, L + N)
        ntiles = (L + N + 63) // 64
        units = B * H * (1 if N <= 64 else (N + 127) // 128)
        assert p["splits"] == p["cluster"] * p["clusters_per_unit"]
        assert 1 <= p["cluster"] <= 8 and p["splits"] <= max(ntiles, 1)
        if p["cluster"] > 1:
            assert units * p["clusters_per_unit"] <= p["capacity"], (B, H, N, L, p)
        ws = rest.tree_attention_workspace_bytes(B, H, N, 128, L + N)
        assert (ws == 0) == (p["clusters_per_unit"] == 1)
        if ws:
            assert ws == B * H * p["clusters_per_unit"] * N * 130 * 4
