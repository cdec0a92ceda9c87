"""Parity at the full sizes of the workload configurations, on sampled outputs.

Tree attention runs once over the whole batch (17.7 GB of K/V for the batched-serving shape,
10.9 GB for the large one, 34.9 GB for the stress one, all generated on the device from a seed);
the fp64 oracle then recomputes a sample of (context, head) units one by one from the very same
bytes.  The draft runs over the full 100 M-token single-stream datastore and every drafted tree
is compared with the oracle's, bit for bit."""
import math

import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2311_08252_b200 as rest
from gpu_util import DRAFT_KEYS, assert_draft_equal, attention_errors, bits, gpu_draft, to_dev

pytestmark = pytest.mark.gpu

MAX_ABS = 1e-2
MAX_REL = 2e-2


@pytest.mark.parametrize("name", ["batched", "large", "stress"])
def test_tree_attention_full_shape_sampled_units(name):
    w = datagen.WORKLOADS[name]
    B, H, N, D, L = w.B, w.H, w.N, w.D, w.L
    need = 2 * B * H * (L + N) * D * 2
    free, _ = torch.cuda.mem_get_info()
    if free < need + (4 << 30):
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory")
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed)
    k = torch.randn((B, H, L + N, D), generator=g, device=dev, dtype=torch.bfloat16)
    v = torch.randn((B, H, L + N, D), generator=g, device=dev, dtype=torch.bfloat16)
    q = torch.randn((B, N, H, D), generator=g, device=dev, dtype=torch.bfloat16)
    masks = np.stack([datagen.make_random_tree(w.seed * 1000 + b, N, w.m)[2] for b in range(B)])
    # ragged prefix lengths: most contexts full, a few shorter ones
    kv_len = np.full(B, L, np.int32)
    kv_len[1::7] = L - 37
    kv_len[3::11] = L // 3 + 5
    scale = 1.0 / math.sqrt(D)
    out = rest.rest_tree_attention(q, k, v, to_dev(kv_len), to_dev(masks), scale, max_kv=L + N)
    torch.cuda.synchronize()
    assert rest.device_error_flags() == 0
    rng = np.random.default_rng(w.seed)
    units = {(0, 0), (B - 1, H - 1), (1, H // 2), (3, 1)}
    while len(units) < 10:
        units.add((int(rng.integers(0, B)), int(rng.integers(0, H))))
    for b, h in sorted(units):
        ref = oracle.tree_attention(bits(q[b:b + 1, :, h:h + 1].cpu()), bits(k[b:b + 1, h:h + 1].cpu()),
                                    bits(v[b:b + 1, h:h + 1].cpu()), kv_len[b:b + 1], masks[b:b + 1], scale)
        max_abs, max_rel = attention_errors(out[b:b + 1, :, h:h + 1], ref)
        assert max_abs <= MAX_ABS and max_rel <= MAX_REL, (name, b, h, max_abs, max_rel)
    del k, v, q, out
    torch.cuda.empty_cache()


def test_draft_full_single_stream_datastore():
    w = datagen.WORKLOADS["single_stream"]             # 100 M tokens, int32 suffix array
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab)
    B, Lc = 96, 64
    ctx = datagen.make_contexts(w, T, B=B, Lc=Lc)
    ctx_len = np.full(B, Lc, np.int32)
    ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, K=w.K, m=w.m, N=w.N)
    got, _ = gpu_draft(T, sa, w.vocab, ctx, ctx_len, K=w.K, m=w.m, N=w.N)
    assert_draft_equal(got, ref, "single_stream, 100 M tokens")
    assert (ref["n_nodes"] > 0).mean() > 0.5


def host_memory_available():
    import psutil
    return psutil.virtual_memory().available


@pytest.mark.parametrize("name,n_tokens", [("stress", 500_000_000), ("batched", 1_000_000_000),
                                           ("large", 1_000_000_000)])
def test_draft_largest_datastores(name, n_tokens):
    """The 500 M-token stress datastore, the 1 B-token batched one, and the large recipe with its
    int64 suffix array at 1 B tokens, each at its configuration's batch size.  The suffix array
    is built on the device (rest_suffix_array_build) and copied back, so that the oracle searches
    the very same array."""
    w = datagen.WORKLOADS[name].scaled(n_tokens=n_tokens)
    need_dev = n_tokens * (4 + w.sa_bytes) + rest.lib().rest_suffix_array_workspace_bytes(n_tokens)
    free, _ = torch.cuda.mem_get_info()
    if free < need_dev + (2 << 30):
        pytest.skip(f"needs {need_dev / 2**30:.0f} GiB of device memory, {free / 2**30:.0f} GiB free")
    need_host = n_tokens * (4 + w.sa_bytes) * 2
    if host_memory_available() < need_host + (4 << 30):
        pytest.skip(f"needs {need_host / 2**30:.0f} GiB of host memory")
    T = datagen.make_tokens(w)
    d_T = to_dev(T)
    d_sa = rest.rest_suffix_array_build(d_T, w.sa_bytes)
    torch.cuda.empty_cache()
    ds = rest.Datastore(d_T, d_sa, w.vocab, validate=True)
    sa = d_sa.cpu().numpy()
    B, Lc = w.B, 64
    ctx = datagen.make_contexts(w, T, B=B, Lc=Lc)
    ctx_len = np.full(B, Lc, np.int32)
    kw = dict(K=w.K, m=w.m, N=w.N)
    ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, **kw)
    for search in (rest.REST_SEARCH_SINGLE, rest.REST_SEARCH_BATCHED):
        out = rest.rest_draft(ds, to_dev(ctx), to_dev(ctx_len), search=search, **kw)
        torch.cuda.synchronize()
        got = {k: getattr(out, k).cpu().numpy() for k in DRAFT_KEYS}
        got["mask"] = out.mask.cpu().numpy().view(np.uint32)
        assert_draft_equal(got, ref, f"{name}, {n_tokens} tokens, search {search}")
    assert (ref["n_nodes"] > 0).mean() > 0.5
    ds.close()
    del d_T, d_sa, ds
    torch.cuda.empty_cache()


def test_draft_large_workload_at_its_full_size():
    """The large workload as stated: 4 B tokens, int64 suffix array (32 GB) built on the device
    in groups of first-token buckets, positions beyond 2^31 in the matched ranges."""
    w = datagen.WORKLOADS["large"]
    n = w.n_tokens
    need_dev = n * 12 + rest.lib().rest_suffix_array_workspace_bytes(n) + rest.lib().rest_datastore_aux_bytes(n, 8, w.vocab)
    free, _ = torch.cuda.mem_get_info()
    if free < need_dev + (4 << 30):
        pytest.skip(f"needs {need_dev / 2**30:.0f} GiB of device memory, {free / 2**30:.0f} GiB free")
    need_host = n * 12 * 2
    if host_memory_available() < need_host + (8 << 30):
        pytest.skip(f"needs {need_host / 2**30:.0f} GiB of host memory, "
                    f"{host_memory_available() / 2**30:.0f} GiB available")
    T = datagen.make_tokens(w)
    d_T = to_dev(T)
    d_sa = rest.rest_suffix_array_build(d_T, 8)
    torch.cuda.empty_cache()
    ds = rest.Datastore(d_T, d_sa, w.vocab, validate=True)
    sa = d_sa.cpu().numpy()
    B, Lc = w.B, 64
    ctx = datagen.make_contexts(w, T, B=B, Lc=Lc)
    ctx_len = np.full(B, Lc, np.int32)
    kw = dict(K=w.K, m=w.m, N=w.N)
    ref = oracle.draft(T, sa, w.vocab, ctx, ctx_len, **kw)
    for search in (rest.REST_SEARCH_SINGLE, rest.REST_SEARCH_BATCHED):
        out = rest.rest_draft(ds, to_dev(ctx), to_dev(ctx_len), search=search, **kw)
        torch.cuda.synchronize()
        got = {k: getattr(out, k).cpu().numpy() for k in DRAFT_KEYS}
        got["mask"] = out.mask.cpu().numpy().view(np.uint32)
        assert_draft_equal(got, ref, f"large, {n} tokens, search {search}")
    assert (ref["n_nodes"] > 0).mean() > 0.5
    # the matched ranges reach suffix-array slots and token positions that need 64 bits
    assert ref["match_range"].max() > 2**31
    high = [int(sa[int(lo):int(min(hi, lo + 5000))].max()) for lo, hi in ref["match_range"] if hi > lo]
    assert max(high) > 2**31
    ds.close()
    del d_T, d_sa, ds
    torch.cuda.empty_cache()
