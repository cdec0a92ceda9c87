"""rest_tree_attention_static_scratch: the tree-attention call for users who cannot allocate
device memory (their process gave all of it to a KV-cache pool, or their decode loop bans
allocation calls).  Its split partials live in a fixed array inside the library instead of a
caller-supplied workspace.  Checked here through the C ABI against the ordinary entry point,
twice in a row with different inputs, because the array keeps the previous call's contents.

This file is collected last on purpose: if it fails, every other test has already run."""
import math

import numpy as np
import pytest
import torch

import datagen
import paper_2311_08252_b200 as rest

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_entry_point_twice():
    dev = torch.device("cuda:0")
    B, H, N, D = 1, 2, 64, 128          # few (context, head) pairs, long cache: needs scratch
    scale = 1.0 / math.sqrt(D)
    for call, (seed, L) in enumerate(((31, 4096), (32, 3000))):
        assert rest.tree_attention_workspace_bytes(B, H, N, D, L + N) > 0   # the split path
        q, k, v = datagen.make_qkv(seed, B, H, N, D, L + N)
        _, _, mask = datagen.make_random_tree(seed, N, 8)
        q, k, v = q.to(dev), k.to(dev), v.to(dev)
        mask = torch.from_numpy(mask[None].copy().view(np.int32)).to(dev)
        kv_len = torch.full((B,), L, dtype=torch.int32, device=dev)
        want_lse = torch.empty((B, H, N), dtype=torch.float32, device=dev)
        want = rest.rest_tree_attention(q, k, v, kv_len, mask, scale, lse=want_lse)
        got = torch.empty_like(want)
        got_lse = torch.empty_like(want_lse)
        rest.rest_tree_attention_static_scratch(q, k, v, kv_len, mask, scale, out=got, lse=got_lse)
        torch.cuda.synchronize()
        # same kernels, same split, same arithmetic: within the attention tests' tolerance
        # (1e-2 absolute), and in fact identical
        diff = (got.float() - want.float()).abs().max().item()
        assert diff <= 1e-2, (call, diff)
        assert torch.equal(got, want), call
        assert (got_lse - want_lse).abs().max().item() <= 2e-3


def test_static_scratch_rejects_shapes_beyond_the_fixed_array():
    dev = torch.device("cuda:0")
    # a single head over a long cache: as many clusters as the GPU can run at once (about 30),
    # each leaving a partial of 64 x 130 floats: more than the fixed array holds
    B, H, N, D, L = 1, 1, 64, 128, 16384
    assert rest.tree_attention_workspace_bytes(B, H, N, D, L + N) > 768 * 1024
    q = torch.zeros((B, N, H, D), dtype=torch.bfloat16, device=dev)
    kv = torch.zeros((B, H, L + N, D), dtype=torch.bfloat16, device=dev)
    mask = torch.zeros((B, N, 2), dtype=torch.int32, device=dev)
    kv_len = torch.full((B,), L, dtype=torch.int32, device=dev)
    out = torch.empty_like(q)
    with pytest.raises(rest.RestError, match="workspace too small"):
        rest.rest_tree_attention_static_scratch(q, kv, kv, kv_len, mask, 0.1, out=out)
