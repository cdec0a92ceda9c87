"""The per-kernel shared-memory attribute is set lazily, the first time a kernel needs more than
it was given before.  Whichever entry point a process calls first, the others must still get
theirs: run draft (every launch form, with the largest shared-memory footprint) before tree
attention (both kernels) in a fresh process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import math, sys
import numpy as np, torch
sys.path.insert(0, %r)
import datagen
import paper_2311_08252_b200 as rest
dev = torch.device("cuda:0")
rng = np.random.default_rng(3)
T = rng.integers(0, 2, 40000).astype(np.int32)
for sa_bytes in (4, 8):
    sa = datagen.build_suffix_array(T, 2, W=32, sa_bytes=sa_bytes)
    ds = rest.Datastore(torch.from_numpy(T).to(dev), torch.from_numpy(sa).to(dev), 2)
    ctx = torch.from_numpy(rng.integers(0, 2, (8, 24)).astype(np.int32)).to(dev)
    ctx_len = torch.full((8,), 24, dtype=torch.int32, device=dev)
    outs = []
    for search, ws in ((rest.REST_SEARCH_SINGLE, None), (rest.REST_SEARCH_BATCHED, False),
                       (rest.REST_SEARCH_BATCHED, None)):
        o = rest.rest_draft(ds, ctx, ctx_len, K=20000, m=16, N=128, search=search, workspace=ws)
        torch.cuda.synchronize()
        outs.append(o.tokens.cpu().numpy())
    assert all(np.array_equal(outs[0], x) for x in outs[1:])
for N, L in ((64, 300), (128, 700)):
    B, H, D = 2, 4, 128
    q, k, v = datagen.make_qkv(5, B, H, N, D, L + N)
    mask = np.zeros((B, N, (N + 31) // 32), np.uint32)
    for i in range(N):
        mask[:, i, i >> 5] = np.uint32(1) << np.uint32(i & 31)
    kv_len = torch.full((B,), L, dtype=torch.int32, device=dev)
    out = rest.rest_tree_attention(q.to(dev), k.to(dev), v.to(dev), kv_len,
                                   torch.from_numpy(mask.view(np.int32)).to(dev), 1.0 / math.sqrt(D))
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
assert rest.device_error_flags() == 0
print("ok")
""" % ROOT


def test_draft_before_attention_in_a_fresh_process():
    r = subprocess.run([sys.executable, "-c", SCRIPT], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stdout + r.stderr
