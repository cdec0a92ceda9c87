"""rest_probe_dependent_reads: the chase ends where a host chase of the same table ends, and the
time per read is that of a memory access, not of a cache hit or of nothing at all."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2311_08252_b200 as rest

pytestmark = pytest.mark.gpu


def test_chase_follows_the_table():
    rng = np.random.default_rng(0)
    n = 1 << 20
    perm = rng.permutation(n)
    nxt = np.empty(n, np.int32)
    nxt[perm] = np.roll(perm, -1)
    nxt[12345] = -7                       # an out-of-range entry sends the chase to slot 0
    d = torch.from_numpy(nxt).cuda()
    out = torch.zeros(2, dtype=torch.int64, device="cuda")
    steps, start = 5000, 17
    rc = rest.lib().rest_probe_dependent_reads(d.data_ptr(), n, start, steps, out.data_ptr(), None)
    torch.cuda.synchronize()
    assert rc == 0
    idx = start
    for _ in range(steps):
        if not (0 <= idx < n):
            idx = 0
        idx = int(np.uint32(nxt[idx]))
    assert int(out[1].item()) == idx
    assert out[0].item() > 0
    L = rest.lib()
    assert L.rest_probe_dependent_reads(None, n, 0, 1, out.data_ptr(), None) == 1
    assert L.rest_probe_dependent_reads(d.data_ptr(), 0, 0, 1, out.data_ptr(), None) == 1


def test_latency_is_that_of_dram():
    ns = rest.dependent_read_latency_ns(table_bytes=1 << 29, steps=2048)
    assert 150.0 < ns < 3000.0, ns
