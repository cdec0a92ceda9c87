"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI binding and
compare with the CPU oracle on the same seeded inputs."""
import numpy as np
import torch

import oracle
import paper_2311_08252_b200 as rest

DRAFT_KEYS = ("tokens", "parents", "depth", "pos_ids", "n_nodes", "match_n", "match_range",
              "node_count", "status")


def dev():
    return torch.device("cuda:0")


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dev())


def gpu_draft(T, sa, vocab, ctx, ctx_len, validate=False, index=True, **kw):
    ds = rest.Datastore(to_dev(T), to_dev(sa), vocab, validate=validate, index=index)
    out = rest.rest_draft(ds, to_dev(ctx), to_dev(np.asarray(ctx_len, np.int32)), **kw)
    torch.cuda.synchronize()
    res = {k: getattr(out, k).cpu().numpy() for k in DRAFT_KEYS}
    res["mask"] = out.mask.cpu().numpy().view(np.uint32)
    ds.close()
    return res, out


def assert_draft_equal(got, ref, what=""):
    for k in DRAFT_KEYS + ("mask",):
        if not np.array_equal(got[k], ref[k]):
            bad = np.nonzero((got[k] != ref[k]).reshape(got[k].shape[0], -1).any(1))[0]
            raise AssertionError(f"{what}: '{k}' differs for contexts {bad[:10].tolist()} "
                                 f"(first: got {got[k][bad[0]].tolist()} want {ref[k][bad[0]].tolist()})")


def bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def attention_errors(out_gpu, ref):
    """Max abs error, and max relative L2 error per (b, i, h) row."""
    got = out_gpu.float().cpu().numpy().astype(np.float64)
    err = got - ref
    max_abs = np.abs(err).max()
    row = np.sqrt((err ** 2).sum(-1)) / np.maximum(np.sqrt((ref ** 2).sum(-1)), 1e-30)
    return max_abs, row.max()
