"""Times rest_tree_attention alone at the attention shapes of the five workloads.

    python -m paper_2311_08252_b200.attention_bench [--workloads tiny single_stream ...]
                                                    [--max-gb 20] [--iters 20]

For every workload: B contexts x H heads x N draft nodes over a KV prefix of L tokens, random
bf16 data, a seeded random tree mask.  The batch is cut down (and said so) when the KV cache
would exceed --max-gb.  Enough distinct KV buffers are rotated that consecutive launches never
hit L2; one pass over them is replayed from a CUDA graph.  Prints one JSON line per workload: microseconds per layer, achieved algorithmic GB/s
and the fraction of the measured HBM copy bandwidth (MEASURED_PEAKS.json, else 6650 GB/s).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    import numpy as np
    import torch

    import datagen
    import paper_2311_08252_b200 as rest

    ap = argparse.ArgumentParser()
    ap.add_argument("--workloads", nargs="*", default=list(datagen.WORKLOADS))
    ap.add_argument("--max-gb", type=float, default=20.0)
    ap.add_argument("--iters", type=int, default=20)
    args = ap.parse_args()
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"])
        peak_kind = "measured"
    except Exception:
        peak, peak_kind = 6650.0, "fallback"
    dev = torch.device("cuda:0")
    for name in args.workloads:
        w = datagen.WORKLOADS[name]
        H, N, D, L = w.H, w.N, w.D, w.L
        per_ctx = H * 2 * (L + N) * D * 2
        B = max(1, min(w.B, int(args.max_gb * 1e9 // per_ctx)))
        kv_bytes = B * per_ctx
        nbuf = max(2, min(32, int(math.ceil(400e6 / kv_bytes)) + 1))   # > 126 MB L2 between reuses
        if nbuf * kv_bytes > 2 * args.max_gb * 1e9:
            nbuf = 2
        g = torch.Generator(device=dev)
        g.manual_seed(w.seed)
        bufs = []
        for _ in range(nbuf):
            k = torch.randn((B, H, L + N, D), generator=g, device=dev, dtype=torch.bfloat16)
            v = torch.randn((B, H, L + N, D), generator=g, device=dev, dtype=torch.bfloat16)
            bufs.append((k, v))
        q = torch.randn((B, N, H, D), generator=g, device=dev, dtype=torch.bfloat16)
        _, _, mask = datagen.make_random_tree(w.seed, N, w.m)
        mask = torch.from_numpy(np.broadcast_to(mask, (B,) + mask.shape).copy().view(np.int32)).to(dev)
        kv_len = torch.full((B,), L, dtype=torch.int32, device=dev)
        out = torch.empty((B, N, H, D), dtype=torch.bfloat16, device=dev)
        ws_bytes = rest.tree_attention_workspace_bytes(B, H, N, D, L + N)
        ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
        scale = 1.0 / math.sqrt(D)

        def call(i):
            k, v = bufs[i % nbuf]
            rest.rest_tree_attention(q, k, v, kv_len, mask, scale, max_kv=L + N, out=out, workspace=ws)

        for i in range(3):
            call(i)
        torch.cuda.synchronize()
        # one pass over the rotating buffers is captured into a CUDA graph and replayed, so that
        # small shapes are timed by their kernels and not by the host's launch path
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(nbuf):
                call(i)
        graph.replay()
        torch.cuda.synchronize()
        reps = max(1, (args.iters + nbuf - 1) // nbuf)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (reps * nbuf)
        alg = B * H * 2 * (L + N) * D * 2 + B * H * 2 * N * D * 2 + B * N * N // 8
        print(json.dumps({
            "workload": name, "B": B, "B_full": w.B, "H": H, "N": N, "L": L,
            "kv_buffers_rotated": nbuf, "us_per_layer": us, "algorithmic_bytes": alg,
            "achieved_gbs": alg / us / 1e3, "peak_gbs": peak, "peak_kind": peak_kind,
            "frac": alg / us / 1e3 / peak, "frac_of_8TBs": alg / us / 1e3 / 8000.0,
            "device_error_flags": rest.device_error_flags()}))
        del bufs, q, out, ws
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
