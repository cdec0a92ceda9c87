"""Times rest_draft alone on the workload recipes, over a range of batch sizes.

    python -m paper_2311_08252_b200.draft_bench [--workloads single_stream stress]
                                                [--n-tokens 100000000] [--batches 1 256 4096]

The datastore is the workload's recipe at --n-tokens tokens; its suffix array is built on the
device (rest_suffix_array_build).  Contexts follow the workload's context recipe.
Prints one JSON line per (workload, batch): microseconds per call, trees/s, the algorithmic
bytes of the call (bisection probes for every suffix length + the candidate rows actually
gathered + outputs), the fraction of the measured HBM copy bandwidth they amount to, and the
latency floor of one call: the measured latency of a dependent DRAM read times the number of
dependent reads on a draft's critical path (no call can finish faster, whatever the batch).
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

    import bench
    import datagen
    import paper_2311_08252_b200 as rest

    ap = argparse.ArgumentParser()
    ap.add_argument("--workloads", nargs="*", default=["single_stream", "stress"])
    ap.add_argument("--n-tokens", type=int, default=100_000_000)
    ap.add_argument("--batches", nargs="*", type=int, default=[1, 64, 256, 1024, 4096])
    ap.add_argument("--iters", type=int, default=20)
    args = ap.parse_args()
    peak, peak_kind = bench.measured_peaks()
    dev = torch.device("cuda:0")
    read_ns = rest.dependent_read_latency_ns(device=dev)
    for name in args.workloads:
        w = datagen.WORKLOADS[name].scaled(n_tokens=min(args.n_tokens, datagen.WORKLOADS[name].n_tokens))
        T = datagen.make_tokens(w)
        d_T = torch.from_numpy(T).to(dev)
        d_sa = rest.rest_suffix_array_build(d_T, w.sa_bytes)
        ds = rest.Datastore(d_T, d_sa, w.vocab)
        Lc = min(w.Lc, 64)                       # only the last n_max tokens are ever read
        for B in args.batches:
            nsets = 4                            # rotate context sets so probes differ call to call
            ctx = [torch.from_numpy(datagen.make_contexts(w, T, B=B, Lc=Lc, salt=s)).to(dev)
                   for s in range(nsets)]
            ctx_len = torch.full((B,), Lc, dtype=torch.int32, device=dev)
            out = rest.alloc_draft_output(B, w.N, dev)
            kw = dict(n_max=w.n_max, n_min=w.n_min, K=w.K, m=w.m, N=w.N, out=out)
            kp = 0
            for s in range(nsets):
                rest.rest_draft(ds, ctx[s], ctx_len, **kw)
                torch.cuda.synchronize()
                rng = out.match_range.cpu().numpy()
                kp += int(np.minimum(rng[:, 1] - rng[:, 0], w.K).sum())
            kp_mean = kp / (nsets * B)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(args.iters):
                rest.rest_draft(ds, ctx[i % nsets], ctx_len, **kw)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / args.iters
            alg = bench.draft_bytes(w.n_tokens, w.sa_bytes, w.n_min, w.n_max, kp_mean, w.m, w.N) * B
            print(json.dumps({
                "workload": name, "datastore_tokens": w.n_tokens, "B": B, "K": w.K, "m": w.m, "N": w.N,
                "mean_candidates": kp_mean, "mean_nodes": float(out.n_nodes.float().mean().item()),
                "us_per_call": us, "trees_per_s": B / us * 1e6, "algorithmic_bytes": alg,
                "achieved_gbs": alg / us / 1e3, "peak_gbs": peak, "peak_kind": peak_kind,
                "frac": alg / us / 1e3 / peak,
                "dependent_read_ns": read_ns,
                "dependent_reads_on_critical_path": bench.draft_chain_reads(w.n_tokens, kp_mean),
                "latency_floor_us": bench.draft_chain_reads(w.n_tokens, kp_mean) * read_ns / 1e3,
                "frac_of_latency_floor": bench.draft_chain_reads(w.n_tokens, kp_mean) * read_ns / 1e3 / us}),
                flush=True)
        ds.close()
        del ds
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
