"""Times rest_draft alone on the workload recipes, over a range of batch sizes.

    python -m paper_2311_08252_b200.draft_bench [--workloads single_stream stress]
                                                [--n-tokens 1000000 100000000] [--n-max 4 16]
                                                [--batches 1 256 4096] [--search auto|single|batched]

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
import time

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
    ap.add_argument("--n-tokens", type=int, nargs="*", default=[100_000_000],
                    help="datastore sizes (tokens); each is capped at the workload's own size")
    ap.add_argument("--n-max", type=int, nargs="*", default=None,
                    help="longest suffix lengths to try (default: the workload's n_max)")
    ap.add_argument("--batches", nargs="*", type=int, default=[1, 64, 256, 1024, 4096])
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--search", choices=["auto", "single", "batched"], default="auto",
                    help="suffix-array search of rest_draft (auto: batched when B exceeds what "
                         "the GPU holds at once)")
    ap.add_argument("--no-workspace", action="store_true",
                    help="pass no scratch: the batched path then runs as a single launch")
    args = ap.parse_args()
    peak, peak_kind = bench.measured_peaks()
    dev = torch.device("cuda:0")
    read_ns = rest.dependent_read_latency_ns(device=dev)
    for name, n_tok in [(nm, nt) for nm in args.workloads for nt in args.n_tokens]:
        w = datagen.WORKLOADS[name].scaled(n_tokens=min(n_tok, datagen.WORKLOADS[name].n_tokens))
        T = datagen.make_tokens(w)
        d_T = torch.from_numpy(T).to(dev)
        torch.cuda.synchronize()
        t_build = time.perf_counter()
        d_sa = rest.rest_suffix_array_build(d_T, w.sa_bytes)
        t_build = time.perf_counter() - t_build
        ds = rest.Datastore(d_T, d_sa, w.vocab)
        Lc = min(w.Lc, 64)                       # only the last n_max tokens are ever read
        for B, n_max in [(B, nx) for B in args.batches for nx in (args.n_max or [w.n_max])]:
            nsets = 4                            # rotate context sets so probes differ call to call
            ctx = [torch.from_numpy(datagen.make_contexts(w, T, B=B, Lc=Lc, salt=s)).to(dev)
                   for s in range(nsets)]
            ctx_len = torch.full((B,), Lc, dtype=torch.int32, device=dev)
            out = rest.alloc_draft_output(B, w.N, dev)
            kw = dict(n_max=n_max, n_min=min(w.n_min, n_max), K=w.K, m=w.m, N=w.N,
                      search={"auto": rest.REST_SEARCH_AUTO, "single": rest.REST_SEARCH_SINGLE,
                              "batched": rest.REST_SEARCH_BATCHED}[args.search])
            ws_bytes = 0 if args.no_workspace else rest.draft_workspace_bytes(B, **kw)
            kw.update(out=out, workspace=torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
                      if ws_bytes else False)
            kp, matched, match_n, nodes = 0, 0, 0, 0
            for s in range(nsets):
                rest.rest_draft(ds, ctx[s], ctx_len, **kw)
                torch.cuda.synchronize()
                rng = out.match_range.cpu().numpy()
                kp += int(np.minimum(rng[:, 1] - rng[:, 0], w.K).sum())
                mn = out.match_n.cpu().numpy()
                matched += int((mn > 0).sum())
                match_n += int(mn.sum())
                nodes += int(out.n_nodes.sum().item())
            kp_mean = kp / (nsets * B)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(args.iters):
                rest.rest_draft(ds, ctx[i % nsets], ctx_len, **kw)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / args.iters
            alg = bench.draft_bytes(w.n_tokens, w.sa_bytes, kw["n_min"], n_max, kp_mean, w.m, w.N) * B
            chain = bench.draft_chain_reads(w.n_tokens, kp_mean)
            print(json.dumps({
                "workload": name, "datastore_tokens": w.n_tokens, "suffix_array_build_s": t_build,
                "B": B, "K": w.K, "m": w.m, "N": w.N, "n_max": n_max, "search": args.search,
                "mean_candidates": kp_mean, "mean_nodes": nodes / (nsets * B),
                "contexts_with_a_match": matched / (nsets * B),
                "mean_matched_length": match_n / max(matched, 1),
                "us_per_call": us, "trees_per_s": B / us * 1e6, "algorithmic_bytes": alg,
                "achieved_gbs": alg / us / 1e3, "peak_gbs": peak, "peak_kind": peak_kind,
                "frac": alg / us / 1e3 / peak,
                "dependent_read_ns": read_ns, "dependent_reads_on_critical_path": chain,
                "latency_floor_us": chain * read_ns / 1e3,
                "frac_of_latency_floor": chain * read_ns / 1e3 / us}), flush=True)
        ds.close()
        del ds, d_T, d_sa
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
