#!/usr/bin/env python
"""Benchmark of one REST decoding step's hot path on B200: rest_draft -> rest_tree_attention
for every layer -> rest_accept, on the seeded synthetic workloads of datagen.WORKLOADS.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

The headline workload is the largest one that fits the GPU: "stress" (500 M-token datastore,
128 contexts, K = 20000, m = 16, N = 128; one layer of 32 heads x 128 over a 16384-token bf16 KV
cache, 34.9 GB), else "batched".  Prints ONE JSON line.  `value` is whole-path draft trees per
second with all inputs resident in HBM; `e2e` is the same with host<->device copies of the
step's inputs and results inside the timed region; `workloads` carries the draft and
tree-attention timings of all five workloads, `sweeps` the retrieval time against datastore
size and against the longest suffix length.  `--impl reference` times the CPU oracle (a
deliberately plain program) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import datagen  # noqa: E402

METRIC = "draft trees/s through retrieve+trie+mask, tree attention (all layers) and accept"
UNIT = "trees/s"
N_CTX_POOL = 16          # distinct context sets rotated through the steps
L2_BYTES = 126e6
# dram__bytes_read.sum + dram__bytes_write.sum per (context, head) unit of one attention launch,
# from the small-case ncu captures summarised under profiles/ (each taken on the kernel as it
# stands; a launch of the full shape is that many units, every unit an independent block that
# reads its own K/V once, so traffic grows in proportion).  Shapes without a capture report null.
NCU_TRAFFIC_PER_UNIT = {
    # (kernel, N, L): bytes per (context, head)
    ("tree_attention_wide_kernel", 128, 16384): 2449.3e6 / (9 * 32),
    ("tree_attention_ws_kernel", 64, 4096): 970.1e6 / (14 * 32),
    ("tree_attention_ws_kernel", 64, 2048): 35_185_408 / 32,
}


# The same for the draft kernel of the single-context path: DRAM bytes of one launch per candidate
# row gathered (stress recipe, 100 M tokens, B = 128, 2409 rows per context on average; the rows
# and their suffix-array entries are nearly all of the traffic, so it grows with the rows).
NCU_DRAFT_TRAFFIC_PER_ROW = {"stress": (73.84e6 + 2.52e6) / (128 * 2408.6)}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="auto", choices=["auto"] + list(datagen.WORKLOADS))
    ap.add_argument("--n-tokens", type=int, default=None,
                    help="override the datastore size (debugging only; changes the workload name)")
    ap.add_argument("--warm-l2", action="store_true",
                    help="--part draft: no L2 flush between small calls (for comparison with older figures)")
    ap.add_argument("--e2e-chunks", default=None,
                    help="end-to-end leg: sizes of the context chunks whose copies overlap the compute of "
                         "their neighbours, e.g. 32,32,32,32 (default: B/8, 3B/8, 3B/8, B/8 for a single-layer "
                         "step of 64 contexts or more, else one chunk)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true",
                    help="skip the table of the other workloads and the sweeps")
    ap.add_argument("--part", default="step", choices=["step", "draft", "attention"],
                    help="time one call alone on a (possibly reduced) case and print its record: what "
                         "the ncu captures under profiles/ run")
    ap.add_argument("--batch", type=int, default=None, help="--part draft: contexts per call")
    ap.add_argument("--max-gb", type=float, default=80.0,
                    help="--part attention: cap on the K/V bytes (the batch is cut to fit)")
    ap.add_argument("--iters", type=int, default=12, help="--part: timed calls")
    return ap.parse_args()


def measured_tensor_peak():
    """Sustained dense bf16 TFLOP/s of the measured-peaks file (fallback: 1400)."""
    try:
        return float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 1400.0, "fallback"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0]))
                mx.append(float(p[1]))
            except ValueError:
                continue
            for nm, val in zip(names, p[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def attention_bytes(B, H, H_kv, N, D, L):
    """Algorithmic bytes of one tree-attention layer: K and V once, Q in, O out, mask."""
    return B * H_kv * 2 * (L + N) * D * 2 + B * H * 2 * N * D * 2 + B * N * N // 8


def draft_bytes(n_tokens, sa_bytes, n_min, n_max, Kp, m, N):
    """Algorithmic bytes of one draft: bisection probes for every suffix length, the gathered
    rows actually used (Kp), and the outputs."""
    lg = math.ceil(math.log2(max(n_tokens, 2)))
    search = sum(2 * lg * (sa_bytes + 4 * n) for n in range(n_min, n_max + 1))
    return search + Kp * (sa_bytes + 4 * m) + N * (16 + N // 8)


def draft_sector_bytes(n_tokens, sa_bytes, n_min, n_max, Kp, m, N):
    """The same accesses counted in whole 32-byte DRAM sectors: a suffix-array entry costs one
    sector, a row of k tokens at an arbitrary 4-byte offset touches ceil((4k + 28) / 32) of
    them.  DRAM counters of the draft kernel sit near this figure, not near the useful bytes."""
    lg = math.ceil(math.log2(max(n_tokens, 2)))
    row = lambda k: 32 * math.ceil((4 * k + 28) / 32)
    search = sum(2 * lg * (32 + row(n)) for n in range(n_min, n_max + 1))
    return search + Kp * (32 + row(m)) + 32 * math.ceil(N * (16 + N // 8) / 32)


def draft_chain_reads(n_tokens, mean_candidates, indexed=True):
    """Dependent global reads on the critical path of one draft.  With the bucket index: the
    context length then its tokens, the index entry, one or two 32-ary rounds inside the pair's
    range (suffix-array entry, then the tokens it points to), the block-wide upper bound (one
    round, a second one when the run is long), one gather round, the emitted tokens.  Without
    it: ceil(log33 n) rounds for the lower bound instead of the index entry."""
    r_upper = 1 + (1 if mean_candidates > 256 else 0)
    if indexed:
        return 2 + 1 + 2 * 2 + 2 * r_upper + 2 + 1
    r_lower = math.ceil(math.log(max(n_tokens, 2)) / math.log(33))
    return 2 + 2 * r_lower + 2 * r_upper + 2 + 1


def attention_kernel_name(B, H, H_kv, N):
    """The kernel rest_tree_attention runs for this shape (see csrc/tree_attention.cu)."""
    packed = N == 64 and (H // H_kv) % 2 == 0 and B * H // 2 >= 2 * 148
    return "tree_attention_wide_kernel" if (N > 64 or packed) else "tree_attention_ws_kernel"


# ---------------------------------------------------------------------------------------
# set-up helpers (untimed)
# ---------------------------------------------------------------------------------------
def sync_all(torch):
    torch.cuda.synchronize()


def device_datastore(rest, torch, w, dev, tokens=None, validate=False):
    """Tokens of workload `w` on the device, its suffix array built there
    (rest_suffix_array_build) and a datastore handle with the bucket index.  `tokens`: a host
    array to take the first w.n_tokens tokens from (the generator's streams are prefix-stable:
    a shorter stream of the same recipe is the beginning of a longer one)."""
    t0 = time.perf_counter()
    T = datagen.make_tokens(w) if tokens is None else np.ascontiguousarray(tokens[:w.n_tokens])
    t_gen = time.perf_counter() - t0
    d_T = torch.from_numpy(T).to(dev)
    sync_all(torch)
    t0 = time.perf_counter()
    d_sa = rest.rest_suffix_array_build(d_T, w.sa_bytes)
    t_sa = time.perf_counter() - t0
    torch.cuda.empty_cache()
    t0 = time.perf_counter()
    ds = rest.Datastore(d_T, d_sa, w.vocab, validate=validate, index=True)
    sync_all(torch)
    t_index = time.perf_counter() - t0
    return T, d_T, d_sa, ds, {"token_generation_s": t_gen, "suffix_array_build_s": t_sa,
                              "index_build_s": t_index}


def time_draft(rest, torch, ds, w, T, B, dev, n_max=None, iters=20, peak=6650.0, read_ns=None, cold=True):
    """rest_draft alone: B contexts of workload w's recipe per call, four context sets rotated so
    that the probes differ from call to call.  CUDA events around replays of a graph of eight
    consecutive calls (at least `iters` calls in all)."""
    n_max = w.n_max if n_max is None else n_max
    n_min = min(w.n_min, n_max)
    Lc = min(w.Lc, 64)                       # only the last n_max tokens are ever read
    nsets = 4
    ctx = [torch.from_numpy(datagen.make_contexts(w, T, B=B, Lc=Lc, salt=s)).to(dev) for s in range(nsets)]
    ctx_len = torch.full((B,), Lc, dtype=torch.int32, device=dev)
    out = rest.alloc_draft_output(B, w.N, dev)
    kw = dict(n_max=n_max, n_min=n_min, K=w.K, m=w.m, N=w.N)
    ws_bytes = rest.draft_workspace_bytes(B, **kw)
    kw.update(out=out, workspace=torch.empty(ws_bytes, dtype=torch.uint8, device=dev) if ws_bytes else False)
    kp, matched, match_n, nodes = 0, 0, 0, 0
    for s in range(nsets):
        rest.rest_draft(ds, ctx[s], ctx_len, **kw)
        sync_all(torch)
        rng = out.match_range.cpu().numpy()
        kp += int(np.minimum(rng[:, 1] - rng[:, 0], w.K).sum())
        mn = out.match_n.cpu().numpy()
        matched += int((mn > 0).sum())
        match_n += int(mn.sum())
        nodes += int(out.n_nodes.sum().item())
    kp_mean = kp / (nsets * B)
    # The calls are replayed from one CUDA graph that holds eight of them back to back (the
    # context sets in turn), like the attention timing: neither the host's launch path nor the
    # start of a graph decides the number.  A call that touches less than L2 holds would find
    # its rows and probes there when its context set comes round again, which a decoding loop
    # (gigabytes of weights and K/V between two drafts) never does: such calls are timed with
    # a fill of 1.5 x L2 before each, and the fills alone are timed and subtracted.
    per_graph = 8
    touched = draft_sector_bytes(w.n_tokens, w.sa_bytes, n_min, n_max, kp_mean, w.m, w.N) * B
    flush = None
    if cold and touched * nsets < 4 * L2_BYTES:
        flush = torch.empty(int(1.5 * L2_BYTES), dtype=torch.uint8, device=dev)

    def graph_of(with_calls):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(per_graph):
                if flush is not None:
                    flush.fill_(i)
                if with_calls:
                    rest.rest_draft(ds, ctx[i % nsets], ctx_len, **kw)
        return g

    def seconds_per_item(g, reps):
        g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync_all(torch)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        sync_all(torch)
        return e0.elapsed_time(e1) / 1e3 / (reps * per_graph)

    reps = max(2, (iters + per_graph - 1) // per_graph)
    graph = graph_of(True)
    us = seconds_per_item(graph, reps) * 1e6
    if flush is not None:
        fill_graph = graph_of(False)
        us -= seconds_per_item(fill_graph, reps) * 1e6
        del fill_graph
    alg = draft_bytes(w.n_tokens, w.sa_bytes, n_min, n_max, kp_mean, w.m, w.N) * B
    res = {"B": B, "n_max": n_max, "us_per_call": us, "trees_per_s": B / us * 1e6,
           "mean_candidates": kp_mean, "mean_nodes": nodes / (nsets * B),
           "contexts_with_a_match": matched / (nsets * B),
           "mean_matched_length": match_n / max(matched, 1),
           "algorithmic_bytes_per_call": alg, "achieved_gbs": alg / us / 1e3,
           "frac": alg / us / 1e3 / peak, "target_50pct_met": bool(alg / us / 1e3 / peak >= 0.5),
           "l2": ("a fill of 1.5 x L2 before every call, the fills timed alone and subtracted" if flush is not None
                  else "four context sets in turn, more bytes between two uses of a set than L2 holds" if cold
                  else "four context sets in turn, nothing flushed: repeated sets may read from L2")}
    if read_ns is not None:
        chain = draft_chain_reads(w.n_tokens, kp_mean)
        res.update({"dependent_reads_on_critical_path": chain, "latency_floor_us": chain * read_ns / 1e3,
                    "frac_of_latency_floor": chain * read_ns / 1e3 / us})
    del graph, flush
    return res


def time_attention(rest, torch, w, dev, B=None, iters=12, peak=6650.0, budget_gb=80.0):
    """rest_tree_attention alone at workload w's attention shape (all B contexts when the KV
    cache fits `budget_gb`): random bf16 data, a seeded random tree mask, enough distinct KV
    buffers rotated that consecutive launches never meet in L2, one pass over them replayed
    from a CUDA graph."""
    H, N, D, L = w.H, w.N, w.D, w.L
    per_ctx = H * 2 * (L + N) * D * 2
    B_full = w.B if B is None else B
    B = max(1, min(B_full, int(budget_gb * 1e9 // per_ctx)))
    kv_bytes = B * per_ctx
    nbuf = 1 if kv_bytes > 4 * L2_BYTES else min(32, int(math.ceil(4 * L2_BYTES / kv_bytes)) + 1)
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
    sync_all(torch)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(nbuf):
            call(i)
    graph.replay()
    sync_all(torch)
    reps = max(1, (iters + nbuf - 1) // nbuf)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    sync_all(torch)
    us = e0.elapsed_time(e1) * 1e3 / (reps * nbuf)
    alg = attention_bytes(B, H, H, N, D, L)
    kernel = attention_kernel_name(B, H, H, N)
    per_unit = NCU_TRAFFIC_PER_UNIT.get((kernel, N, L))
    res = {"B": B, "B_of_workload": w.B, "H": H, "N": N, "L": L, "kv_buffers_rotated": nbuf,
           "kernel": kernel, "us_per_layer": us, "algorithmic_bytes_per_launch": alg,
           "achieved_gbs": alg / us / 1e3, "frac": alg / us / 1e3 / peak,
           "frac_of_nominal_8TBs": alg / us / 1e3 / 8000.0,
           "target_50pct_met": bool(alg / us / 1e3 / peak >= 0.5),
           "traffic": None if per_unit is None else per_unit * B * H,
           "plan": rest.tree_attention_plan(B, H, N, D, L + N)}
    # the same launch against the tensor roofline (S = Q K^T and O = P V: 4 N D (L + N) flops per
    # (context, head)): wide trees are bound by both
    tpeak, tkind = measured_tensor_peak()
    tflops = 4.0 * N * D * (L + N) * H * B / us / 1e6
    res.update({"tensor_tflops": tflops, "frac_of_tensor_sustained": tflops / tpeak, "tensor_peak_kind": tkind})
    del bufs, q, out, ws, graph
    torch.cuda.empty_cache()
    return res


# ---------------------------------------------------------------------------------------
# the CPU oracle on a bounded sample of one step (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------
def oracle_step_sample(w, T, sa, ctxs, n_ctx, n_heads_ctx, seed):
    """Times the CPU oracle on a bounded sample of one step of workload w and scales linearly:
    n_ctx drafts and accepts; fp64 attention for all heads of n_heads_ctx contexts plus one
    head of every context (seeded N(0,1) bf16 tensors of the workload's shape, a seeded random
    tree).  Returns (seconds per full step, details)."""
    import oracle
    import torch
    Lc = ctxs.shape[1]
    n_ctx = min(n_ctx, ctxs.shape[0])
    t0 = time.perf_counter()
    d = oracle.draft(T, sa, w.vocab, ctxs[:n_ctx], np.full(n_ctx, Lc, np.int32),
                     K=w.K, m=w.m, N=w.N, n_max=w.n_max, n_min=w.n_min)
    t_draft = (time.perf_counter() - t0) / n_ctx
    ver = datagen.make_verifier_tokens(seed, d["tokens"], d["parents"], d["n_nodes"], w.vocab)
    t0 = time.perf_counter()
    oracle.accept(d["tokens"], d["parents"], d["n_nodes"], ver, w.m)
    t_accept = (time.perf_counter() - t0) / n_ctx
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    _, _, mask = datagen.make_random_tree(w.seed, w.N, w.m)
    units, t_attn = 0, 0.0
    for B_s, H_s in ((n_heads_ctx, w.H), (w.B, 1)):
        if B_s <= 0:
            continue
        q, k, v = datagen.make_qkv(seed + H_s, B_s, H_s, w.N, w.D, w.L + w.N)
        mk = np.broadcast_to(mask, (B_s,) + mask.shape).copy()
        t0 = time.perf_counter()
        oracle.tree_attention(bits(q), bits(k), bits(v), np.full(B_s, w.L, np.int32), mk, 1.0 / math.sqrt(w.D))
        t_attn += time.perf_counter() - t0
        units += B_s * H_s
    t_unit = t_attn / max(units, 1)
    per_step = w.B * (t_draft + t_accept) + w.layers * w.B * w.H * t_unit
    sample = ("%d of %d drafts+accepts; fp64 attention for all %d heads of %d context(s) plus one head of "
              "all %d contexts (%d of %d (context, head) units of one layer); scaled linearly to one "
              "step of %d layer(s)" % (n_ctx, w.B, w.H, n_heads_ctx, w.B, units, w.B * w.H, w.layers))
    return per_step, {"sample": sample, "t_draft_s": t_draft, "t_accept_s": t_accept,
                      "t_attn_unit_s": t_unit}


def host_datastore(w):
    """Tokens and host-built suffix array for the CPU arm; cached on local disk between runs
    (set-up only)."""
    cache = os.environ.get("REST_B200_CACHE", os.path.join(tempfile.gettempdir(), "rest_b200_cache"))
    tag = f"{w.name}_{w.n_tokens}_{w.seed}_sa{w.sa_bytes}_v2"
    tp, sp = os.path.join(cache, tag + "_tok.npy"), os.path.join(cache, tag + "_sa.npy")
    try:
        if os.path.exists(tp) and os.path.exists(sp):
            T, sa = np.load(tp), np.load(sp)
            if T.size == w.n_tokens and sa.size == w.n_tokens:
                return T, sa
    except Exception:
        pass
    T = datagen.make_tokens(w)
    sa = datagen.build_suffix_array(T, w.vocab, W=32, sa_bytes=w.sa_bytes)
    try:
        os.makedirs(cache, exist_ok=True)
        np.save(tp, T)
        np.save(sp, sa)
    except Exception:
        pass
    return T, sa


def workload_config(w, args, extra=None):
    cfg = {"workload": w.name + ("" if args.n_tokens is None else f"@{w.n_tokens}"),
           "datastore_tokens": w.n_tokens, "sa_bytes": w.sa_bytes, "contexts_per_step": w.B,
           "context_len": w.Lc, "K": w.K, "m": w.m, "N": w.N, "n_max": w.n_max, "n_min": w.n_min,
           "layers": w.layers, "heads": w.H, "head_dim": w.D, "kv_len": w.L,
           "parallelism": "contexts sharded over GPUs, datastore replicated, no collective"}
    if extra:
        cfg.update(extra)
    return cfg


def pick_workload(args, free_bytes=None):
    """The headline workload: the one asked for, else the largest that fits this GPU."""
    if args.workload != "auto":
        w = datagen.WORKLOADS[args.workload]
    else:
        w = datagen.WORKLOADS["stress"]
        need = attention_bytes(w.B, w.H, w.H, w.N, w.D, w.L) + 8 * w.n_tokens + 32 * w.n_tokens + (8 << 30)
        if free_bytes is not None and free_bytes < need:
            w = datagen.WORKLOADS["batched"]
    if args.n_tokens is not None:
        w = w.scaled(n_tokens=args.n_tokens)
    return w


def run_reference(args, rank):
    """The CPU oracle as it stands, on the host cores, on a bounded sample per step."""
    if rank != 0:
        return
    import oracle
    w = pick_workload(args)
    T, sa = host_datastore(w)
    ctxs = datagen.make_contexts(w, T, B=max(w.B, 8), Lc=w.Lc)
    times, parts = [], {}
    for i in range(args.warmup + args.steps):
        per_step, parts = oracle_step_sample_small(w, T, sa, ctxs, w.seed + i)
        if i >= args.warmup:
            times.append(per_step)
    sec = float(np.mean(times))
    value = w.B / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": parts.get("sample")},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def oracle_step_sample_small(w, T, sa, ctxs, seed):
    """One step's sample for the reference arm: small enough that the arm's steps take about a
    second each (4 drafts+accepts, 8 (context, head) attention units), scaled to a full step."""
    import oracle
    import torch
    Lc = ctxs.shape[1]
    n_ctx = min(4, ctxs.shape[0])
    t0 = time.perf_counter()
    d = oracle.draft(T, sa, w.vocab, ctxs[:n_ctx], np.full(n_ctx, Lc, np.int32),
                     K=w.K, m=w.m, N=w.N, n_max=w.n_max, n_min=w.n_min)
    ver = datagen.make_verifier_tokens(seed, d["tokens"], d["parents"], d["n_nodes"], w.vocab)
    oracle.accept(d["tokens"], d["parents"], d["n_nodes"], ver, w.m)
    t_ctx = (time.perf_counter() - t0) / n_ctx
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    H_s = min(8, w.H)
    q, k, v = datagen.make_qkv(seed, 1, H_s, w.N, w.D, w.L + w.N)
    t0 = time.perf_counter()
    oracle.tree_attention(bits(q), bits(k), bits(v), np.full(1, w.L, np.int32), d["mask"][:1], 1.0 / math.sqrt(w.D))
    t_unit = (time.perf_counter() - t0) / H_s
    per_step = w.B * t_ctx + w.layers * w.B * w.H * t_unit
    sample = ("per step: %d of %d drafts+accepts and %d of %d (context, head) fp64 attention units of one "
              "layer, scaled linearly to one step of %d layer(s)" % (n_ctx, w.B, H_s, w.B * w.H, w.layers))
    return per_step, {"sample": sample}


# ---------------------------------------------------------------------------------------
# the GPU arm
# ---------------------------------------------------------------------------------------
def run_ours(args, rank, world, local_rank):
    import torch
    import paper_2311_08252_b200 as rest
    from paper_2311_08252_b200.sharding import max_over_ranks, shard_bounds, whole_job_throughput

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peak, peak_kind = measured_peaks()
    free_bytes, _ = torch.cuda.mem_get_info()
    w = pick_workload(args, free_bytes)

    # ---- inputs (set-up, untimed) --------------------------------------------------------
    # every rank generates the same seeded token stream and builds its own copy of the suffix
    # array and of the bucket index on its GPU (the datastore is replicated; nothing is exchanged)
    T, d_T, d_sa, ds, setup = device_datastore(rest, torch, w, dev, validate=True)
    B, N, H, D, L, layers = w.B, w.N, w.H, w.D, w.L, w.layers
    pool = N_CTX_POOL
    Lc = w.Lc
    # the global batch of every pooled step is world*B contexts; this rank owns one slice
    all_ctx = datagen.make_contexts(w, T, B=pool * B * world, Lc=Lc).reshape(pool, B * world, Lc)
    c0, c1 = shard_bounds(B * world, rank, world)
    ctx_np = np.ascontiguousarray(all_ctx[:, c0:c1])
    d_ctx = torch.from_numpy(ctx_np).to(dev)
    d_ctx_len = torch.full((B,), Lc, dtype=torch.int32, device=dev)
    scale = 1.0 / math.sqrt(D)
    # KV buffers: one per layer when they fit, else as many as fit, used round robin; for
    # shapes that L2 could hold, enough extra buffers that a buffer is never met again in L2
    layer_bytes = 2 * B * H * (L + N) * D * 2
    free_bytes, _ = torch.cuda.mem_get_info()
    nbuf = max(1, min(layers, int(0.7 * free_bytes // layer_bytes)))
    if nbuf * layer_bytes < 4 * L2_BYTES:
        nbuf = min(64, int(math.ceil(4 * L2_BYTES / layer_bytes)) + 1)
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed * 1000 + 100 * rank)
    ks = [torch.randn((B, H, L + N, D), generator=g, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
    vs = [torch.randn((B, H, L + N, D), generator=g, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
    q_all = torch.randn((layers, B, N, H, D), generator=g, device=dev, dtype=torch.bfloat16)
    out_all = torch.empty((layers, B, N, H, D), dtype=torch.bfloat16, device=dev)
    d_kv_len = torch.full((B,), L, dtype=torch.int32, device=dev)
    ws_bytes = rest.tree_attention_workspace_bytes(B, H, N, D, L + N)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
    tree = rest.alloc_draft_output(B, N, dev)
    acc = (torch.empty(B, dtype=torch.int32, device=dev),
           torch.empty((B, w.m), dtype=torch.int32, device=dev),
           torch.empty((B, w.m + 1), dtype=torch.int32, device=dev))
    dkw = dict(n_max=w.n_max, n_min=w.n_min, K=w.K, m=w.m, N=N)
    dws_bytes = rest.draft_workspace_bytes(B, **dkw)
    dkw["workspace"] = torch.empty(dws_bytes, dtype=torch.uint8, device=dev) if dws_bytes else False

    # verifier tokens for every pooled context set (seeded input; depends on the drafted trees)
    ver_np = np.empty((pool, B, N + 1), np.int32)
    kp_sum, nodes_sum, matched = 0, 0, 0
    for i in range(pool):
        rest.rest_draft(ds, d_ctx[i], d_ctx_len, out=tree, **dkw)
        torch.cuda.synchronize()
        tk, pr, nn = tree.tokens.cpu().numpy(), tree.parents.cpu().numpy(), tree.n_nodes.cpu().numpy()
        ver_np[i] = datagen.make_verifier_tokens(w.seed + i, tk, pr, nn, w.vocab)
        rng = tree.match_range.cpu().numpy()
        kp_sum += int(np.minimum(rng[:, 1] - rng[:, 0], w.K).sum())
        nodes_sum += int(nn.sum())
        matched += int((nn > 0).sum())
    d_ver = torch.from_numpy(ver_np).to(dev)
    kp_mean = kp_sum / (pool * B)

    def buf_of(j, layer):
        return (j * layers + layer) % nbuf

    def attn_calls(j):
        for layer in range(layers):
            bi = buf_of(j, layer)
            rest.rest_tree_attention(q_all[layer], ks[bi], vs[bi], d_kv_len, tree.mask, scale,
                                     max_kv=L + N, out=out_all[layer], workspace=ws)

    def draft_calls(j):
        rest.rest_draft(ds, d_ctx[j], d_ctx_len, out=tree, **dkw)

    def accept_calls(j):
        rest.rest_accept(tree.tokens, tree.parents, tree.n_nodes, d_ver[j], w.m, out=acc)

    def step_calls(j):
        draft_calls(j)
        attn_calls(j)
        accept_calls(j)

    def capture(fn, j):
        """Records the library calls of fn(j) into a CUDA graph (the launch-bound loop is
        replayed from the graph; the kernels are the library's own).  Returns the graph and
        the number of kernel launches it holds."""
        gr = torch.cuda.CUDAGraph()
        n0 = rest.launch_count()
        with torch.cuda.graph(gr):
            fn(j)
        return gr, rest.launch_count() - n0

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, iters):
        """Seconds for `iters` calls of fn(i), CUDA events on the launching stream, max over ranks."""
        stream = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for i in range(iters):
            fn(i)
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1) / 1e3, dist, dev)

    for j in range(3):          # plain calls first (also sets kernel attributes before capture)
        step_calls(j)
    torch.cuda.synchronize()
    step_graphs, launches_per_step = [], 0
    for j in range(pool):
        gr, launches_per_step = capture(step_calls, j)
        step_graphs.append(gr)
    warmup = max(args.warmup, 3)
    for i in range(warmup):
        step_graphs[i % pool].replay()
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    if rank == 0:
        sampler.start()
    sec = timed(lambda i: step_graphs[i % pool].replay(), args.steps)
    launches = launches_per_step * args.steps

    # ---- per-part timings (same buffers, each part replayed from its own graph; each part
    # is looped for about a second so that short parts are not decided by a few replays) ----
    est = sec / args.steps

    def part_iters(share):
        return int(min(20000, max(20, 1.0 / max(est * share, 2e-6))))
    draft_graphs = [capture(draft_calls, j)[0] for j in range(pool)]
    attn_graphs = [capture(attn_calls, j)[0] for j in range(min(pool, 4))]
    accept_graphs = [capture(accept_calls, j)[0] for j in range(pool)]
    for i in range(3):
        draft_graphs[i].replay(); attn_graphs[i % len(attn_graphs)].replay(); accept_graphs[i].replay()
    n_d, n_a, n_c = part_iters(0.1), part_iters(0.9), part_iters(0.01)
    t_draft = timed(lambda i: draft_graphs[i % pool].replay(), n_d) / n_d
    t_attn = timed(lambda i: attn_graphs[i % len(attn_graphs)].replay(), n_a) / (n_a * layers)
    t_accept = timed(lambda i: accept_graphs[i % pool].replay(), n_c) / n_c
    del draft_graphs, attn_graphs, accept_graphs
    long_run = None
    if sec < 1.0:               # the K timed steps took under a second: a longer run beside them
        n_long = int(min(20000, max(args.steps, math.ceil(1.2 / est))))
        sec_long = timed(lambda i: step_graphs[i % pool].replay(), n_long)
        long_run = {"steps": n_long, "ms_per_step": sec_long / n_long * 1e3,
                    "value": whole_job_throughput(B, n_long, world, sec_long)}

    # ---- end to end: host buffers, copies inside the timed region ---------------------------
    # The caller fills pinned host buffers (context, verifier tokens, per-layer queries), one
    # graph replay copies them in, runs the step and copies the results out, then the host waits.
    h_ctx = torch.empty((B, Lc), dtype=torch.int32).pin_memory()
    h_ver = torch.empty((B, N + 1), dtype=torch.int32).pin_memory()
    # queries and outputs of all layers in one buffer each, copied in groups of layers: fewer
    # cross-stream dependencies in the graph than one copy per layer
    group = min(4, layers)
    h_q = q_all.cpu().pin_memory()
    h_out = torch.empty((layers, B, N, H, D), dtype=torch.bfloat16).pin_memory()
    h_tree = {k: torch.empty_like(getattr(tree, k), device="cpu").pin_memory()
              for k in ("tokens", "parents", "depth", "pos_ids", "mask", "n_nodes", "match_n")}
    h_acc = [torch.empty_like(a, device="cpu").pin_memory() for a in acc]
    s_ctx = torch.empty((B, Lc), dtype=torch.int32, device=dev)
    s_ver = torch.empty((B, N + 1), dtype=torch.int32, device=dev)
    h2d = s_ctx.numel() * 4 + s_ver.numel() * 4 + q_all.numel() * 2
    d2h = sum(t.numel() * t.element_size() for t in h_tree.values()) + \
        sum(t.numel() * 4 for t in h_acc) + h_out.numel() * 2
    ctx_t, ver_t = torch.from_numpy(ctx_np), torch.from_numpy(ver_np)

    # Two copy streams run beside the compute stream inside the graph: all inputs go in on one
    # (a layer's attention waits only for its own group of queries), each group of layers'
    # outputs goes out on the other as soon as the group is done.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    # A single layer over a large batch has no second layer to hide its copies behind: the batch
    # is then cut into chunks of contexts (one attention call each), so that the queries of
    # chunk i + 1 arrive and the outputs of chunk i - 1 leave while chunk i is computed.
    # The first chunk's queries and the last chunk's outputs cannot hide behind anything: those two
    # chunks are small (an eighth of the batch each), the two in between large.
    if layers == 1 and B >= 64:
        edges = [0, B // 8, B // 2, B - B // 8, B]
        bounds = list(zip(edges[:-1], edges[1:]))
    else:
        bounds = [(0, B)]
    if args.e2e_chunks:                      # explicit chunk sizes (contexts), e.g. 16,48,48,16
        sizes = [int(x) for x in args.e2e_chunks.split(",")]
        if sum(sizes) != B or min(sizes) < 1:
            raise SystemExit("--e2e-chunks must be positive sizes that add up to the contexts per step")
        edges = np.cumsum([0] + sizes).tolist()
        bounds = list(zip(edges[:-1], edges[1:]))

    def e2e_calls(_):
        main = torch.cuda.current_stream()
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        q_ready = {}
        with torch.cuda.stream(s_in):
            s_ctx.copy_(h_ctx, non_blocking=True)
            s_ver.copy_(h_ver, non_blocking=True)
            in_ready = torch.cuda.Event()
            in_ready.record(s_in)
            for l0 in range(0, layers, group):
                for c, (b0, b1) in enumerate(bounds):
                    q_all[l0:l0 + group, b0:b1].copy_(h_q[l0:l0 + group, b0:b1], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(s_in)
                    q_ready[(l0 // group, c)] = ev
        main.wait_event(in_ready)
        rest.rest_draft(ds, s_ctx, d_ctx_len, out=tree, **dkw)
        for layer in range(layers):
            bi = buf_of(0, layer)
            for c, (b0, b1) in enumerate(bounds):
                if layer % group == 0:
                    main.wait_event(q_ready[(layer // group, c)])
                rest.rest_tree_attention(q_all[layer, b0:b1], ks[bi][b0:b1], vs[bi][b0:b1], d_kv_len[b0:b1],
                                         tree.mask[b0:b1], scale, max_kv=L + N, out=out_all[layer, b0:b1],
                                         workspace=ws)
                if layer % group == group - 1 or layer == layers - 1:
                    l0 = layer - layer % group
                    done = torch.cuda.Event()
                    done.record(main)
                    s_out.wait_event(done)
                    with torch.cuda.stream(s_out):
                        h_out[l0:layer + 1, b0:b1].copy_(out_all[l0:layer + 1, b0:b1], non_blocking=True)
        rest.rest_accept(tree.tokens, tree.parents, tree.n_nodes, s_ver, w.m, out=acc)
        for k, t in h_tree.items():
            t.copy_(getattr(tree, k), non_blocking=True)
        for hacc, dacc in zip(h_acc, acc):
            hacc.copy_(dacc, non_blocking=True)
        main.wait_stream(s_in)
        main.wait_stream(s_out)

    e2e_graph, _ = capture(e2e_calls, 0)

    def e2e_step(i):
        j = i % pool
        h_ctx.copy_(ctx_t[j])           # host-side fill of the pinned input buffers
        h_ver.copy_(ver_t[j])
        e2e_graph.replay()
        torch.cuda.current_stream().synchronize()   # accepted tokens are needed before the next step

    for i in range(3):
        e2e_step(i)
    n_e2e = max(50, args.steps)
    t_e2e = timed(e2e_step, n_e2e) / n_e2e
    clocks = sampler.stop() if rank == 0 else None

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- rank 0: the line ---------------------------------------------------------------------
    a_bytes = attention_bytes(B, H, H, N, D, L)
    kernel = attention_kernel_name(B, H, H, N)
    per_unit = NCU_TRAFFIC_PER_UNIT.get((kernel, N, L))
    d_bytes = draft_bytes(w.n_tokens, w.sa_bytes, w.n_min, w.n_max, kp_mean, w.m, N) * B
    l2_policy = ("inputs larger than L2: %d KV buffer(s) of %.2f GB used round robin by the layers "
                 "(%.2f GB read per step), contexts rotate over %d sets"
                 % (nbuf, layer_bytes / 1e9, layers * a_bytes / 1e9, pool))
    del step_graphs, e2e_graph, ks, vs, q_all, out_all, h_q, h_out
    torch.cuda.empty_cache()
    read_ns = rest.dependent_read_latency_ns(device=dev)
    chain = draft_chain_reads(w.n_tokens, kp_mean)
    a_frac = a_bytes / t_attn / 1e9 / peak
    d_frac = d_bytes / t_draft / 1e9 / peak
    line = {
        "metric": METRIC, "value": whole_job_throughput(B, args.steps, world, sec), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": sec / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": workload_config(w, args, {"l2_policy": l2_policy}),
        "setup": setup, "long_run": long_run,
        "parts": {"draft_us": t_draft * 1e6, "draft_trees_per_s": world * B / t_draft,
                  "tree_attn_us_per_layer": t_attn * 1e6, "accept_us": t_accept * 1e6,
                  "mean_candidates_per_context": kp_mean,
                  "mean_nodes_per_tree": nodes_sum / (pool * B),
                  "contexts_with_a_match": matched / (pool * B)},
        "roofline": {"kernel": kernel + ", one layer", "bound": "hbm",
                     "achieved": a_bytes / t_attn / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": a_frac, "peak_kind": "of " + peak_kind,
                     "frac_of_nominal_8TBs": a_bytes / t_attn / 1e9 / 8000.0,
                     "algorithmic_bytes_per_launch": a_bytes, "target_50pct_met": bool(a_frac >= 0.5),
                     "traffic": None if per_unit is None or args.n_tokens is not None else per_unit * B * H,
                     "traffic_source": None if per_unit is None else
                     "small-case ncu capture of the same kernel and shape (profiles/), scaled by "
                     "the (context, head) units of this launch"},
        "roofline_draft": {"kernel": "rest_draft_kernel", "bound": "hbm (latency-bound at small B)",
                           "achieved": d_bytes / t_draft / 1e9, "peak": peak, "unit": "GB/s",
                           "frac": d_frac, "target_50pct_met": bool(d_frac >= 0.5),
                           "algorithmic_bytes_per_launch": d_bytes,
                           "sector_granular_bytes_per_launch": draft_sector_bytes(
                               w.n_tokens, w.sa_bytes, w.n_min, w.n_max, kp_mean, w.m, N) * B,
                           "traffic": None if w.name not in NCU_DRAFT_TRAFFIC_PER_ROW or args.n_tokens is not None
                           else NCU_DRAFT_TRAFFIC_PER_ROW[w.name] * kp_mean * B,
                           "traffic_source": "ncu capture of the same kernel on the same recipe at 100 M tokens "
                                             "(profiles/), scaled by the candidate rows of this launch",
                           "dependent_read_ns": read_ns, "dependent_reads_on_critical_path": chain,
                           "latency_floor_us": chain * read_ns / 1e3,
                           "frac_of_latency_floor": chain * read_ns / 1e3 / (t_draft * 1e6)},
        "e2e": {"value": world * B / t_e2e, "unit": UNIT, "ms_per_step": t_e2e * 1e3, "steps": n_e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "device_error_flags": rest.device_error_flags(),
        "clocks": clocks,
    }
    headline_row = {"workload": w.name, "datastore_tokens": w.n_tokens,
                    "draft": {"B": B, "us_per_call": t_draft * 1e6, "trees_per_s": B / t_draft,
                              "mean_candidates": kp_mean, "frac": d_frac,
                              "target_50pct_met": bool(d_frac >= 0.5), "measured": "inside the step's buffers"},
                    "attention": {"B": B, "kernel": kernel, "us_per_layer": t_attn * 1e6, "frac": a_frac,
                                  "frac_of_nominal_8TBs": a_bytes / t_attn / 1e9 / 8000.0,
                                  "target_50pct_met": bool(a_frac >= 0.5)}}
    if world == 1 and not args.no_workloads:
        line["workloads"], line["sweeps"] = other_workloads(rest, torch, dev, w, T, ds, headline_row,
                                                            peak, read_ns)
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        sa = d_sa.cpu().numpy()
        per_step, parts = oracle_step_sample(w, T, sa, ctx_np.reshape(pool * B, Lc), min(pool * B, 32),
                                             max(1, (B + 31) // 32) if B * H > 32 else 1, w.seed)
        line["cpu_baseline"] = {"value": B / per_step, "unit": UNIT, "cores": oracle.threads(),
                                "kind": "oracle", **parts}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def other_workloads(rest, torch, dev, headline, headline_T, headline_ds, headline_row, peak, read_ns):
    """Draft and tree-attention timings of all five workloads (the headline's own row comes
    from its step), then the sweeps: retrieval time against the datastore size (the shape of
    the paper's datastore-size table) and against the longest suffix length (its n_max figure)."""
    rows, sweeps = [], {"datastore_size": [], "n_max": []}
    keep_tokens = {}

    def fits(n_tokens, sa_bytes, extra=0):
        free, _ = torch.cuda.mem_get_info()
        need = n_tokens * (4 + sa_bytes) + rest.lib().rest_suffix_array_workspace_bytes(n_tokens) + extra
        return free > need + (2 << 30)

    for name, w0 in datagen.WORKLOADS.items():
        if name == headline.name:
            rows.append(headline_row)
            continue
        w, note = w0, None
        if w.n_tokens > 0x7FFFFFFF and rest.lib().rest_suffix_array_workspace_bytes(w.n_tokens) == 0:
            w = w0.scaled(n_tokens=1_000_000_000)
            note = ("stand-in: the recipe and the int64 suffix array of this workload at 1 B tokens "
                    "(the device builder takes up to 2^31 - 1 tokens)")
        row = {"workload": name, "datastore_tokens": w.n_tokens, "datastore_tokens_of_workload": w0.n_tokens}
        if note:
            row["note"] = note
        if fits(w.n_tokens, w.sa_bytes):
            T, d_T, d_sa, ds, setup = device_datastore(rest, torch, w, dev)
            row["setup"] = setup
            row["draft"] = time_draft(rest, torch, ds, w, T, w.B, dev, peak=peak, read_ns=read_ns)
            if name == "single_stream":      # the suffix-length sweep runs on this datastore
                for n_max in (2, 3, 4, 6, 8, 12, 16):
                    r = time_draft(rest, torch, ds, w, T, 256, dev, n_max=n_max, peak=peak)
                    sweeps["n_max"].append({k: r[k] for k in ("n_max", "B", "us_per_call", "trees_per_s",
                                                              "mean_candidates", "mean_nodes",
                                                              "mean_matched_length", "contexts_with_a_match")})
                sweeps["n_max_workload"] = "single_stream recipe, %d tokens, B = 256" % w.n_tokens
            if name == "batched":
                keep_tokens["batched"] = T
                for B in (1, 256):
                    r = time_draft(rest, torch, ds, w, T, B, dev, peak=peak)
                    sweeps["datastore_size"].append({"datastore_tokens": w.n_tokens, **setup, **{
                        k: r[k] for k in ("B", "us_per_call", "trees_per_s", "mean_candidates",
                                          "contexts_with_a_match", "mean_matched_length")}})
            ds.close()
            del ds, d_T, d_sa
            torch.cuda.empty_cache()
        else:
            row["draft"] = None
            row["note"] = "not enough free device memory for this datastore"
        row["attention"] = time_attention(rest, torch, w0, dev, peak=peak)
        rows.append(row)

    # the largest tree the library takes (N = 256: two 128-row blocks per head) on the stress shape
    w256 = dataclasses.replace(datagen.WORKLOADS["stress"], N=256)
    rows.append({"workload": "stress shape with N = 256 draft rows (attention only)",
                 "attention": time_attention(rest, torch, w256, dev, peak=peak)})

    # datastore-size sweep on the batched recipe: shorter streams are prefixes of the longest one
    wb = datagen.WORKLOADS["batched"]
    Tb = keep_tokens.get("batched")
    for n_tok in (1_000_000, 10_000_000, 100_000_000):
        w = wb.scaled(n_tokens=n_tok)
        T, d_T, d_sa, ds, setup = device_datastore(rest, torch, w, dev, tokens=Tb)
        for B in (1, 256):
            r = time_draft(rest, torch, ds, w, T, B, dev, peak=peak)
            sweeps["datastore_size"].append({"datastore_tokens": n_tok, **setup, **{
                k: r[k] for k in ("B", "us_per_call", "trees_per_s", "mean_candidates",
                                  "contexts_with_a_match", "mean_matched_length")}})
        ds.close()
        del ds, d_T, d_sa
        torch.cuda.empty_cache()
    sweeps["datastore_size"].sort(key=lambda r: (r["datastore_tokens"], r["B"]))
    sweeps["datastore_size_workload"] = "batched recipe (order 3, Zipf 1.1), K = 5000, m = 10, N = 64"
    return rows, sweeps


def run_part(args):
    """One call alone, on workload --workload (default stress), possibly reduced: the draft over a
    datastore of --n-tokens tokens with --batch contexts, or the attention layer with its batch
    cut to --max-gb of K/V.  Prints one JSON record."""
    import torch
    import paper_2311_08252_b200 as rest
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peaks()
    w = datagen.WORKLOADS["stress" if args.workload == "auto" else args.workload]
    if args.n_tokens is not None:
        w = w.scaled(n_tokens=args.n_tokens)
    if args.part == "draft":
        T, d_T, d_sa, ds, setup = device_datastore(rest, torch, w, dev)
        rec = time_draft(rest, torch, ds, w, T, args.batch or w.B, dev, iters=args.iters, peak=peak,
                         cold=not args.warm_l2)
        rec.update(setup)
    else:
        rec = time_attention(rest, torch, w, dev, iters=args.iters, peak=peak, budget_gb=args.max_gb)
    rec.update({"part": args.part, "workload": w.name, "datastore_tokens": w.n_tokens, "peak_gbs": peak,
                "peak_kind": peak_kind, "device_error_flags": rest.device_error_flags()})
    print(json.dumps(rec))


def spawn_ranks(args):
    """`bench.py --gpus N` started plainly (no launcher in the environment): start the N ranks
    through torch.distributed.run and pass their output through."""
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.part != "step":
        run_part(args)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
