#!/usr/bin/env python
"""Benchmark of one REST decoding step's hot path on B200: rest_draft -> rest_tree_attention
for every layer -> rest_accept, on the seeded "single_stream" workload (100M-token code-like
datastore, one 2048-token context, K=5000, m=10, N=64; 32 layers of 32 heads x 128 over a
2048-token bf16 KV cache).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is whole-path draft trees per second with all inputs resident
in HBM; `e2e` is the same with host<->device copies of the step's inputs and results inside
the timed region.  `--impl reference` times the CPU oracle (a deliberately plain program) on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
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
# dram__bytes_read.sum + dram__bytes_write.sum of one tree_attention_ws_kernel launch at the
# single_stream attention shape, from the ncu capture summarised under profiles/ (taken on the
# kernel as it stands); other shapes have no capture and report null.
NCU_TRAFFIC_BYTES = {("single_stream", "tree_attention_ws_kernel"): 35_185_920}
UNIT = "trees/s"
N_CTX_POOL = 64          # distinct contexts rotated through the steps


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="single_stream", choices=list(datagen.WORKLOADS))
    ap.add_argument("--n-tokens", type=int, default=None,
                    help="override the datastore size (debugging only; changes the workload name)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def load_datastore(w):
    """Tokens and host-built suffix array; cached on local disk between runs (setup only)."""
    cache = os.environ.get("REST_B200_CACHE", os.path.join(tempfile.gettempdir(), "rest_b200_cache"))
    tag = f"{w.name}_{w.n_tokens}_{w.seed}_sa{w.sa_bytes}_v2"
    tp, sp = os.path.join(cache, tag + "_tok.npy"), os.path.join(cache, tag + "_sa.npy")
    try:
        if os.path.exists(tp) and os.path.exists(sp):
            T, sa = np.load(tp), np.load(sp)
            if T.size == w.n_tokens and sa.size == w.n_tokens:
                return T, sa, True
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
    return T, sa, False


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


def draft_chain_reads(n_tokens, mean_candidates):
    """Dependent global reads on the critical path of one draft: every 32-ary search round is a
    suffix-array read followed by the token read it points to; lower bound over the whole array,
    one galloping round plus the upper bound over the matched range, one gather round, and the
    final token read of the emitted nodes."""
    r_lower = math.ceil(math.log(max(n_tokens, 2)) / math.log(33))
    r_upper = 1 + math.ceil(math.log(max(mean_candidates, 2)) / math.log(33))
    return 2 * (r_lower + r_upper + 1) + 1


def oracle_step_sample(w, T, sa, ctxs, q, k, v, kv_len, n_ctx, scale):
    """Times the CPU oracle on a bounded sample of one step: n_ctx drafts and accepts, and one
    attention layer (all heads).  Returns per-step seconds extrapolated to all layers."""
    import oracle
    import torch
    Lc = ctxs.shape[1]
    t0 = time.perf_counter()
    d = oracle.draft(T, sa, w.vocab, ctxs[:n_ctx], np.full(n_ctx, Lc, np.int32),
                     K=w.K, m=w.m, N=w.N, n_max=w.n_max, n_min=w.n_min)
    t_draft = (time.perf_counter() - t0) / n_ctx
    ver = datagen.make_verifier_tokens(w.seed, d["tokens"], d["parents"], d["n_nodes"], w.vocab)
    t0 = time.perf_counter()
    oracle.accept(d["tokens"], d["parents"], d["n_nodes"], ver, w.m)
    t_accept = (time.perf_counter() - t0) / n_ctx
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    t0 = time.perf_counter()
    oracle.tree_attention(bits(q), bits(k), bits(v), kv_len, d["mask"][:q.shape[0]], scale)
    t_layer = time.perf_counter() - t0
    per_step = w.B * (t_draft + t_accept) + w.layers * t_layer
    return per_step, dict(t_draft_s=t_draft, t_accept_s=t_accept, t_attn_layer_s=t_layer)


def run_reference(args, w, rank, world):
    """The CPU oracle as it stands, on the host cores, on a bounded sample per step."""
    if rank != 0:
        return
    import oracle
    T, sa, _ = load_datastore(w)
    ctxs = datagen.make_contexts(w, T, B=N_CTX_POOL, Lc=w.Lc)
    q, k, v = datagen.make_qkv(w.seed, w.B, w.H, w.N, w.D, w.L + w.N)
    kv_len = np.full(w.B, w.L, np.int32)
    scale = 1.0 / math.sqrt(w.D)
    times = []
    for i in range(args.warmup + args.steps):
        per_step, parts = oracle_step_sample(w, T, sa, ctxs, q, k, v, kv_len, 8, scale)
        if i >= args.warmup:
            times.append(per_step)
    sec = float(np.mean(times))
    value = w.B / sec
    sample = ("per step: 8 drafts+accepts and 1 of %d attention layers (all %d heads) in fp64, "
              "extrapolated linearly to one full step" % (w.layers, w.H))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w, args):
    return {"workload": w.name + ("" if args.n_tokens is None else f"@{w.n_tokens}"),
            "datastore_tokens": w.n_tokens, "sa_bytes": w.sa_bytes, "contexts_per_step": w.B,
            "context_len": w.Lc, "K": w.K, "m": w.m, "N": w.N, "n_max": w.n_max, "n_min": w.n_min,
            "layers": w.layers, "heads": w.H, "head_dim": w.D, "kv_len": w.L,
            "l2_policy": "inputs larger than L2: every layer has its own KV buffer "
                         "(%.2f GB per step), contexts rotate over %d samples"
                         % (w.layers * attention_bytes(w.B, w.H, w.H, w.N, w.D, w.L) / 1e9, N_CTX_POOL),
            "parallelism": "contexts sharded over GPUs, datastore replicated, no collective"}


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = datagen.WORKLOADS[args.workload]
    if args.n_tokens is not None:
        w = w.scaled(n_tokens=args.n_tokens)
    if args.impl == "reference":
        run_reference(args, w, rank, world)
        return

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

    # ---- inputs (setup, untimed) -------------------------------------------------------
    # every rank generates the same seeded token stream and builds its own copy of the suffix
    # array on its GPU (the datastore is replicated; nothing is exchanged)
    T = datagen.make_tokens(w)
    d_T = torch.from_numpy(T).to(dev)
    d_sa = rest.rest_suffix_array_build(d_T, w.sa_bytes)
    sa = None
    ds = rest.Datastore(d_T, d_sa, w.vocab, validate=True)

    B, N, H, D, L, layers = w.B, w.N, w.H, w.D, w.L, w.layers
    pool = N_CTX_POOL
    # the global batch of every pooled step is world*B contexts; this rank owns one slice
    all_ctx = datagen.make_contexts(w, T, B=pool * B * world, Lc=w.Lc).reshape(pool, B * world, w.Lc)
    c0, c1 = shard_bounds(B * world, rank, world)
    ctx_np = np.ascontiguousarray(all_ctx[:, c0:c1])
    ctx_len_np = np.full(B, w.Lc, np.int32)
    d_ctx = torch.from_numpy(ctx_np).to(dev)
    d_ctx_len = torch.from_numpy(ctx_len_np).to(dev)
    scale = 1.0 / math.sqrt(D)
    qs, ks, vs, outs = [], [], [], []
    for layer in range(layers):
        q, k, v = datagen.make_qkv(w.seed * 1000 + layer + 100 * rank, B, H, N, D, L + N, device=dev)
        qs.append(q); ks.append(k); vs.append(v)
        outs.append(torch.empty((B, N, H, D), dtype=torch.bfloat16, device=dev))
    d_kv_len = torch.full((B,), L, dtype=torch.int32, device=dev)
    ws_bytes = rest.tree_attention_workspace_bytes(B, H, N, D, L + N)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
    tree = rest.alloc_draft_output(B, N, dev)
    acc = (torch.empty(B, dtype=torch.int32, device=dev),
           torch.empty((B, w.m), dtype=torch.int32, device=dev),
           torch.empty((B, w.m + 1), dtype=torch.int32, device=dev))
    dkw = dict(n_max=w.n_max, n_min=w.n_min, K=w.K, m=w.m, N=N)

    # verifier tokens for every pooled context (seeded input; depends on the drafted trees)
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

    def step_calls(j):
        rest.rest_draft(ds, d_ctx[j], d_ctx_len, out=tree, **dkw)
        for layer in range(layers):
            rest.rest_tree_attention(qs[layer], ks[layer], vs[layer], d_kv_len, tree.mask, scale,
                                     max_kv=L + N, out=outs[layer], workspace=ws)
        rest.rest_accept(tree.tokens, tree.parents, tree.n_nodes, d_ver[j], w.m, out=acc)

    def draft_calls(j):
        rest.rest_draft(ds, d_ctx[j], d_ctx_len, out=tree, **dkw)

    def attn_calls(_):
        for layer in range(layers):
            rest.rest_tree_attention(qs[layer], ks[layer], vs[layer], d_kv_len, tree.mask, scale,
                                     max_kv=L + N, out=outs[layer], workspace=ws)

    def accept_calls(j):
        rest.rest_accept(tree.tokens, tree.parents, tree.n_nodes, d_ver[j], w.m, out=acc)

    def capture(fn, j):
        """Records the library calls of fn(j) into a CUDA graph (the launch-bound loop is
        replayed from the graph; the kernels are the library's own).  Returns the graph and
        the number of kernel launches it holds."""
        g = torch.cuda.CUDAGraph()
        n0 = rest.launch_count()
        with torch.cuda.graph(g):
            fn(j)
        return g, rest.launch_count() - n0

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
        g, launches_per_step = capture(step_calls, j)
        step_graphs.append(g)
    for i in range(max(args.warmup, 3)):
        step_graphs[i % pool].replay()
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    if rank == 0:
        sampler.start()
    sec = timed(lambda i: step_graphs[i % pool].replay(), args.steps)
    launches = launches_per_step * args.steps

    # ---- per-part timings (same buffers, each part replayed from its own graph) ------------
    draft_graphs = [capture(draft_calls, j)[0] for j in range(pool)]
    attn_graph, _ = capture(attn_calls, 0)
    accept_graphs = [capture(accept_calls, j)[0] for j in range(pool)]
    n_part = max(args.steps, 3)
    for i in range(3):
        draft_graphs[i].replay(); attn_graph.replay(); accept_graphs[i].replay()
    t_draft = timed(lambda i: draft_graphs[i % pool].replay(), n_part) / n_part
    t_attn = timed(lambda i: attn_graph.replay(), n_part) / (n_part * layers)
    t_accept = timed(lambda i: accept_graphs[i % pool].replay(), n_part) / n_part

    # ---- end to end: host buffers, copies inside the timed region ---------------------------
    # The caller fills pinned host buffers (context, verifier tokens, per-layer queries), one
    # graph replay copies them in, runs the step and copies the results out, then the host waits.
    h_ctx = torch.empty((B, w.Lc), dtype=torch.int32).pin_memory()
    h_ver = torch.empty((B, N + 1), dtype=torch.int32).pin_memory()
    # queries and outputs of all layers in one buffer each, copied in groups of layers: fewer
    # cross-stream dependencies in the graph than one copy per layer
    group = 4
    q_all = torch.stack(qs)                                   # [layers, B, N, H, D] on the device
    out_all = torch.empty((layers, B, N, H, D), dtype=torch.bfloat16, device=dev)
    h_q = q_all.cpu().pin_memory()
    h_out = torch.empty((layers, B, N, H, D), dtype=torch.bfloat16).pin_memory()
    h_tree = {k: torch.empty_like(getattr(tree, k), device="cpu").pin_memory()
              for k in ("tokens", "parents", "depth", "pos_ids", "mask", "n_nodes", "match_n")}
    h_acc = [torch.empty_like(a, device="cpu").pin_memory() for a in acc]
    s_ctx = torch.empty((B, w.Lc), dtype=torch.int32, device=dev)
    s_ver = torch.empty((B, N + 1), dtype=torch.int32, device=dev)
    h2d = s_ctx.numel() * 4 + s_ver.numel() * 4 + sum(q.numel() * 2 for q in qs)
    d2h = sum(t.numel() * t.element_size() for t in h_tree.values()) + \
        sum(t.numel() * 4 for t in h_acc) + h_out.numel() * 2
    ctx_t, ver_t = torch.from_numpy(ctx_np), torch.from_numpy(ver_np)

    # Two copy streams run beside the compute stream inside the graph: all inputs go in on one
    # (a layer's attention waits only for its own group of queries), each group of layers'
    # outputs goes out on the other as soon as the group is done.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def e2e_calls(_):
        main = torch.cuda.current_stream()
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        q_ready = []
        with torch.cuda.stream(s_in):
            s_ctx.copy_(h_ctx, non_blocking=True)
            s_ver.copy_(h_ver, non_blocking=True)
            in_ready = torch.cuda.Event()
            in_ready.record(s_in)
            for l0 in range(0, layers, group):
                q_all[l0:l0 + group].copy_(h_q[l0:l0 + group], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(s_in)
                q_ready.append(ev)
        main.wait_event(in_ready)
        rest.rest_draft(ds, s_ctx, d_ctx_len, out=tree, **dkw)
        for layer in range(layers):
            if layer % group == 0:
                main.wait_event(q_ready[layer // group])
            rest.rest_tree_attention(q_all[layer], ks[layer], vs[layer], d_kv_len, tree.mask, scale,
                                     max_kv=L + N, out=out_all[layer], workspace=ws)
            if layer % group == group - 1 or layer == layers - 1:
                l0 = layer - layer % group
                done = torch.cuda.Event()
                done.record(main)
                s_out.wait_event(done)
                with torch.cuda.stream(s_out):
                    h_out[l0:layer + 1].copy_(out_all[l0:layer + 1], non_blocking=True)
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
    n_e2e = max(3, args.steps // 4)
    t_e2e = timed(e2e_step, n_e2e) / n_e2e
    clocks = sampler.stop() if rank == 0 else None

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    read_ns = rest.dependent_read_latency_ns(device=dev)
    chain = draft_chain_reads(w.n_tokens, kp_sum / (pool * B))
    a_bytes = attention_bytes(B, H, H, N, D, L)
    d_bytes = draft_bytes(w.n_tokens, w.sa_bytes, w.n_min, w.n_max, kp_sum / (pool * B), w.m, N) * B
    line = {
        "metric": METRIC, "value": whole_job_throughput(B, args.steps, world, sec), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": sec / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": workload_config(w, args),
        "parts": {"draft_us": t_draft * 1e6, "draft_trees_per_s": world * B / t_draft,
                  "tree_attn_us_per_layer": t_attn * 1e6, "accept_us": t_accept * 1e6,
                  "mean_candidates_per_context": kp_sum / (pool * B),
                  "mean_nodes_per_tree": nodes_sum / (pool * B),
                  "contexts_with_a_match": matched / (pool * B)},
        "roofline": {"kernel": "tree_attention_ws_kernel, one layer", "bound": "hbm",
                     "achieved": a_bytes / t_attn / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": a_bytes / t_attn / 1e9 / peak, "peak_kind": "of " + peak_kind,
                     "frac_of_nominal_8TBs": a_bytes / t_attn / 1e9 / 8000.0,
                     "algorithmic_bytes_per_launch": a_bytes,
                     "traffic": NCU_TRAFFIC_BYTES.get((w.name, "tree_attention_ws_kernel"))
                     if args.n_tokens is None else None},
        "roofline_draft": {"kernel": "rest_draft_kernel", "bound": "hbm (latency-bound at B=1)",
                           "achieved": d_bytes / t_draft / 1e9, "peak": peak, "unit": "GB/s",
                           "frac": d_bytes / t_draft / 1e9 / peak,
                           "algorithmic_bytes_per_launch": d_bytes,
                           "sector_granular_bytes_per_launch": draft_sector_bytes(
                               w.n_tokens, w.sa_bytes, w.n_min, w.n_max, kp_sum / (pool * B), w.m, N) * B,
                           "dependent_read_ns": read_ns, "dependent_reads_on_critical_path": chain,
                           "latency_floor_us": chain * read_ns / 1e3,
                           "frac_of_latency_floor": chain * read_ns / 1e3 / (t_draft * 1e6)},
        "e2e": {"value": world * B / t_e2e, "unit": UNIT, "ms_per_step": t_e2e * 1e3,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "device_error_flags": rest.device_error_flags(),
        "clocks": clocks,
    }
    if not args.no_cpu_baseline:
        import oracle
        if sa is None:
            sa = d_sa.cpu().numpy()
        q0, k0, v0 = qs[0].cpu(), ks[0].cpu(), vs[0].cpu()
        per_step, parts = oracle_step_sample(w, T, sa, ctx_np.reshape(pool * B, w.Lc), q0, k0, v0,
                                             np.full(B, L, np.int32), min(pool * B, 32), scale)
        line["cpu_baseline"] = {
            "value": B / per_step, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "32 drafts+accepts and 1 of %d attention layers (all %d heads, fp64), "
                      "extrapolated linearly to one step" % (layers, H), **parts}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
