"""Python binding of librest.so, the CUDA (sm_100a) hot path of one REST decoding step.

Argument marshalling only: every step runs in the library's kernels.  torch is used to own
device memory and to supply the current CUDA stream.  There is no CPU fallback: importing
works without the library, but every call raises if librest.so is missing or cannot load.

The four entry points mirror include/rest.h:
    rest_datastore_create / Datastore   Sec. 3.2, datastore = token stream + suffix array
    rest_draft                          Algorithms 1 and 2, breadth-first tree + mask
    rest_tree_attention                 Sec. 3.2, draft verification (tree attention)
    rest_accept                         Sec. 3.2, draft acceptance
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "librest.so")

REST_OK = 0
REST_SAMPLE_STRIDED = 0
REST_SAMPLE_FIRST_K = 1
REST_SEARCH_AUTO = 0
REST_SEARCH_SINGLE = 1
REST_SEARCH_BATCHED = 2
REST_DS_VALIDATE = 1
REST_DS_INDEX = 2

EXPORTS = (
    "rest_datastore_aux_bytes", "rest_datastore_create", "rest_datastore_create_shard",
    "rest_datastore_destroy", "rest_draft_workspace_bytes", "rest_draft",
    "rest_retrieve", "rest_gather_rows", "rest_draft_from_runs_workspace_bytes", "rest_draft_from_runs",
    "rest_tree_attention_workspace_bytes", "rest_tree_attention",
    "rest_tree_attention_static_scratch",
    "rest_device_error_flags", "rest_kv_commit", "rest_probe_dependent_reads",
    "rest_suffix_array_workspace_bytes", "rest_suffix_array_min_workspace_bytes",
    "rest_suffix_array_build", "rest_suffix_array_build_in_groups", "rest_suffix_array_build_full",
    "rest_suffix_array_append_workspace_bytes", "rest_suffix_array_append", "rest_tree_attention_plan",
    "rest_accept", "rest_status_string", "rest_last_cuda_error", "rest_launch_count",
)


class RestError(RuntimeError):
    pass


class _Params(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_max", "n_min", "K", "m", "N", "sample_mode",
                                              "search_path")]


_lib = None


def library_path() -> str:
    return _SO


def lib():
    """Loads librest.so; raises RestError when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_SO):
        raise RestError(f"{_SO} is missing: build it with `python -m paper_2311_08252_b200.build` "
                        "(there is no CPU fallback)")
    L = ctypes.CDLL(_SO)
    vp, i32, i64, u32, u64, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                                  ctypes.c_uint32, ctypes.c_uint64, ctypes.c_size_t)
    L.rest_datastore_aux_bytes.restype = sz
    L.rest_datastore_aux_bytes.argtypes = [u64, i32, u32]
    L.rest_datastore_create.restype = i32
    L.rest_datastore_create.argtypes = [vp, u64, vp, i32, u32, u32, vp, sz, vp,
                                        ctypes.POINTER(vp)]
    L.rest_datastore_create_shard.restype = i32
    L.rest_datastore_create_shard.argtypes = [vp, u64, vp, u64, i32, u32, u32, vp, sz, vp,
                                              ctypes.POINTER(vp)]
    L.rest_retrieve.restype = i32
    L.rest_retrieve.argtypes = [vp, ctypes.POINTER(_Params), vp, i64, vp, i32, vp, vp, vp, vp]
    L.rest_gather_rows.restype = i32
    L.rest_gather_rows.argtypes = [vp, ctypes.POINTER(_Params), vp, vp, vp, i32, i32, vp, vp, vp, vp]
    L.rest_draft_from_runs_workspace_bytes.restype = sz
    L.rest_draft_from_runs_workspace_bytes.argtypes = [i32, i32, i32]
    L.rest_draft_from_runs.restype = i32
    L.rest_draft_from_runs.argtypes = [ctypes.POINTER(_Params), vp, vp, vp, i32, i32, vp, i32] + [vp] * 8 + \
        [vp, sz, vp]
    L.rest_datastore_destroy.restype = None
    L.rest_datastore_destroy.argtypes = [vp]
    L.rest_draft_workspace_bytes.restype = sz
    L.rest_draft_workspace_bytes.argtypes = [ctypes.POINTER(_Params), i32]
    L.rest_draft.restype = i32
    L.rest_draft.argtypes = [vp, ctypes.POINTER(_Params), vp, i64, vp, i32] + [vp] * 10 + [vp, sz, vp]
    L.rest_tree_attention_workspace_bytes.restype = sz
    L.rest_tree_attention_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    L.rest_tree_attention.restype = i32
    L.rest_tree_attention.argtypes = [vp, vp, vp, ctypes.POINTER(i64), vp, vp, i32, i32, i32, i32,
                                      i32, i32, ctypes.c_float, vp, vp, vp, sz, vp]
    L.rest_tree_attention_static_scratch.restype = i32
    L.rest_tree_attention_static_scratch.argtypes = [vp, vp, vp, ctypes.POINTER(i64), vp, vp, i32,
                                                     i32, i32, i32, i32, i32, ctypes.c_float, vp,
                                                     vp, vp]
    L.rest_accept.restype = i32
    L.rest_accept.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp]
    L.rest_kv_commit.restype = i32
    L.rest_kv_commit.argtypes = [vp, vp, ctypes.POINTER(i64), vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
    L.rest_suffix_array_workspace_bytes.restype = sz
    L.rest_suffix_array_workspace_bytes.argtypes = [u64]
    L.rest_suffix_array_min_workspace_bytes.restype = sz
    L.rest_suffix_array_min_workspace_bytes.argtypes = [u64, u64]
    L.rest_suffix_array_build.restype = i32
    L.rest_suffix_array_build.argtypes = [vp, u64, i32, vp, vp, sz, vp]
    L.rest_suffix_array_append_workspace_bytes.restype = sz
    L.rest_suffix_array_append_workspace_bytes.argtypes = [u64]
    L.rest_suffix_array_append.restype = i32
    L.rest_suffix_array_append.argtypes = [vp, u64, u64, vp, i32, vp, vp, sz, vp]
    L.rest_suffix_array_build_full.restype = i32
    L.rest_suffix_array_build_full.argtypes = [vp, u64, i32, vp, vp, sz, vp]
    L.rest_suffix_array_build_in_groups.restype = i32
    L.rest_suffix_array_build_in_groups.argtypes = [vp, u64, i32, vp, u64, vp, sz, vp]
    L.rest_tree_attention_plan.restype = i32
    L.rest_tree_attention_plan.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(i32)]
    L.rest_probe_dependent_reads.restype = i32
    L.rest_probe_dependent_reads.argtypes = [vp, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, vp, vp]
    L.rest_device_error_flags.restype = i32
    L.rest_device_error_flags.argtypes = [ctypes.POINTER(u32)]
    L.rest_status_string.restype = ctypes.c_char_p
    L.rest_status_string.argtypes = [i32]
    L.rest_last_cuda_error.restype = ctypes.c_char_p
    L.rest_launch_count.restype = u64
    _lib = L
    return L


def _check(rc: int, what: str):
    if rc != REST_OK:
        L = lib()
        msg = L.rest_status_string(rc).decode()
        if rc == 4:
            msg += ": " + L.rest_last_cuda_error().decode()
        raise RestError(f"{what} failed: {msg} (status {rc})")


def _stream(stream=None) -> int:
    import torch
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _dev_i32(t, name):
    import torch
    if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
        raise RestError(f"{name} must be a contiguous int32 CUDA tensor")
    return t


def device_error_flags() -> int:
    """Reads and clears the device-side error bits (0 = no kernel ever gave up on a wait)."""
    v = ctypes.c_uint32(0)
    _check(lib().rest_device_error_flags(ctypes.byref(v)), "rest_device_error_flags")
    return int(v.value)


def launch_count() -> int:
    return int(lib().rest_launch_count())


class Datastore:
    """Handle over device-resident tokens int32[n] and suffix array int32[n] / int64[n].
    The tensors are borrowed: this object keeps references so they outlive the handle.
    index=True also builds the bucket index (token and token-pair ranges of the suffix array)
    that lets rest_draft start its searches inside a small range; results do not depend on it."""

    def __init__(self, tokens, sa, vocab: int, validate: bool = False, stream=None,
                 index: bool = True):
        import torch
        if not (tokens.is_cuda and tokens.dtype == torch.int32 and tokens.is_contiguous()):
            raise RestError("tokens must be a contiguous int32 CUDA tensor")
        if not (sa.is_cuda and sa.dtype in (torch.int32, torch.int64) and sa.is_contiguous()
                and 0 < sa.numel() <= tokens.numel()):
            raise RestError("sa must be a contiguous int32/int64 CUDA tensor, at most as long as tokens")
        self.tokens, self.sa, self.vocab = tokens, sa, int(vocab)
        self.n_tokens = tokens.numel()
        self.sa_bytes = sa.element_size()
        L = lib()
        aux, aux_bytes = None, 0
        flags = (REST_DS_VALIDATE if validate else 0) | (REST_DS_INDEX if index else 0)
        if flags:
            aux_bytes = L.rest_datastore_aux_bytes(self.n_tokens, self.sa_bytes, self.vocab)
            aux = torch.empty(aux_bytes, dtype=torch.uint8, device=tokens.device)
        h = ctypes.c_void_p()
        # a suffix array shorter than the token stream lists the positions of a shard's own range
        rc = L.rest_datastore_create_shard(tokens.data_ptr(), self.n_tokens, sa.data_ptr(), sa.numel(),
                                           self.sa_bytes, self.vocab, flags, _ptr(aux), aux_bytes,
                                           _stream(stream), ctypes.byref(h))
        _check(rc, "rest_datastore_create")
        self._h = h
        self._aux = aux if index else None      # the handle reads the index for its whole life

    def close(self):
        if getattr(self, "_h", None):
            lib().rest_datastore_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def rest_datastore_create(tokens, sa, vocab, validate=False, stream=None, index=True) -> Datastore:
    return Datastore(tokens, sa, vocab, validate, stream, index)


@dataclass
class DraftOutput:
    tokens: "object"
    parents: "object"
    depth: "object"
    pos_ids: "object"
    mask: "object"
    n_nodes: "object"
    match_n: "object"
    match_range: "object"
    node_count: "object"
    status: "object"


def alloc_draft_output(B: int, N: int, device) -> DraftOutput:
    import torch
    i32 = dict(dtype=torch.int32, device=device)
    Wm = (N + 31) // 32
    return DraftOutput(
        torch.empty((B, N), **i32), torch.empty((B, N), **i32), torch.empty((B, N), **i32),
        torch.empty((B, N), **i32), torch.empty((B, N, Wm), **i32), torch.empty(B, **i32),
        torch.empty(B, **i32), torch.empty((B, 2), dtype=torch.int64, device=device),
        torch.empty((B, N), **i32), torch.empty(B, **i32))


def draft_workspace_bytes(B: int, n_max=16, n_min=2, K=5000, m=10, N=64,
                          sample_mode=REST_SAMPLE_STRIDED, search=REST_SEARCH_AUTO) -> int:
    """Scratch bytes rest_draft can use for a call of B contexts on the current device (0 when
    a scratch would not make the call faster)."""
    prm = _Params(n_max, n_min, K, m, N, sample_mode, search)
    return int(lib().rest_draft_workspace_bytes(ctypes.byref(prm), B))


def rest_draft(ds: Datastore, ctx, ctx_len, n_max=16, n_min=2, K=5000, m=10, N=64,
               sample_mode=REST_SAMPLE_STRIDED, out: DraftOutput | None = None, stream=None,
               search=REST_SEARCH_AUTO, workspace=None) -> DraftOutput:
    """Draft trees for contexts ctx int32[B, Lc] (row b holds ctx_len[b] tokens).  The mask
    tensor is int32 storage of the uint32 words.  `search` (REST_SEARCH_*) picks the
    single-context or the batched path; the results do not depend on it.  `workspace`: a uint8
    CUDA tensor of rest_draft_workspace_bytes() bytes, None to allocate one when the library
    asks for it, False to pass none (the batched path then runs as a single launch)."""
    L = lib()
    _dev_i32(ctx_len, "ctx_len")
    import torch
    if not (ctx.is_cuda and ctx.dtype == torch.int32 and ctx.dim() == 2 and ctx.stride(1) == 1):
        raise RestError("ctx must be an int32 CUDA tensor [B, Lc] with contiguous rows")
    B = ctx.shape[0]
    if out is None:
        out = alloc_draft_output(B, N, ctx.device)
    prm = _Params(n_max, n_min, K, m, N, sample_mode, search)
    ws_ptr, ws_bytes = 0, 0
    if workspace is None:
        need = L.rest_draft_workspace_bytes(ctypes.byref(prm), B)
        if need:
            workspace = torch.empty(need, dtype=torch.uint8, device=ctx.device)
    if workspace is not None and workspace is not False:
        ws_ptr, ws_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    rc = L.rest_draft(ds._h, ctypes.byref(prm), ctx.data_ptr(), ctx.stride(0), ctx_len.data_ptr(), B,
                      out.tokens.data_ptr(), out.parents.data_ptr(), out.depth.data_ptr(),
                      out.pos_ids.data_ptr(), out.mask.data_ptr(), out.n_nodes.data_ptr(),
                      out.match_n.data_ptr(), out.match_range.data_ptr(), _ptr(out.node_count),
                      out.status.data_ptr(), ws_ptr, ws_bytes, _stream(stream))
    _check(rc, "rest_draft")
    return out


def rest_retrieve(ds: Datastore, ctx, ctx_len, n_max=16, n_min=2, stream=None):
    """Algorithm 1 alone: returns (match_n int32[B], match_range int64[B,2], status int32[B])."""
    import torch
    L = lib()
    _dev_i32(ctx_len, "ctx_len")
    if not (ctx.is_cuda and ctx.dtype == torch.int32 and ctx.dim() == 2 and ctx.stride(1) == 1):
        raise RestError("ctx must be an int32 CUDA tensor [B, Lc] with contiguous rows")
    B = ctx.shape[0]
    match_n = torch.empty(B, dtype=torch.int32, device=ctx.device)
    match_range = torch.empty((B, 2), dtype=torch.int64, device=ctx.device)
    status = torch.empty(B, dtype=torch.int32, device=ctx.device)
    prm = _Params(n_max, n_min, 1, 1, 1, 0, 0)
    _check(L.rest_retrieve(ds._h, ctypes.byref(prm), ctx.data_ptr(), ctx.stride(0), ctx_len.data_ptr(), B,
                           match_n.data_ptr(), match_range.data_ptr(), status.data_ptr(), _stream(stream)),
           "rest_retrieve")
    return match_n, match_range, status


def rest_gather_rows(ds: Datastore, match_n, match_range, take, Kr: int, m=10,
                     sample_mode=REST_SAMPLE_STRIDED, status=None, stream=None):
    """The take[b] sampled candidate rows of every context's matched range: returns
    (rows int32[B,Kr,m], row_len int32[B,Kr], status int32[B])."""
    import torch
    L = lib()
    for t, nm in ((match_n, "match_n"), (take, "take")):
        _dev_i32(t, nm)
    B = match_n.shape[0]
    rows = torch.empty((B, Kr, m), dtype=torch.int32, device=match_n.device)
    row_len = torch.empty((B, Kr), dtype=torch.int32, device=match_n.device)
    if status is None:
        status = torch.zeros(B, dtype=torch.int32, device=match_n.device)
    prm = _Params(16, 2, Kr, m, 1, sample_mode, 0)
    _check(L.rest_gather_rows(ds._h, ctypes.byref(prm), match_n.data_ptr(), match_range.data_ptr(),
                              take.data_ptr(), B, Kr, rows.data_ptr(), row_len.data_ptr(),
                              status.data_ptr(), _stream(stream)), "rest_gather_rows")
    return rows, row_len, status


def rest_draft_from_runs(rows, row_len, run_rows, ctx_len, m=None, N=64, out: DraftOutput | None = None,
                         stream=None) -> DraftOutput:
    """Trees from candidate rows handed in as sorted runs: rows int32[B,R,Kr,m], row_len
    int32[B,R,Kr], run_rows int32[B,R].  match_n / match_range of the result are not written."""
    import torch
    L = lib()
    for t, nm in ((rows, "rows"), (row_len, "row_len"), (run_rows, "run_rows"), (ctx_len, "ctx_len")):
        _dev_i32(t, nm)
    B, R, Kr, mm = rows.shape
    m = mm if m is None else m
    if m != mm or row_len.shape != (B, R, Kr) or run_rows.shape != (B, R):
        raise RestError("rows [B,R,Kr,m], row_len [B,R,Kr] and run_rows [B,R] do not fit together")
    if out is None:
        out = alloc_draft_output(B, N, rows.device)
    ws_bytes = L.rest_draft_from_runs_workspace_bytes(B, R, Kr)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=rows.device)
    prm = _Params(16, 2, R * Kr, m, N, 0, 0)
    _check(L.rest_draft_from_runs(ctypes.byref(prm), rows.data_ptr(), row_len.data_ptr(), run_rows.data_ptr(),
                                  R, Kr, ctx_len.data_ptr(), B, out.tokens.data_ptr(), out.parents.data_ptr(),
                                  out.depth.data_ptr(), out.pos_ids.data_ptr(), out.mask.data_ptr(),
                                  out.n_nodes.data_ptr(), _ptr(out.node_count), out.status.data_ptr(),
                                  ws.data_ptr(), ws_bytes, _stream(stream)), "rest_draft_from_runs")
    return out


def tree_attention_workspace_bytes(B, H, N, D, max_kv) -> int:
    return int(lib().rest_tree_attention_workspace_bytes(B, H, N, D, max_kv))


def rest_tree_attention(q, k, v, kv_len, mask, scale, max_kv=None, out=None, lse=None,
                        workspace=None, stream=None):
    """q bf16 [B,N,H,D]; k, v bf16 [B,H_kv,Lcap,D] (tree rows at kv_len[b]..kv_len[b]+N-1);
    kv_len int32[B]; mask int32/uint32 words [B,N,ceil(N/32)].  Returns out bf16 [B,N,H,D]."""
    import torch
    L = lib()
    B, N, H, D = q.shape
    H_kv, Lcap = k.shape[1], k.shape[2]
    for t, nm in ((q, "q"), (k, "k"), (v, "v")):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.stride(-1) == 1):
            raise RestError(f"{nm} must be a bf16 CUDA tensor with a contiguous last dimension")
    if k.stride() != v.stride() or k.shape != v.shape:
        raise RestError("k and v must have the same shape and strides")
    _dev_i32(kv_len, "kv_len")
    if not (mask.is_cuda and mask.is_contiguous() and mask.element_size() == 4):
        raise RestError("mask must be a contiguous 32-bit CUDA tensor")
    if out is None:
        out = torch.empty((B, N, H, D), dtype=torch.bfloat16, device=q.device)
    max_kv = Lcap if max_kv is None else int(max_kv)
    need = L.rest_tree_attention_workspace_bytes(B, H, N, D, max_kv)
    if need and (workspace is None or workspace.numel() * workspace.element_size() < need):
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    strides = (ctypes.c_int64 * 9)(q.stride(0), q.stride(1), q.stride(2),
                                   k.stride(0), k.stride(1), k.stride(2),
                                   out.stride(0), out.stride(1), out.stride(2))
    rc = L.rest_tree_attention(q.data_ptr(), k.data_ptr(), v.data_ptr(), strides, kv_len.data_ptr(),
                               mask.data_ptr(), B, H, H_kv, N, D, max_kv, float(scale),
                               out.data_ptr(), _ptr(lse), _ptr(workspace),
                               0 if workspace is None else workspace.numel() * workspace.element_size(),
                               _stream(stream))
    _check(rc, "rest_tree_attention")
    return out


def rest_tree_attention_static_scratch(q, k, v, kv_len, mask, scale, out, max_kv=None, lse=None,
                                       stream=None):
    """rest_tree_attention without a workspace argument, for callers that must not allocate:
    the split partials go to a fixed 768 KiB array inside the library.  `out` (bf16 [B,N,H,D])
    is supplied by the caller, so this wrapper allocates nothing on the device either.
    Raises RestError (workspace too small) when the shape needs more than the fixed array.
    Calls share that array: do not let two of them overlap on the GPU."""
    L = lib()
    B, N, H, D = q.shape
    H_kv, Lcap = k.shape[1], k.shape[2]
    max_kv = Lcap if max_kv is None else int(max_kv)
    strides = (ctypes.c_int64 * 9)(q.stride(0), q.stride(1), q.stride(2),
                                   k.stride(0), k.stride(1), k.stride(2),
                                   out.stride(0), out.stride(1), out.stride(2))
    rc = L.rest_tree_attention_static_scratch(
        q.data_ptr(), k.data_ptr(), v.data_ptr(), strides, kv_len.data_ptr(), mask.data_ptr(),
        B, H, H_kv, N, D, max_kv, float(scale), out.data_ptr(), _ptr(lse), _stream(stream))
    _check(rc, "rest_tree_attention_static_scratch")
    return out


def rest_accept(tokens, parents, n_nodes, verifier_tokens, max_depth, out=None, stream=None):
    """Returns (accept_len int32[B], accept_nodes int32[B,max_depth], out_tokens int32[B,max_depth+1])."""
    import torch
    L = lib()
    for t, nm in ((tokens, "tokens"), (parents, "parents"), (n_nodes, "n_nodes"),
                  (verifier_tokens, "verifier_tokens")):
        _dev_i32(t, nm)
    B, N = tokens.shape
    if verifier_tokens.shape != (B, N + 1):
        raise RestError("verifier_tokens must be [B, N+1]")
    if out is None:
        i32 = dict(dtype=torch.int32, device=tokens.device)
        out = (torch.empty(B, **i32), torch.empty((B, max_depth), **i32),
               torch.empty((B, max_depth + 1), **i32))
    rc = L.rest_accept(tokens.data_ptr(), parents.data_ptr(), n_nodes.data_ptr(),
                       verifier_tokens.data_ptr(), B, N, max_depth, out[0].data_ptr(),
                       out[1].data_ptr(), out[2].data_ptr(), _stream(stream))
    _check(rc, "rest_accept")
    return out


def rest_kv_commit(k, v, kv_len, accept_nodes, accept_len, N, new_kv_len=None, stream=None):
    """Moves the K/V rows of the accepted draft nodes (tree slots kv_len[b] + node) to the
    contiguous slots kv_len[b] .. kv_len[b] + accept_len[b] - 1 of k, v bf16 [B,H_kv,Lcap,D], in
    place.  new_kv_len (optional int32[B]) receives kv_len + accept_len."""
    import torch
    L = lib()
    for t, nm in ((k, "k"), (v, "v")):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.stride(-1) == 1):
            raise RestError(f"{nm} must be a bf16 CUDA tensor with a contiguous last dimension")
    if k.stride() != v.stride() or k.shape != v.shape:
        raise RestError("k and v must have the same shape and strides")
    for t, nm in ((kv_len, "kv_len"), (accept_nodes, "accept_nodes"), (accept_len, "accept_len")):
        _dev_i32(t, nm)
    B, H_kv, _, D = k.shape
    max_depth = accept_nodes.shape[1]
    strides = (ctypes.c_int64 * 3)(k.stride(0), k.stride(1), k.stride(2))
    rc = L.rest_kv_commit(k.data_ptr(), v.data_ptr(), strides, kv_len.data_ptr(), _ptr(accept_nodes),
                          accept_len.data_ptr(), B, H_kv, N, D, max_depth, _ptr(new_kv_len),
                          _stream(stream))
    _check(rc, "rest_kv_commit")
    return new_kv_len


def dependent_read_latency_ns(table_bytes: int = 1 << 30, steps: int = 4096, device=None, seed: int = 1) -> float:
    """Nanoseconds per dependent DRAM read on this GPU: builds a random single-cycle table of
    table_bytes (much larger than L2) with torch, then one device thread chases it
    (rest_probe_dependent_reads).  A measurement aid for the draft path's latency floor."""
    import torch
    L = lib()
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    n = table_bytes // 4
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    perm = torch.randperm(n, generator=g, device=device)
    nxt = torch.empty(n, dtype=torch.int32, device=device)
    nxt[perm] = torch.roll(perm, -1).to(torch.int32)       # values < 2^31 for n <= 2^31
    del perm
    out = torch.zeros(2, dtype=torch.int64, device=device)
    best = None
    for rep in range(3):                                   # different stretches of the cycle
        start = int(nxt[rep * 7919 % n].item())
        torch.cuda.synchronize(device)
        _check(L.rest_probe_dependent_reads(nxt.data_ptr(), n, start, steps, out.data_ptr(), _stream(None)),
               "rest_probe_dependent_reads")
        torch.cuda.synchronize(device)
        ns = float(out[0].item()) / steps
        best = ns if best is None else min(best, ns)
    return best


def rest_suffix_array_build(tokens, sa_bytes: int = 4, stream=None, max_group: int | None = None,
                            full: bool = False):
    """Suffix array of the int32 CUDA tensor `tokens`, built on the device and ordered on the
    first 32 tokens of each suffix (ties by position).  Returns an int32 or int64 CUDA tensor.
    max_group: sort the stream in groups of first-token buckets of at most that many positions
    (the method for streams beyond 2^31 - 1 tokens), whatever its size.  full=True: the true
    suffix array (whole suffixes compared) instead of the order on 32 tokens."""
    import torch
    L = lib()
    _dev_i32(tokens, "tokens")
    n = tokens.numel()
    sa = torch.empty(n, dtype=torch.int32 if sa_bytes == 4 else torch.int64, device=tokens.device)
    if max_group is None:
        ws_bytes = L.rest_suffix_array_workspace_bytes(n)
    else:
        ws_bytes = L.rest_suffix_array_min_workspace_bytes(n, int(max_group))
    if ws_bytes == 0:
        raise RestError("rest_suffix_array_build: between 1 and 2^40 tokens are supported")
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=tokens.device)
    if full:
        rc = L.rest_suffix_array_build_full(tokens.data_ptr(), n, sa_bytes, sa.data_ptr(), ws.data_ptr(),
                                            ws_bytes, _stream(stream))
    elif max_group is None:
        rc = L.rest_suffix_array_build(tokens.data_ptr(), n, sa_bytes, sa.data_ptr(), ws.data_ptr(),
                                       ws_bytes, _stream(stream))
    else:
        rc = L.rest_suffix_array_build_in_groups(tokens.data_ptr(), n, sa_bytes, sa.data_ptr(), int(max_group),
                                                 ws.data_ptr(), ws_bytes, _stream(stream))
    _check(rc, "rest_suffix_array_build")
    # set-up call: wait here, so that the scratch can be released whatever stream was used
    torch.cuda.synchronize(tokens.device)
    return sa


def rest_suffix_array_append(tokens, sa_old, stream=None):
    """Suffix array of `tokens` (int32 CUDA tensor: the old stream followed by the appended
    tokens) from the array `sa_old` of its first sa_old.numel() tokens."""
    import torch
    L = lib()
    _dev_i32(tokens, "tokens")
    n, n_old = tokens.numel(), sa_old.numel()
    if not (sa_old.is_cuda and sa_old.dtype in (torch.int32, torch.int64) and sa_old.is_contiguous()) or n_old >= n:
        raise RestError("sa_old must be a contiguous int32/int64 CUDA tensor shorter than tokens")
    sa = torch.empty(n, dtype=sa_old.dtype, device=tokens.device)
    ws_bytes = L.rest_suffix_array_append_workspace_bytes(n - n_old)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=tokens.device)
    _check(L.rest_suffix_array_append(tokens.data_ptr(), n_old, n - n_old, _ptr(sa_old) if n_old else 0,
                                      sa_old.element_size(), sa.data_ptr(), ws.data_ptr(), ws_bytes,
                                      _stream(stream)), "rest_suffix_array_append")
    torch.cuda.synchronize(tokens.device)
    return sa


def tree_attention_plan(B, H, N, D, max_kv) -> dict:
    """Key ranges per (context, head), blocks per cluster, clusters per (context, head), and how
    many clusters of that size the current device runs at once."""
    out = (ctypes.c_int32 * 4)()
    _check(lib().rest_tree_attention_plan(B, H, N, D, max_kv, out), "rest_tree_attention_plan")
    return {"splits": out[0], "cluster": out[1], "clusters_per_unit": out[2], "capacity": out[3]}
