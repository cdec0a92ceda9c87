"""ctypes wrapper around the CPU oracle (rest_oracle.cpp).

Test infrastructure only: imported by tests/, the smoke check and the benchmark's
CPU-baseline leg.  The CUDA package never imports this module and this module never
imports the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "librest_oracle.so")
_SRC = os.path.join(_HERE, "rest_oracle.cpp")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-O2", "-fopenmp", "-std=c++17", "-shared", "-fPIC", _SRC, "-o", _SO])
    return _SO


class _Params(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_max", "n_min", "K", "m", "N", "sample_mode")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(lib().oracle_threads())


def _p(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def suffix_array(tokens: np.ndarray) -> np.ndarray:
    """True suffix array (int64) by comparison sort; small inputs only."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    sa = np.empty(tokens.size, dtype=np.int64)
    lib().oracle_suffix_array(_p(tokens), ctypes.c_int64(tokens.size), _p(sa))
    return sa


def retrieve(tokens, sa, ctx, n_max=16, n_min=2):
    """Algorithm 1 for one context: (match_n, lo, hi)."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    sa = np.ascontiguousarray(sa)
    ctx = np.ascontiguousarray(ctx, dtype=np.int32)
    mn = ctypes.c_int32(0)
    lo = ctypes.c_int64(0)
    hi = ctypes.c_int64(0)
    lib().oracle_retrieve(_p(tokens), ctypes.c_int64(tokens.size), _p(sa),
                          ctypes.c_int(sa.dtype.itemsize), _p(ctx), ctypes.c_int32(ctx.size),
                          ctypes.c_int(n_max), ctypes.c_int(n_min),
                          ctypes.byref(mn), ctypes.byref(lo), ctypes.byref(hi))
    return mn.value, lo.value, hi.value


def draft(tokens, sa, vocab, ctx, ctx_len, n_max=16, n_min=2, K=5000, m=10, N=64, sample_mode=0):
    """Draft trees for contexts ctx [B, Lc] (only the first ctx_len[b] tokens of a row count).

    Returns a dict of numpy arrays: tokens, parents, depth, pos_ids [B,N] int32,
    mask [B,N,ceil(N/32)] uint32, n_nodes, match_n, status [B] int32, match_range [B,2] int64,
    node_count [B,N] int32."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    sa = np.ascontiguousarray(sa)
    ctx = np.ascontiguousarray(ctx, dtype=np.int32)
    if ctx.ndim == 1:
        ctx = ctx[None, :]
    B = ctx.shape[0]
    ctx_len = np.ascontiguousarray(ctx_len, dtype=np.int32).reshape(B)
    Wm = (N + 31) // 32
    out = {
        "tokens": np.empty((B, N), np.int32), "parents": np.empty((B, N), np.int32),
        "depth": np.empty((B, N), np.int32), "pos_ids": np.empty((B, N), np.int32),
        "mask": np.empty((B, N, Wm), np.uint32), "n_nodes": np.empty(B, np.int32),
        "match_n": np.empty(B, np.int32), "match_range": np.empty((B, 2), np.int64),
        "node_count": np.empty((B, N), np.int32), "status": np.empty(B, np.int32),
    }
    prm = _Params(n_max, n_min, K, m, N, sample_mode)
    lib().oracle_draft(_p(tokens), ctypes.c_int64(tokens.size), _p(sa),
                       ctypes.c_int(sa.dtype.itemsize), ctypes.c_uint32(vocab), ctypes.byref(prm),
                       _p(ctx), ctypes.c_int64(ctx.shape[1]), _p(ctx_len), ctypes.c_int32(B),
                       _p(out["tokens"]), _p(out["parents"]), _p(out["depth"]), _p(out["pos_ids"]),
                       _p(out["mask"]), _p(out["n_nodes"]), _p(out["match_n"]),
                       _p(out["match_range"]), _p(out["node_count"]), _p(out["status"]))
    return out


def tree_attention(q_bits, k_bits, v_bits, kv_len, mask, scale, H_kv=None, want_lse=False):
    """fp64 tree attention.  q_bits [B,N,H,D], k_bits/v_bits [B,H_kv,Lcap,D]: uint16 arrays
    holding bf16 bit patterns (any strides with D contiguous); kv_len [B]; mask [B,N,Wm] uint32.
    Returns out [B,N,H,D] float64 (and lse [B,H,N] when asked)."""
    B, N, H, D = q_bits.shape
    H_kv = k_bits.shape[1] if H_kv is None else H_kv
    assert q_bits.dtype == np.uint16 and k_bits.dtype == np.uint16 and v_bits.dtype == np.uint16
    assert q_bits.strides[3] == 2 and k_bits.strides[3] == 2 and v_bits.strides == k_bits.strides
    strides = np.array([q_bits.strides[0] // 2, q_bits.strides[1] // 2, q_bits.strides[2] // 2,
                        k_bits.strides[0] // 2, k_bits.strides[1] // 2, k_bits.strides[2] // 2,
                        0, 0, 0], dtype=np.int64)
    kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    out = np.empty((B, N, H, D), np.float64)
    lse = np.empty((B, H, N), np.float64) if want_lse else None
    lib().oracle_tree_attention(_p(q_bits), _p(k_bits), _p(v_bits), _p(strides), _p(kv_len),
                                _p(mask), ctypes.c_int32(B), ctypes.c_int32(H),
                                ctypes.c_int32(H_kv), ctypes.c_int32(N), ctypes.c_int32(D),
                                ctypes.c_double(scale), _p(out), _p(lse))
    return (out, lse) if want_lse else out


def accept(tokens, parents, n_nodes, verifier_tokens, max_depth):
    """Draft acceptance: (accept_len [B], accept_nodes [B,max_depth], out_tokens [B,max_depth+1])."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    parents = np.ascontiguousarray(parents, dtype=np.int32)
    n_nodes = np.ascontiguousarray(n_nodes, dtype=np.int32)
    verifier_tokens = np.ascontiguousarray(verifier_tokens, dtype=np.int32)
    B, N = tokens.shape
    assert verifier_tokens.shape == (B, N + 1)
    al = np.empty(B, np.int32)
    an = np.empty((B, max_depth), np.int32)
    ot = np.empty((B, max_depth + 1), np.int32)
    lib().oracle_accept(_p(tokens), _p(parents), _p(n_nodes), _p(verifier_tokens),
                        ctypes.c_int32(B), ctypes.c_int32(N), ctypes.c_int32(max_depth),
                        _p(al), _p(an), _p(ot))
    return al, an, ot


def kv_commit(k_bits, v_bits, kv_len, accept_nodes, accept_len):
    """Plain restatement of "the accepted path becomes part of the prefix": returns copies of
    the uint16 K/V arrays [B,H_kv,Lcap,D] in which row kv_len[b] + i holds what row
    kv_len[b] + accept_nodes[b][i] held, i < accept_len[b], and the new lengths."""
    k2, v2 = k_bits.copy(), v_bits.copy()
    new_len = np.asarray(kv_len, np.int32).copy()
    for b in range(k_bits.shape[0]):
        L = int(kv_len[b])
        for i in range(int(accept_len[b])):
            k2[b, :, L + i] = k_bits[b, :, L + int(accept_nodes[b, i])]
            v2[b, :, L + i] = v_bits[b, :, L + int(accept_nodes[b, i])]
        new_len[b] = L + int(accept_len[b])
    return k2, v2, new_len
