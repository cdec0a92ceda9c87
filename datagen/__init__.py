"""Seeded synthetic inputs for the REST draft / verify path.

Input data only: token datastores, the host-built suffix array, query contexts,
attention tensors and verifier tokens.  None of the method's arithmetic lives
here; the CUDA library and the CPU oracle both consume these arrays and share
nothing else.

Recipe (all draws from a counter-based splitmix64 mixer, master seed 20231108):
an order-k Markov chain over a 32000-token vocabulary whose successor candidates
are hashed from the state and whose candidate rank is Zipf-distributed, cut in
independent 2^16-token segments; optional copy runs (code-like repetition) and
mixed segment kinds.  Contexts are 70 % fresh chain samples, 20 % datastore
slices with one token edited 3..17 places from the end, 5 % unmodified slices
and 5 % uniform noise.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libdatagen.so")
_SRC = os.path.join(_HERE, "gen.cpp")

MASTER_SEED = 20231108
VOCAB = 32000


def build(force: bool = False) -> str:
    """Compile gen.cpp into libdatagen.so (g++, OpenMP)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", _SRC, "-o", _SO])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.dg_mix.restype = ctypes.c_uint64
        L.dg_mix.argtypes = [ctypes.c_uint64] * 3
        L.dg_markov_tokens.restype = None
        L.dg_markov_tokens.argtypes = [
            ctypes.c_uint64, ctypes.c_int64, ctypes.c_uint32, ctypes.c_int, ctypes.c_double,
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        L.dg_contexts.restype = None
        L.dg_contexts.argtypes = [
            ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint32, ctypes.c_int,
            ctypes.c_double, ctypes.c_int, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
        L.dg_build_sa.restype = ctypes.c_int
        L.dg_build_sa.argtypes = [
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint32, ctypes.c_int, ctypes.c_int,
            ctypes.c_void_p]
        L.dg_verify_sa.restype = ctypes.c_int
        L.dg_verify_sa.argtypes = [
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        _lib = L
    return _lib


@dataclass(frozen=True)
class Workload:
    """One synthetic workload: datastore recipe, draft call shape, attention shape."""
    name: str
    index: int            # seed = MASTER_SEED + index
    n_tokens: int
    order: int
    zipf_s: float
    R: int
    copy_runs: bool
    mixed: bool
    sa_bytes: int
    B: int
    Lc: int               # context length (tokens)
    K: int
    m: int
    N: int
    H: int
    D: int
    L: int                # KV prefix length
    layers: int
    n_max: int = 16
    n_min: int = 2
    vocab: int = VOCAB

    @property
    def seed(self) -> int:
        return MASTER_SEED + self.index

    def scaled(self, n_tokens: int | None = None, B: int | None = None, L: int | None = None,
               layers: int | None = None, H: int | None = None) -> "Workload":
        """Same recipe at a reduced size (used by tests that must finish in seconds)."""
        kw = {}
        if n_tokens is not None:
            kw["n_tokens"] = n_tokens
        if B is not None:
            kw["B"] = B
        if L is not None:
            kw["L"] = L
        if layers is not None:
            kw["layers"] = layers
        if H is not None:
            kw["H"] = H
        return replace(self, **kw)


# The five workloads, in order: tiny, single-stream code-like, batched serving,
# large datastore, stress.
WORKLOADS = {
    "tiny": Workload("tiny", 0, 1_000_000, 3, 1.1, 64, False, False, 4,
                     1, 256, 5000, 10, 64, 32, 128, 256, 1),
    "single_stream": Workload("single_stream", 1, 100_000_000, 4, 1.1, 64, True, False, 4,
                              1, 2048, 5000, 10, 64, 32, 128, 2048, 32),
    "batched": Workload("batched", 2, 1_000_000_000, 3, 1.1, 64, False, False, 4,
                        256, 1024, 5000, 10, 64, 32, 128, 4096, 1),
    "large": Workload("large", 3, 4_000_000_000, 5, 1.1, 64, False, True, 8,
                      64, 4096, 5000, 12, 64, 40, 128, 8192, 40),
    "stress": Workload("stress", 4, 500_000_000, 2, 1.5, 64, False, False, 4,
                       128, 512, 20000, 16, 128, 32, 128, 16384, 1),
}


def make_tokens(w: Workload) -> np.ndarray:
    """The datastore token stream T[0..n) as int32."""
    out = np.empty(w.n_tokens, dtype=np.int32)
    lib().dg_markov_tokens(w.seed, w.n_tokens, w.vocab, w.order, w.zipf_s, w.R,
                           int(w.copy_runs), int(w.mixed), out.ctypes.data)
    return out


def build_suffix_array(tokens: np.ndarray, vocab: int, W: int = 32, sa_bytes: int = 4) -> np.ndarray:
    """Host suffix array of `tokens`, ordered on the first W tokens of each suffix
    (W=0: full suffixes), ties by ascending position."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    out = np.empty(tokens.size, dtype=np.int32 if sa_bytes == 4 else np.int64)
    rc = lib().dg_build_sa(tokens.ctypes.data, tokens.size, vocab, W, sa_bytes, out.ctypes.data)
    if rc != 0:
        raise ValueError(f"dg_build_sa failed with code {rc}")
    return out


def verify_suffix_array(tokens: np.ndarray, sa: np.ndarray, W: int = 32) -> int:
    """0 when `sa` is a permutation ordered on the first W tokens (ties by position)."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    sa = np.ascontiguousarray(sa)
    return lib().dg_verify_sa(tokens.ctypes.data, tokens.size, W, sa.dtype.itemsize, sa.ctypes.data)


def make_contexts(w: Workload, tokens: np.ndarray, B: int | None = None, Lc: int | None = None,
                  salt: int = 0) -> np.ndarray:
    """[B, Lc] int32 query contexts for workload `w` over its datastore `tokens`."""
    B = w.B if B is None else B
    Lc = w.Lc if Lc is None else Lc
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    out = np.empty((B, Lc), dtype=np.int32)
    lib().dg_contexts(w.seed + 7919 * (salt + 1), tokens.ctypes.data, tokens.size, w.vocab,
                      w.order, w.zipf_s, w.R, B, Lc, out.ctypes.data)
    return out


def make_verifier_tokens(seed: int, tokens: np.ndarray, parents: np.ndarray,
                         n_nodes: np.ndarray, vocab: int) -> np.ndarray:
    """[B, N+1] int32 stand-ins for the verifier's sampled tokens.

    Slot 0 is the token after the prefix, slot i+1 the token after tree node i.  Half of
    the slots copy the token of a random child of that node (so non-empty acceptances
    occur), the rest are uniform over the vocabulary.  `tokens`/`parents` describe draft
    trees [B, N]; pure data shuffling, no acceptance logic.
    """
    B, N = tokens.shape
    rng = np.random.Generator(np.random.Philox(seed))
    out = rng.integers(0, vocab, size=(B, N + 1), dtype=np.int64).astype(np.int32)
    coin = rng.random((B, N + 1)) < 0.5
    pick = rng.integers(0, 1 << 30, size=(B, N + 1))
    for b in range(B):
        nn = int(n_nodes[b])
        for slot in range(nn + 1):
            if not coin[b, slot]:
                continue
            node = slot - 1
            kids = np.nonzero(parents[b, :nn] == node)[0]
            if kids.size:
                out[b, slot] = tokens[b, kids[pick[b, slot] % kids.size]]
    return out


def make_random_tree(seed: int, N: int, max_depth: int, n_nodes: int | None = None):
    """A seeded random tree in breadth-first order for standalone attention runs:
    returns (parents[N] int32, depth[N] int32, mask[N, ceil(N/32)] uint32) where mask row
    i has bit j set iff j is i or an ancestor of i.  Slots >= n_nodes keep only their own bit."""
    n_nodes = N if n_nodes is None else n_nodes
    rng = np.random.Generator(np.random.Philox(seed))
    depth = np.zeros(N, dtype=np.int32)
    parents = np.full(N, -1, dtype=np.int32)
    # split n_nodes into consecutive levels of at least one node each
    n_levels = max(1, min(max_depth, n_nodes))
    cuts = np.sort(rng.choice(np.arange(1, n_nodes), size=n_levels - 1, replace=False)) \
        if n_levels > 1 else np.array([], dtype=np.int64)
    bounds = np.concatenate([[0], cuts, [n_nodes]]).astype(np.int64)
    for lv in range(n_levels):
        s, e = int(bounds[lv]), int(bounds[lv + 1])
        depth[s:e] = lv + 1
        if lv > 0:
            ps, pe = int(bounds[lv - 1]), int(bounds[lv])
            parents[s:e] = np.sort(rng.integers(ps, pe, size=e - s))
    Wm = (N + 31) // 32
    mask = np.zeros((N, Wm), dtype=np.uint32)
    for i in range(N):
        if i < n_nodes and parents[i] >= 0:
            mask[i] = mask[parents[i]]
        mask[i, i >> 5] |= np.uint32(1 << (i & 31))
    return parents, depth, mask


def make_qkv(seed: int, B: int, H: int, N: int, D: int, Lcap: int, device="cpu", H_kv=None):
    """Seeded N(0,1) attention inputs rounded to bf16 (torch Philox/MT generator on `device`):
    q [B,N,H,D], k and v [B,H_kv,Lcap,D]."""
    import torch
    H_kv = H if H_kv is None else H_kv
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    q = torch.randn((B, N, H, D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    k = torch.randn((B, H_kv, Lcap, D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    v = torch.randn((B, H_kv, Lcap, D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    return q, k, v
