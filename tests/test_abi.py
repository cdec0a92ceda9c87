"""The C-ABI library builds, loads and exports every function the header declares."""
import ctypes
import os
import re

import paper_2311_08252_b200 as rest
from paper_2311_08252_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    inc = os.path.join(ROOT, "include")
    text = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rest_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    so = cuda_build.build()
    L = ctypes.CDLL(so)
    names = declared_functions()
    assert {"rest_datastore_create", "rest_draft", "rest_tree_attention", "rest_accept"} <= set(names)
    for n in names:
        assert hasattr(L, n), n
    assert set(rest.EXPORTS) == set(names)


def test_status_strings_and_size_queries_without_a_gpu():
    L = rest.lib()
    assert L.rest_status_string(0) == b"ok"
    assert b"workspace" in L.rest_status_string(3)
    # validation scratch (a bit per position + flags) plus the bucket index (a 256-byte header, the
    # first-token table rounded to 256 bytes, and at least 4096 pair entries of 32 bytes)
    assert L.rest_datastore_aux_bytes(64, 4, 10) == (2 * 4 + 256) + (256 + 256 + 4096 * 32)
    assert L.rest_datastore_aux_bytes(64, 4, (1 << 22) + 1) == 2 * 4 + 256     # vocabulary too large to index
    # many (context, head) units -> a single key split, no scratch
    assert rest.tree_attention_workspace_bytes(256, 32, 64, 128, 4160) == 0
    # single stream, 32 heads -> one 8-block cluster per head merges on chip, no scratch
    assert rest.tree_attention_workspace_bytes(1, 32, 64, 128, 2112) == 0
    # very few heads, long cache -> several clusters per head, fp32 partials of N*(D+2) floats
    n = rest.tree_attention_workspace_bytes(1, 2, 64, 128, 8256)
    assert n > 0 and n % (2 * 64 * 130 * 4) == 0
    assert rest.tree_attention_workspace_bytes(1, 32, 64, 64, 2112) == 0   # unsupported D


def test_host_argument_checks_return_status_codes():
    L = rest.lib()
    h = ctypes.c_void_p()
    assert L.rest_datastore_create(None, 10, None, 4, 10, 0, None, 0, None, ctypes.byref(h)) == 1
    assert L.rest_datastore_create(8, 10, 8, 5, 10, 0, None, 0, None, ctypes.byref(h)) == 1
    assert L.rest_datastore_create(8, 1 << 33, 8, 4, 10, 0, None, 0, None, ctypes.byref(h)) == 1
    assert L.rest_datastore_create(8, 10, 8, 4, 10, 1, None, 0, None, ctypes.byref(h)) == 1
    # a handle over (never dereferenced) fake pointers: argument validation only, B = 0 launches nothing
    assert L.rest_datastore_create(256, 10, 512, 4, 10, 0, None, 0, None, ctypes.byref(h)) == 0
    prm = rest._Params(16, 2, 5000, 10, 64, 0)
    args = [256, 8, 256, 0] + [256] * 10 + [0, 0, None]
    assert L.rest_draft(h, ctypes.byref(prm), *args) == 0              # B = 0
    args[3] = 1
    bad = rest._Params(17, 2, 5000, 10, 64, 0)
    assert L.rest_draft(h, ctypes.byref(bad), *args) == 2
    bad = rest._Params(16, 2, 5000, 17, 64, 0)
    assert L.rest_draft(h, ctypes.byref(bad), *args) == 2
    bad = rest._Params(16, 2, 5000, 10, 257, 0)
    assert L.rest_draft(h, ctypes.byref(bad), *args) == 2
    bad = rest._Params(16, 0, 5000, 10, 64, 0)
    assert L.rest_draft(h, ctypes.byref(bad), *args) == 1
    bad = rest._Params(16, 2, 5000, 10, 64, 7)
    assert L.rest_draft(h, ctypes.byref(bad), *args) == 1
    L.rest_datastore_destroy(h)
    strides = (ctypes.c_int64 * 9)(*([128] * 9))
    att = lambda N, D, H, Hkv, st=strides: L.rest_tree_attention(
        256, 256, 256, st, 256, 256, 1, H, Hkv, N, D, 512, 1.0, 256, None, None, 0, None)
    assert att(64, 64, 4, 4) == 2
    assert att(64, 128, 4, 3) == 2
    assert att(272, 128, 4, 4) == 2
    assert L.rest_tree_attention(256, 256, 256, strides, 256, 256, 1, 4, 4, 64, 128, 512, 0.0, 256,
                                 None, None, 0, None) == 1       # the softmax scale must be positive
    assert L.rest_tree_attention(256, 256, 256, strides, 256, 256, 1, 2, 2, 64, 128, 8256, 1.0, 256,
                                 None, None, 0, None) == 1       # needs a workspace, none given
    odd = (ctypes.c_int64 * 9)(*([124] * 9))
    assert att(64, 128, 4, 4, odd) == 1
    assert L.rest_accept(None, None, None, None, 1, 64, 10, None, None, None, None) == 1
    assert L.rest_accept(None, None, None, None, 0, 64, 10, None, None, None, None) == 0
