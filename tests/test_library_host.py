"""Host-side checks that need no GPU: the library loads, exports what the header declares, sizes
its workspaces and rejects bad arguments before anything is enqueued."""
import ctypes
import os
import re

import pytest

from paper_2509_00419_b200 import binding as L
from paper_2509_00419_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return L.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "lvlm.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(lvlm_[a-z_]+)\s*\(", header))
    assert set(L.EXPORTS) <= declared and len(declared) >= 8
    for name in declared:
        assert hasattr(lib, name), name
    assert "sm_100a" in L.version()
    assert L.status_string(L.ERR_WORKSPACE).startswith("workspace")


def test_dims_struct_matches_header():
    header = open(os.path.join(ROOT, "include", "lvlm.h")).read()
    body = header[header.index("typedef struct lvlm_dims {"):header.index("} lvlm_dims;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for ctype, decl in re.findall(r"(int32_t|int64_t)\s+([^;]+);", body):
        for nm in decl.split(","):
            names.append((nm.strip(), ctype))
    assert [(n, "int32_t" if t is ctypes.c_int32 else "int64_t") for n, t in L.Dims._fields_] == names


def test_workspace_sizes(lib):
    d = L.Dims(B=16, H=32, Hkv=8, D=128, N=1888, C=4096, cap=1888, i0=0, n=1792, k=1059,
               q_lo=1792, q_hi=1888, causal=1)
    for op in range(5):
        assert L.workspace_bytes(op, d) % 256 == 0 and L.workspace_bytes(op, d) > 0
    assert L.workspace_bytes(L.OP_MERGE_COMPACT, L.Dims()) == 0       # invalid dims
    assert L.workspace_bytes(99, d) == 0
    assert L.workspace_bytes(L.OP_SCORE_TOKENS, d) >= 16 * 32 * 1792 * 4


def test_bad_arguments_are_rejected_on_the_host(lib):
    p = ctypes.c_void_p(0x1000)           # never dereferenced: every call below fails validation
    odd = ctypes.c_void_p(0x1008)
    ws, n_ws = ctypes.c_void_p(0x10000), ctypes.c_size_t(1 << 40)
    d = L.Dims(B=1, H=8, Hkv=8, D=128, N=640, C=1024, cap=640, i0=0, n=576, k=287, q_lo=576,
               q_hi=640, causal=1)
    ref = ctypes.byref

    def score(dd, Q=p, K=p, out=p, w=ws, wn=n_ws):
        return lib.lvlm_score_tokens(Q, K, None, ref(dd), ctypes.c_float(0.1), out, None, w, wn, None, None)

    assert score(d, Q=None) == L.ERR_INVALID_ARG
    assert score(d, out=None) == L.ERR_INVALID_ARG
    assert score(d, Q=odd) == L.ERR_ALIGNMENT
    assert score(d, w=None) == L.ERR_WORKSPACE
    assert score(d, wn=ctypes.c_size_t(16)) == L.ERR_WORKSPACE
    for field, val, code in (("D", 64, L.ERR_UNSUPPORTED), ("q_hi", 641, L.ERR_INVALID_ARG),
                             ("q_lo", 640, L.ERR_INVALID_ARG), ("n", 641, L.ERR_INVALID_ARG),
                             ("Hkv", 3, L.ERR_INVALID_ARG), ("cap", 600, L.ERR_INVALID_ARG),
                             ("q_stride_n", 1028, L.ERR_ALIGNMENT)):
        dd = L.Dims.from_buffer_copy(d)
        setattr(dd, field, val)
        assert score(dd) == code, field

    sel = lambda n, k, s=p, r=p: lib.lvlm_select_topk(s, 1, n, 0, k, r, None, None, None, 0, None, None)
    assert sel(10, 11) == L.ERR_INVALID_ARG and sel(10, -1) == L.ERR_INVALID_ARG
    assert sel(0, 0) == L.ERR_INVALID_ARG and sel(10, 5, s=None) == L.ERR_INVALID_ARG
    assert sel(65537, 5) == L.ERR_UNSUPPORTED

    def merge(dd, h=p, rk=p, Kc=None, Vc=None, mode=0, wc=None, w=ws, wn=n_ws):
        return lib.lvlm_merge_compact(h, None, Kc, Vc, None, rk, ref(dd), mode, wc, None, None, w, wn, None, None)

    assert merge(d, h=None) == L.ERR_INVALID_ARG and merge(d, rk=None) == L.ERR_INVALID_ARG
    assert merge(d, Kc=p) == L.ERR_INVALID_ARG                       # K without V
    assert merge(d, mode=L.W_CUSTOM) == L.ERR_INVALID_ARG            # no weight list
    assert merge(d, mode=7) == L.ERR_INVALID_ARG
    assert merge(d, h=odd) == L.ERR_ALIGNMENT
    assert merge(d, w=None) == L.ERR_WORKSPACE
    for field, val in (("k", 577), ("k", -1), ("C", 1023), ("i0", 100), ("B", 0)):
        dd = L.Dims.from_buffer_copy(d)
        setattr(dd, field, val)
        assert merge(dd) == L.ERR_INVALID_ARG, field

    def kvc(dd, beta=0.995, Kc=p, Vc=p, acc=p, ln=p, lo=None, hi=None, w=ws):
        return lib.lvlm_kv_compress(Kc, Vc, acc, None, ln, lo, hi, ref(dd), ctypes.c_float(beta), 0, w, n_ws, None, None)

    assert kvc(d, beta=0.0) == L.ERR_INVALID_ARG and kvc(d, beta=1.5) == L.ERR_INVALID_ARG
    assert kvc(d, ln=None) == L.ERR_INVALID_ARG and kvc(d, lo=p) == L.ERR_INVALID_ARG
    assert kvc(d, Kc=odd) == L.ERR_ALIGNMENT and kvc(d, w=None) == L.ERR_WORKSPACE
    dd = L.Dims.from_buffer_copy(d); dd.cap = 20000
    assert kvc(dd) == L.ERR_UNSUPPORTED

    def dec(dd, q=p, kn=None, vn=None, out=p, w=ws):
        return lib.lvlm_decode_attn(q, p, p, p, kn, vn, None, ref(dd), ctypes.c_float(0.1), out, w, n_ws, None, None)

    assert dec(d, q=None) == L.ERR_INVALID_ARG and dec(d, kn=p) == L.ERR_INVALID_ARG
    assert dec(d, out=odd) == L.ERR_ALIGNMENT and dec(d, w=None) == L.ERR_WORKSPACE
    dd = L.Dims.from_buffer_copy(d); dd.H, dd.Hkv = 32, 2
    assert dec(dd) == L.ERR_UNSUPPORTED                              # 16 query heads per KV head
    dd = L.Dims.from_buffer_copy(d); dd.D = 64
    assert dec(dd) == L.ERR_UNSUPPORTED


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(TypeError):
        L.select_topk(torch.zeros(1, 4), 2)


def test_schedule_host_function():
    from paper_2509_00419_b200 import pipeline as P
    assert P.pyramid_schedule(2880, 0.03, 3) == [895, 278, 86]
    assert P.pyramid_schedule(1792, 0.35, 2) == [1060, 627]
    assert L.merged_rows(640, 576, 287) == 352 and L.merged_rows(640, 576, 576) == 640
