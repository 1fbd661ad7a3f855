"""Thin ctypes binding of ``liblvlm.so`` (declared in ``include/lvlm.h``).

Each function marshals torch CUDA tensors into the C call of the same name and returns the
output tensors; no step of the method runs in Python.  torch is used for device memory and
streams only.  There is no CPU path: a missing library or a non-CUDA tensor is an error.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "liblvlm.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA = range(6)
DEV_NONFINITE, DEV_TIMEOUT, DEV_BOUNDS = 1, 2, 4
W_LINEAR_RANK, W_GEOMETRIC, W_UNIFORM, W_CUSTOM, W_NEAREST_KEPT = range(5)
OP_SCORE_TOKENS, OP_SELECT_TOPK, OP_MERGE_COMPACT, OP_KV_COMPRESS, OP_DECODE_ATTN, OP_PREFILL_ATTN = range(6)

EXPORTS = ("lvlm_version", "lvlm_status_string", "lvlm_workspace_bytes", "lvlm_score_tokens",
           "lvlm_select_topk", "lvlm_merge_compact", "lvlm_kv_compress", "lvlm_decode_attn",
           "lvlm_decode_attn_static", "lvlm_prefill_attn")
STATIC_SCRATCH_BYTES = 4 << 20


class Dims(ctypes.Structure):
    """Mirror of ``lvlm_dims``."""
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "H", "Hkv", "D", "N", "C", "cap", "i0", "n", "k", "q_lo", "q_hi", "causal",
                 "recent", "merge_mode", "cache_stable")] + \
               [(n, ctypes.c_int64) for n in
                ("q_stride_b", "q_stride_n", "q_stride_h", "kv_stride_b", "kv_stride_h",
                 "hid_stride_b", "out_stride_b", "head_stride")]


class LvlmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (lvlm_status {code})")


_lib = None


def use_library(path: Optional[str]) -> None:
    """Makes the binding load another build of the library at its next use (the tests load the build
    with test hooks this way); None goes back to ``liblvlm.so``."""
    global _lib, _LIB_PATH
    _lib = None
    _LIB_PATH = path or os.path.join(_PKG, "liblvlm.so")


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if ``liblvlm.so`` has not been built (see build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2509_00419_b200.build` "
                "(there is no fallback implementation)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, f32, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float,
                                 ctypes.c_size_t)
        dp = ctypes.POINTER(Dims)
        L.lvlm_version.restype = ctypes.c_char_p
        L.lvlm_version.argtypes = []
        L.lvlm_status_string.restype = ctypes.c_char_p
        L.lvlm_status_string.argtypes = [ctypes.c_int]
        L.lvlm_workspace_bytes.restype = sz
        L.lvlm_workspace_bytes.argtypes = [ctypes.c_int, dp]
        L.lvlm_score_tokens.restype = ctypes.c_int
        L.lvlm_score_tokens.argtypes = [vp, vp, vp, dp, f32, vp, vp, vp, sz, vp, vp]
        L.lvlm_select_topk.restype = ctypes.c_int
        L.lvlm_select_topk.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp, vp, sz, vp, vp]
        L.lvlm_merge_compact.restype = ctypes.c_int
        L.lvlm_merge_compact.argtypes = [vp, vp, vp, vp, vp, vp, dp, ctypes.c_int, vp, vp, vp, vp,
                                         sz, vp, vp]
        L.lvlm_kv_compress.restype = ctypes.c_int
        L.lvlm_kv_compress.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, f32, i32, vp, sz, vp, vp]
        L.lvlm_decode_attn.restype = ctypes.c_int
        L.lvlm_decode_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, f32, vp, vp, sz, vp, vp]
        L.lvlm_decode_attn_static.restype = ctypes.c_int
        L.lvlm_decode_attn_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, f32, vp, vp, vp]
        L.lvlm_prefill_attn.restype = ctypes.c_int
        L.lvlm_prefill_attn.argtypes = [vp, vp, vp, dp, f32, vp, vp, vp, vp, vp, sz, vp, vp]
        _lib = L
    return _lib


def version() -> str:
    return lib().lvlm_version().decode()


def status_string(code: int) -> str:
    return lib().lvlm_status_string(int(code)).decode()


def workspace_bytes(op: int, dims: Dims) -> int:
    return int(lib().lvlm_workspace_bytes(int(op), ctypes.byref(dims)))


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError("lvlm works on CUDA tensors only; there is no CPU path")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(code: int, where: str):
    if code != OK:
        raise LvlmError(code, where)


def alloc_workspace(op: int, dims: Dims, device) -> torch.Tensor:
    nbytes = max(workspace_bytes(op, dims), 256)
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def _ws(ws, op, dims, device):
    if ws is None:
        ws = alloc_workspace(op, dims, device)
    return ws, ctypes.c_void_p(ws.data_ptr()), ctypes.c_size_t(ws.numel() * ws.element_size())


# ----------------------------------------------------------------------------------------------
def score_tokens(Q, K, *, N, i0, n, q_lo, q_hi, causal=True, scale=None, lse=None,
                 want_head=False, score_out=None, head_out=None, ws=None, dev_status=None,
                 stream=None):
    """lvlm_score_tokens.  Q [B,q_hi-q_lo,H,D] (a view with strides is fine), K [B,Hkv,cap,D].
    Returns (score [B,n], score_head [B,Hkv,n] or None)."""
    B, Nq, H, D = Q.shape
    Hkv, cap = K.shape[1], K.shape[2]
    d = Dims(B=B, H=H, Hkv=Hkv, D=D, N=N, cap=cap, i0=i0, n=n, q_lo=q_lo, q_hi=q_hi,
             causal=int(causal))
    d.q_stride_b, d.q_stride_n, d.q_stride_h = Q.stride(0), Q.stride(1), Q.stride(2)
    d.kv_stride_b, d.kv_stride_h = K.stride(0), K.stride(1)
    assert Q.stride(3) == 1 and K.stride(3) == 1 and K.stride(2) == D
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    score = score_out if score_out is not None else \
        torch.empty(B, n, dtype=torch.float32, device=Q.device)
    head = head_out
    if head is None and want_head:
        head = torch.empty(B, Hkv, n, dtype=torch.float32, device=Q.device)
    if head is not None:
        assert head.stride(2) == 1 and head.stride(0) == Hkv * head.stride(1)
        d.head_stride = head.stride(1)
    ws, wsp, wsn = _ws(ws, OP_SCORE_TOKENS, d, Q.device)
    _check(lib().lvlm_score_tokens(_ptr(Q), _ptr(K), _ptr(lse), ctypes.byref(d),
                                   ctypes.c_float(scale), _ptr(score), _ptr(head), wsp, wsn,
                                   _ptr(dev_status), _stream(stream)), "lvlm_score_tokens")
    return score, head


def prefill_attn(Q, K, V, *, N, causal=True, scale=None, window=None, i0=0, n=0, want_head=False,
                 out=None, lse=None, score_out=None, head_out=None, ws=None, dev_status=None, stream=None):
    """lvlm_prefill_attn.  Q [B,N,H,D], K, V [B,Hkv,cap,D].  Returns (out [B,N,H,D] bf16, lse [B,H,N],
    score [B,n] or None, score_head [B,Hkv,n] or None); the scores are asked for with
    ``window=(q_lo, q_hi)`` and the image span ``i0, n``."""
    B, Nq, H, D = Q.shape
    Hkv, cap = K.shape[1], K.shape[2]
    assert Nq == N and Q.stride(3) == 1 and K.stride(3) == 1 and K.stride(2) == D and V.stride() == K.stride()
    d = Dims(B=B, H=H, Hkv=Hkv, D=D, N=N, cap=cap, causal=int(causal))
    d.q_stride_b, d.q_stride_n, d.q_stride_h = Q.stride(0), Q.stride(1), Q.stride(2)
    d.kv_stride_b, d.kv_stride_h = K.stride(0), K.stride(1)
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    if out is None:
        out = torch.empty(B, N, H, D, dtype=Q.dtype, device=Q.device)
    if lse is None:
        lse = torch.empty(B, H, N, dtype=torch.float32, device=Q.device)
    score = head = None
    wsp, wsn = None, 0
    if window is not None:
        d.q_lo, d.q_hi, d.i0, d.n = window[0], window[1], i0, n
        score = score_out if score_out is not None else torch.empty(B, n, dtype=torch.float32, device=Q.device)
        head = head_out
        if head is None and want_head:
            head = torch.empty(B, Hkv, n, dtype=torch.float32, device=Q.device)
        if head is not None:
            assert head.stride(2) == 1 and head.stride(0) == Hkv * head.stride(1)
            d.head_stride = head.stride(1)
        ws, wsp, wsn = _ws(ws, OP_PREFILL_ATTN, d, Q.device)
    _check(lib().lvlm_prefill_attn(_ptr(Q), _ptr(K), _ptr(V), ctypes.byref(d), ctypes.c_float(scale), _ptr(out),
                                   _ptr(lse), _ptr(score), _ptr(head), wsp, wsn, _ptr(dev_status),
                                   _stream(stream)), "lvlm_prefill_attn")
    return out, lse, score, head


def select_topk(score, k, *, want_kept=True, want_near=False, rank_out=None, kept_out=None,
                dev_status=None, stream=None):
    """lvlm_select_topk.  score [B,n] fp32 (row stride may exceed n).
    Returns (rank [B,n], kept_idx [B,k] or None, near_tie [B] or None)."""
    B, n = score.shape
    assert score.stride(1) == 1
    rank = rank_out if rank_out is not None else \
        torch.empty(B, n, dtype=torch.int32, device=score.device)
    kept = kept_out
    if kept is None and want_kept:
        kept = torch.empty(B, k, dtype=torch.int32, device=score.device)
    near = torch.empty(B, dtype=torch.int32, device=score.device) if want_near else None
    _check(lib().lvlm_select_topk(_ptr(score), B, n, score.stride(0), k, _ptr(rank), _ptr(kept),
                                  _ptr(near), None, 0, _ptr(dev_status), _stream(stream)),
           "lvlm_select_topk")
    return rank, kept, near


def merge_dims(hidden, rank, *, i0, k, Kc=None) -> Dims:
    B, N, C = hidden.shape
    n = rank.shape[1]
    d = Dims(B=B, N=N, C=C, i0=i0, n=n, k=k, D=128)
    d.hid_stride_b = hidden.stride(0)
    if Kc is not None:
        d.Hkv, d.cap, d.D = Kc.shape[1], Kc.shape[2], Kc.shape[3]
        d.kv_stride_b, d.kv_stride_h = Kc.stride(0), Kc.stride(1)
    return d


def merged_rows(N, n, k, mode=W_LINEAR_RANK) -> int:
    """Rows of a sequence after lvlm_merge_compact."""
    if mode == W_NEAREST_KEPT:
        return N - (n - k)
    return N - max(n - k - 1, 0)


def merge_compact(hidden, rank, *, i0, k, mode=W_LINEAR_RANK, Kc=None, Vc=None, pos_ids=None,
                  w_custom=None, mass=None, in_place=False, out=None, new_len=None, ws=None,
                  dev_status=None, stream=None):
    """lvlm_merge_compact.  Returns (hidden_out or the compacted `hidden`, new_len [B]).
    With in_place=True `hidden` is compacted in place and its first new_len rows are valid.
    Kc, Vc and pos_ids are always compacted in place."""
    B, N, C = hidden.shape
    n = rank.shape[1]
    d = merge_dims(hidden, rank, i0=i0, k=k, Kc=Kc)
    d.merge_mode = int(mode)
    rows = merged_rows(N, n, k, mode)
    if in_place:
        out = None
    elif out is None:
        out = torch.empty(B, rows, C, dtype=hidden.dtype, device=hidden.device)
    if out is not None:
        d.out_stride_b = out.stride(0)
    if new_len is None:
        new_len = torch.empty(B, dtype=torch.int32, device=hidden.device)
    ws, wsp, wsn = _ws(ws, OP_MERGE_COMPACT, d, hidden.device)
    _check(lib().lvlm_merge_compact(_ptr(hidden), _ptr(out), _ptr(Kc), _ptr(Vc), _ptr(pos_ids),
                                    _ptr(rank), ctypes.byref(d), int(mode), _ptr(w_custom),
                                    _ptr(mass), _ptr(new_len), wsp, wsn, _ptr(dev_status),
                                    _stream(stream)), "lvlm_merge_compact")
    return (hidden if in_place else out), new_len


def nearest_assignment(ws: torch.Tensor, B: int, r: int) -> torch.Tensor:
    """Assignment lvlm_merge_compact leaves at the start of its workspace in mode NEAREST_KEPT:
    [B, r] int32, for the dropped tokens in ascending order the index of their kept token."""
    return ws[:B * r * 4].view(torch.int32).view(B, r)


def kv_dims(Kc, *, H=None, recent=0) -> Dims:
    B, Hkv, cap, D = Kc.shape
    d = Dims(B=B, Hkv=Hkv, H=H if H is not None else Hkv, D=D, cap=cap, recent=recent)
    d.kv_stride_b, d.kv_stride_h = Kc.stride(0), Kc.stride(1)
    return d


def kv_compress(Kc, Vc, acc_score, length, *, beta=1.0, budget=0, recent=0, e_lo=None, e_hi=None,
                pos=None, ws=None, dev_status=None, stream=None):
    """lvlm_kv_compress: everything is updated in place (Kc, Vc, acc_score, pos, length)."""
    d = kv_dims(Kc, recent=recent)
    ws, wsp, wsn = _ws(ws, OP_KV_COMPRESS, d, Kc.device)
    _check(lib().lvlm_kv_compress(_ptr(Kc), _ptr(Vc), _ptr(acc_score), _ptr(pos), _ptr(length),
                                  _ptr(e_lo), _ptr(e_hi), ctypes.byref(d), ctypes.c_float(beta),
                                  int(budget), wsp, wsn, _ptr(dev_status), _stream(stream)),
           "lvlm_kv_compress")


def decode_attn(q, Kc, Vc, length, *, k_new=None, v_new=None, acc_score=None, scale=None, out=None,
                ws=None, dev_status=None, stream=None, cache_stable=False):
    """lvlm_decode_attn.  q [B,H,D]; returns out [B,H,D] bf16.  Kc, Vc, length and acc_score are
    updated in place when k_new/v_new or acc_score are given."""
    B, H, D = q.shape
    d = kv_dims(Kc, H=H)
    d.cache_stable = int(bool(cache_stable))
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    if out is None:
        out = torch.empty(B, H, D, dtype=q.dtype, device=q.device)
    ws, wsp, wsn = _ws(ws, OP_DECODE_ATTN, d, q.device)
    _check(lib().lvlm_decode_attn(_ptr(q), _ptr(Kc), _ptr(Vc), _ptr(length), _ptr(k_new),
                                  _ptr(v_new), _ptr(acc_score), ctypes.byref(d),
                                  ctypes.c_float(scale), _ptr(out), wsp, wsn, _ptr(dev_status),
                                  _stream(stream)), "lvlm_decode_attn")
    return out


def decode_attn_static(q, Kc, Vc, length, *, k_new=None, v_new=None, acc_score=None, scale=None,
                       out=None, dev_status=None, stream=None):
    """lvlm_decode_attn_static: lvlm_decode_attn for callers that have no way to get device
    scratch memory (all of it belongs to someone else's pool, or allocating would stall the
    device).  The scratch is a fixed array inside the library, at most STATIC_SCRATCH_BYTES per
    problem, shared by every call on the device: calls must not overlap on the GPU.  ``out`` is
    required to come from the caller as well when nothing may be allocated; it is created here
    only as a convenience when omitted."""
    B, H, D = q.shape
    d = kv_dims(Kc, H=H)
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    if out is None:
        out = torch.empty(B, H, D, dtype=q.dtype, device=q.device)
    _check(lib().lvlm_decode_attn_static(_ptr(q), _ptr(Kc), _ptr(Vc), _ptr(length), _ptr(k_new),
                                         _ptr(v_new), _ptr(acc_score), ctypes.byref(d),
                                         ctypes.c_float(scale), _ptr(out), _ptr(dev_status),
                                         _stream(stream)), "lvlm_decode_attn_static")
    return out
