"""ctypes binding of ``libmala.so`` (C ABI in ``include/mala.h``): argument marshalling only.

PyTorch is used for device memory and the current stream; every step of the attention path runs in
the library's kernels.  There is no CPU or eager fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIBPATH = os.path.join(_HERE, "libmala.so")
_lib = None

OP_FWD, OP_BWD, OP_DECODE = 0, 1, 2


class MalaError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {lib().mala_strerror(code).decode()} (code {code})")
        self.code = code


class _TIn(ctypes.Structure):
    _fields_ = [("p", ctypes.c_void_p), ("sb", ctypes.c_int64), ("sn", ctypes.c_int64), ("sh", ctypes.c_int64)]


class _TOut(ctypes.Structure):
    _fields_ = [("p", ctypes.c_void_p), ("sb", ctypes.c_int64), ("sn", ctypes.c_int64), ("sh", ctypes.c_int64)]


class _Stats(ctypes.Structure):
    _fields_ = [("retained_per_block", ctypes.c_void_p), ("tile_bitmask", ctypes.c_void_p),
                ("totals", ctypes.c_void_p)]


def lib():
    """Loads libmala.so (built in-tree by ``paper_2609_32712_b200.build``); fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIBPATH):
            raise ImportError(f"{_LIBPATH} is missing: run `python -m paper_2609_32712_b200.build` (needs nvcc)")
        L = ctypes.CDLL(_LIBPATH)
        i, f, vp, sz = ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
        L.mala_fwd.argtypes = [_TIn, _TIn, _TIn, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, f, f, vp, sz, vp]
        L.mala_bwd.argtypes = [_TIn, _TIn, _TIn, _TIn, _TIn, vp, _TOut, _TOut, _TOut, ctypes.POINTER(_Stats),
                               i, i, i, i, i, i, f, f, vp, sz, vp]
        L.mala_fwd_chunk.argtypes = [_TIn, _TIn, _TIn, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, i, f, f, vp,
                                     sz, vp]
        L.mala_bwd_chunk.argtypes = [_TIn, _TIn, _TIn, _TIn, _TIn, vp, _TOut, _TOut, _TOut, ctypes.POINTER(_Stats),
                                     i, i, i, i, i, i, i, f, f, vp, sz, vp]
        L.mala_fwd_chunk.restype = i
        L.mala_bwd_chunk.restype = i
        L.mala_fwd_chunk_split.argtypes = [_TIn, _TIn, _TIn, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, i, f, f,
                                           i, vp, sz, vp]
        L.mala_fwd_chunk_split.restype = i
        L.mala_fwd_varlen.argtypes = [_TIn, _TIn, _TIn, vp, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, i, f, f,
                                      vp, sz, vp]
        L.mala_bwd_varlen.argtypes = [_TIn, _TIn, _TIn, _TIn, _TIn, vp, vp, _TOut, _TOut, _TOut, ctypes.POINTER(_Stats),
                                      i, i, i, i, i, i, i, f, f, vp, sz, vp]
        L.mala_fwd_varlen_prefix.argtypes = [_TIn, _TIn, _TIn, vp, vp, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i,
                                             i, i, i, f, f, vp, sz, vp]
        L.mala_fwd_varlen_prefix.restype = i
        L.mala_bwd_varlen_prefix.argtypes = [_TIn, _TIn, _TIn, _TIn, _TIn, vp, vp, vp, _TOut, _TOut, _TOut,
                                             ctypes.POINTER(_Stats), i, i, i, i, i, i, i, i, i, f, f, vp, sz, vp]
        L.mala_bwd_varlen_prefix.restype = i
        L.mala_fwd_paged.argtypes = [_TIn, _TIn, _TIn, vp, vp, vp, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, i, i,
                                     i, i, f, f, vp, sz, vp]
        L.mala_fwd_paged.restype = i
        L.mala_fwd_varlen.restype = i
        L.mala_bwd_varlen.restype = i
        L.mala_decode.argtypes = [_TIn, _TIn, _TIn, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, f, f, i, vp, sz, vp]
        L.mala_decode_multi.argtypes = [_TIn, _TIn, _TIn, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, f, f, i,
                                        vp, sz, vp]
        L.mala_decode_multi.restype = i
        L.mala_decode_paged.argtypes = [_TIn, _TIn, _TIn, vp, vp, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, i, i,
                                        f, f, i, vp, sz, vp]
        L.mala_decode_paged.restype = i
        L.mala_decode_fp8.argtypes = [_TIn, _TIn, _TIn, vp, vp, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, f, f, i, vp,
                                      sz, vp]
        L.mala_decode_fp8.restype = i
        L.mala_decode_fp8_multi.argtypes = [_TIn, _TIn, _TIn, vp, vp, _TOut, vp, ctypes.POINTER(_Stats), i, i, i, i, i, i, f,
                                            f, i, vp, sz, vp]
        L.mala_decode_fp8_multi.restype = i
        L.mala_decode_fp8_paged.argtypes = [_TIn, _TIn, _TIn, vp, vp, vp, vp, _TOut, vp, ctypes.POINTER(_Stats),
                                            i, i, i, i, i, i, i, f, f, i, vp, sz, vp]
        L.mala_decode_fp8_paged.restype = i
        L.mala_decode_static.argtypes = [_TIn, _TIn, _TIn, _TOut, vp, i, i, i, i, i, f, f, i, vp]
        L.mala_decode_static.restype = i
        L.mala_test_expire_wait.argtypes = [ctypes.c_longlong, vp]
        L.mala_test_expire_wait.restype = i
        L.mala_workspace_bytes.argtypes = [i, i, i, i, i, i, i]
        L.mala_workspace_bytes.restype = sz
        L.mala_tile_shape.argtypes = [i, i, ctypes.POINTER(i), ctypes.POINTER(i)]
        L.mala_decode_suggest_splits.argtypes = [i, i, i, i]
        L.mala_decode_suggest_splits.restype = i
        L.mala_device_status.argtypes = [ctypes.POINTER(i), i]
        L.mala_strerror.argtypes = [i]
        L.mala_strerror.restype = ctypes.c_char_p
        L.mala_version.restype = i
        for n in ("mala_fwd", "mala_bwd", "mala_decode", "mala_tile_shape", "mala_device_status"):
            getattr(L, n).restype = i
        _lib = L
    return _lib


def _view(t: torch.Tensor, cls):
    assert t.dtype == torch.bfloat16 and t.dim() == 4 and t.stride(3) == 1, "expects bf16 [B,N,H,d], last dim contiguous"
    return cls(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def tile_shape(op: int, d: int):
    bq, bk = ctypes.c_int(0), ctypes.c_int(0)
    rc = lib().mala_tile_shape(op, d, ctypes.byref(bq), ctypes.byref(bk))
    if rc != 0:
        raise MalaError(rc, "mala_tile_shape")
    return bq.value, bk.value


def decode_suggest_splits(B: int, Hkv: int, Nk: int, sm_count: int = 0) -> int:
    """mala_decode_suggest_splits: the smallest split count that still fills the SMs evenly."""
    rc = int(lib().mala_decode_suggest_splits(B, Hkv, Nk, sm_count))
    if rc < 0:
        raise MalaError(rc, "mala_decode_suggest_splits")
    return rc


def workspace_bytes(op: int, B: int, Hq: int, Hkv: int, N: int, d: int, num_splits: int = 0) -> int:
    return int(lib().mala_workspace_bytes(op, B, Hq, Hkv, N, d, num_splits))


def device_status(clear: bool = True) -> int:
    code = ctypes.c_int(0)
    rc = lib().mala_device_status(ctypes.byref(code), int(clear))
    if rc != 0:
        raise MalaError(rc, "mala_device_status")
    return code.value


def test_expire_wait(limit_cycles: int = 100000) -> None:
    """mala_test_expire_wait: makes one bounded device-side wait run out (test support)."""
    rc = lib().mala_test_expire_wait(limit_cycles, _stream())
    if rc != 0:
        raise MalaError(rc, "mala_test_expire_wait")


class Stats:
    """Device tensors for the optional telemetry of one call."""

    def __init__(self, retained_shape, words: int, device):
        self.retained = torch.zeros(retained_shape, dtype=torch.int32, device=device)
        self.bitmask = torch.zeros(tuple(retained_shape) + (words,), dtype=torch.int32, device=device)
        self.totals = torch.zeros(2, dtype=torch.int64, device=device)
        self.c = _Stats(self.retained.data_ptr(), self.bitmask.data_ptr(), self.totals.data_ptr())

    def mask(self, n_bits: int) -> torch.Tensor:
        """Boolean [..., n_bits] expansion of the bitmask (bit x of a row = tile x retained)."""
        w = self.bitmask.to(torch.int64) & 0xFFFFFFFF
        bits = (w.unsqueeze(-1) >> torch.arange(32, device=w.device)) & 1
        return bits.flatten(-2)[..., :n_bits].bool()


def _ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def fwd(q, k, v, scale: float, tau: float, causal: bool = True, stats: bool = False, out=None, lse=None, ws=None):
    """mala_fwd: returns (o [B,N,Hq,d] bf16, lse [B,Hq,N] fp32, Stats or None)."""
    B, N, Hq, d = q.shape
    Hkv = k.shape[2]
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq, N), dtype=torch.float32, device=q.device) if lse is None else lse
    T = -(-N // 128)
    st = Stats((B, Hq, T), -(-T // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_FWD, B, Hq, Hkv, N, d), q.device) if ws is None else ws
    rc = lib().mala_fwd(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), _view(o, _TOut), lse.data_ptr(),
                        ctypes.byref(st.c) if st else None, B, Hq, Hkv, N, d, int(causal), scale, tau,
                        ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_fwd")
    return o, lse, st


def bwd(q, k, v, o, do, lse, scale: float, tau: float, causal: bool = True, stats: bool = False, ws=None,
        dq=None, dk=None, dv=None):
    """mala_bwd: returns (dq, dk, dv, Stats or None)."""
    B, N, Hq, d = q.shape
    Hkv = k.shape[2]
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    T = -(-N // 128)
    st = Stats((B, Hq, T), -(-T // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_BWD, B, Hq, Hkv, N, d), q.device) if ws is None else ws
    rc = lib().mala_bwd(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), _view(o, _TIn), _view(do, _TIn),
                        lse.data_ptr(), _view(dq, _TOut), _view(dk, _TOut), _view(dv, _TOut),
                        ctypes.byref(st.c) if st else None, B, Hq, Hkv, N, d, int(causal), scale, tau,
                        ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_bwd")
    return dq, dk, dv, st


def fwd_chunk(q, k, v, scale: float, tau: float, causal: bool = True, stats: bool = False, out=None, lse=None):
    """mala_fwd_chunk: q [B,Nq,Hq,d] against k, v [B,Nk,Hkv,d] (causal: the queries are the last Nq positions).
    Returns (o [B,Nq,Hq,d] bf16, lse [B,Hq,Nq] fp32, Stats or None); the telemetry's query blocks follow the key
    positions (block i = rows q with 128 i <= q + (Nk - Nq) % 128 < 128 (i + 1))."""
    B, Nq, Hq, d = q.shape
    Nk, Hkv = k.shape[1], k.shape[2]
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq, Nq), dtype=torch.float32, device=q.device) if lse is None else lse
    Tq, Tk = -(-(Nq + ((Nk - Nq) % 128 if causal else 0)) // 128), -(-Nk // 128)
    st = Stats((B, Hq, Tq), -(-Tk // 32), q.device) if stats else None
    rc = lib().mala_fwd_chunk(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), _view(o, _TOut), lse.data_ptr(),
                              ctypes.byref(st.c) if st else None, B, Hq, Hkv, Nq, Nk, d, int(causal), scale, tau,
                              None, 0, _stream())
    if rc != 0:
        raise MalaError(rc, "mala_fwd_chunk")
    return o, lse, st


def fwd_chunk_split(q, k, v, scale: float, tau: float, num_splits: int, causal: bool = True, stats: bool = False,
                    out=None, lse=None, ws=None):
    """mala_fwd_chunk_split: mala_fwd_chunk with the keys cut into num_splits ranges (split-local test, merged)."""
    B, Nq, Hq, d = q.shape
    Nk, Hkv = k.shape[1], k.shape[2]
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq, Nq), dtype=torch.float32, device=q.device) if lse is None else lse
    Tq, Tk = -(-(Nq + ((Nk - Nq) % 128 if causal else 0)) // 128), -(-Nk // 128)
    st = Stats((B, Hq, Tq), -(-Tk // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_FWD, B, Hq, Hkv, Nq, d, num_splits), q.device) if ws is None else ws
    rc = lib().mala_fwd_chunk_split(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), _view(o, _TOut), lse.data_ptr(),
                                    ctypes.byref(st.c) if st else None, B, Hq, Hkv, Nq, Nk, d, int(causal), scale, tau,
                                    num_splits, ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_fwd_chunk_split")
    return o, lse, st


def bwd_chunk(q, k, v, o, do, lse, scale: float, tau: float, causal: bool = True, stats: bool = False, ws=None,
              dq=None, dk=None, dv=None):
    """mala_bwd_chunk: returns (dq [B,Nq,Hq,d], dk, dv [B,Nk,Hkv,d], Stats or None)."""
    B, Nq, Hq, d = q.shape
    Nk, Hkv = k.shape[1], k.shape[2]
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    shift = (Nk - Nq) % 128 if causal and Nk >= Nq else 0     # query blocks follow the positions
    Tq, Tk = -(-(Nq + shift) // 128), -(-Nk // 128)
    st = Stats((B, Hq, Tk), -(-Tq // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_BWD, B, Hq, Hkv, Nq + shift, d), q.device) if ws is None else ws
    rc = lib().mala_bwd_chunk(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), _view(o, _TIn), _view(do, _TIn),
                              lse.data_ptr(), _view(dq, _TOut), _view(dk, _TOut), _view(dv, _TOut),
                              ctypes.byref(st.c) if st else None, B, Hq, Hkv, Nq, Nk, d, int(causal), scale, tau,
                              ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_bwd_chunk")
    return dq, dk, dv, st


def fwd_varlen(q, k, v, cu_seqlens, max_seqlen: int, scale: float, tau: float, causal: bool = True, stats: bool = False):
    """mala_fwd_varlen: q [1,total,Hq,d], k, v [1,total,Hkv,d] packed sequences; cu_seqlens int32 [B+1] on the device.
    Returns (o [1,total,Hq,d] bf16, lse [Hq,total] fp32, Stats or None)."""
    one, total, Hq, d = q.shape
    assert one == 1 and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    B, Hkv = cu_seqlens.numel() - 1, k.shape[2]
    o = torch.empty_like(q)
    lse = torch.empty((Hq, total), dtype=torch.float32, device=q.device)
    T = -(-max_seqlen // 128)
    st = Stats((B, Hq, T), -(-T // 32), q.device) if stats else None
    rc = lib().mala_fwd_varlen(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), cu_seqlens.data_ptr(), _view(o, _TOut),
                               lse.data_ptr(), ctypes.byref(st.c) if st else None, B, Hq, Hkv, total, max_seqlen, d,
                               int(causal), scale, tau, None, 0, _stream())
    if rc != 0:
        raise MalaError(rc, "mala_fwd_varlen")
    return o, lse, st


def fwd_varlen_prefix(q, k, v, cu_seqlens_q, cu_seqlens_k, max_seqlen_q: int, max_seqlen_k: int, scale: float, tau: float,
                      causal: bool = True, stats: bool = False):
    """mala_fwd_varlen_prefix: packed q [1,total_q,Hq,d] against packed k, v [1,total_k,Hkv,d], every sequence with at
    least as many keys as queries.  Returns (o, lse [Hq,total_q], Stats or None)."""
    one, total_q, Hq, d = q.shape
    total_k, Hkv = k.shape[1], k.shape[2]
    B = cu_seqlens_q.numel() - 1
    o = torch.empty_like(q)
    lse = torch.empty((Hq, total_q), dtype=torch.float32, device=q.device)
    Tq, Tk = -(-(max_seqlen_q + 127) // 128), -(-max_seqlen_k // 128)
    st = Stats((B, Hq, Tq), -(-Tk // 32), q.device) if stats else None
    rc = lib().mala_fwd_varlen_prefix(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), cu_seqlens_q.data_ptr(),
                                      cu_seqlens_k.data_ptr(), _view(o, _TOut), lse.data_ptr(),
                                      ctypes.byref(st.c) if st else None, B, Hq, Hkv, total_q, total_k, max_seqlen_q,
                                      max_seqlen_k, d, int(causal), scale, tau, None, 0, _stream())
    if rc != 0:
        raise MalaError(rc, "mala_fwd_varlen_prefix")
    return o, lse, st


def fwd_paged(q, kpages, vpages, cu_seqlens_q, block_table, seqlens_k, max_seqlen_q: int, scale: float, tau: float,
              causal: bool = True, stats: bool = False):
    """mala_fwd_paged: packed q [1,total_q,Hq,d] against keys / values in pages [num_pages, page_size, Hkv, d]
    (block_table int32 [B, max_pages], seqlens_k int32 [B]).  Returns (o, lse [Hq,total_q], Stats or None)."""
    one, total_q, Hq, d = q.shape
    num_pages, page_size, Hkv = kpages.shape[0], kpages.shape[1], kpages.shape[2]
    B, max_pages = block_table.shape
    o = torch.empty_like(q)
    lse = torch.empty((Hq, total_q), dtype=torch.float32, device=q.device)
    Tq, Tk = -(-(max_seqlen_q + 127) // 128), -(-(max_pages * page_size) // 128)
    st = Stats((B, Hq, Tq), -(-Tk // 32), q.device) if stats else None
    rc = lib().mala_fwd_paged(_view(q, _TIn), _view(kpages, _TIn), _view(vpages, _TIn), cu_seqlens_q.data_ptr(),
                              block_table.data_ptr(), seqlens_k.data_ptr(), _view(o, _TOut), lse.data_ptr(),
                              ctypes.byref(st.c) if st else None, B, Hq, Hkv, total_q, max_seqlen_q, num_pages,
                              page_size, max_pages, d, int(causal), scale, tau, None, 0, _stream())
    if rc != 0:
        raise MalaError(rc, "mala_fwd_paged")
    return o, lse, st


def bwd_varlen(q, k, v, o, do, lse, cu_seqlens, max_seqlen: int, scale: float, tau: float, causal: bool = True,
               stats: bool = False, ws=None):
    """mala_bwd_varlen: returns (dq [1,total,Hq,d], dk, dv [1,total,Hkv,d], Stats or None)."""
    one, total, Hq, d = q.shape
    assert one == 1 and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    B, Hkv = cu_seqlens.numel() - 1, k.shape[2]
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    T = -(-max_seqlen // 128)
    st = Stats((B, Hq, T), -(-T // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_BWD, 1, Hq, Hkv, total + 128 * B, d), q.device) if ws is None else ws
    rc = lib().mala_bwd_varlen(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), _view(o, _TIn), _view(do, _TIn),
                               lse.data_ptr(), cu_seqlens.data_ptr(), _view(dq, _TOut), _view(dk, _TOut),
                               _view(dv, _TOut), ctypes.byref(st.c) if st else None, B, Hq, Hkv, total, max_seqlen, d,
                               int(causal), scale, tau, ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_bwd_varlen")
    return dq, dk, dv, st


def bwd_varlen_prefix(q, k, v, o, do, lse, cu_seqlens_q, cu_seqlens_k, max_seqlen_q: int, max_seqlen_k: int,
                      scale: float, tau: float, causal: bool = True, stats: bool = False, ws=None):
    """mala_bwd_varlen_prefix: returns (dq [1,total_q,Hq,d], dk, dv [1,total_k,Hkv,d], Stats or None)."""
    one, total_q, Hq, d = q.shape
    total_k, Hkv = k.shape[1], k.shape[2]
    for cu in (cu_seqlens_q, cu_seqlens_k):
        assert cu.dtype == torch.int32 and cu.is_contiguous()
    B = cu_seqlens_q.numel() - 1
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    Tq, Tk = -(-(max_seqlen_q + 127) // 128), -(-max_seqlen_k // 128)
    st = Stats((B, Hq, Tk), -(-Tq // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_BWD, 1, Hq, Hkv, total_q + 384 * B, d), q.device) if ws is None else ws
    rc = lib().mala_bwd_varlen_prefix(_view(q, _TIn), _view(k, _TIn), _view(v, _TIn), _view(o, _TIn), _view(do, _TIn),
                                      lse.data_ptr(), cu_seqlens_q.data_ptr(), cu_seqlens_k.data_ptr(),
                                      _view(dq, _TOut), _view(dk, _TOut), _view(dv, _TOut),
                                      ctypes.byref(st.c) if st else None, B, Hq, Hkv, total_q, total_k, max_seqlen_q,
                                      max_seqlen_k, d, int(causal), scale, tau, ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_bwd_varlen_prefix")
    return dq, dk, dv, st


def decode(q, kcache, vcache, scale: float, tau: float, num_splits: int, stats: bool = False, ws=None, out=None,
           want_lse: bool = True):
    """mala_decode: q [B,1,Hq,d]; returns (o [B,1,Hq,d] bf16, lse [B,Hq] fp32 or None, Stats or None)."""
    B, one, Hq, d = q.shape
    assert one == 1
    Nk, Hkv = kcache.shape[1], kcache.shape[2]
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    tps = -(-(-(-Nk // num_splits)) // 128)
    st = Stats((B, Hkv, num_splits), -(-tps // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_DECODE, B, Hq, Hkv, Nk, d, num_splits), q.device) if ws is None else ws
    rc = lib().mala_decode(_view(q, _TIn), _view(kcache, _TIn), _view(vcache, _TIn), _view(o, _TOut),
                           lse.data_ptr() if lse is not None else None, ctypes.byref(st.c) if st else None,
                           B, Hq, Hkv, Nk, d, scale, tau, num_splits, ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_decode")
    return o, lse, st


def _view8(t: torch.Tensor):
    assert t.dtype in (torch.uint8, torch.float8_e4m3fn) and t.dim() == 4 and t.stride(3) == 1, \
        "expects 8-bit [B,N,H,d], last dim contiguous"
    return _TIn(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def decode_fp8(q, kcache8, vcache8, kscale, vscale, scale: float, tau: float, num_splits: int, stats: bool = False,
               ws=None, out=None, want_lse: bool = True):
    """mala_decode_fp8: q [B,1,Hq,d] bf16; kcache8, vcache8 e4m3 codes [B,Nk,Hkv,d] (uint8 or float8_e4m3fn);
    kscale, vscale fp32 [B,Hkv,ceil(Nk/128)].  Returns (o [B,1,Hq,d] bf16, lse [B,Hq] fp32 or None, Stats or None)."""
    B, one, Hq, d = q.shape
    assert one == 1
    Nk, Hkv = kcache8.shape[1], kcache8.shape[2]
    assert kscale.dtype == torch.float32 and kscale.is_contiguous() and tuple(kscale.shape) == (B, Hkv, -(-Nk // 128))
    assert vscale.dtype == torch.float32 and vscale.is_contiguous() and tuple(vscale.shape) == (B, Hkv, -(-Nk // 128))
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    tps = -(-(-(-Nk // num_splits)) // 128)
    st = Stats((B, Hkv, num_splits), -(-tps // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_DECODE, B, Hq, Hkv, Nk, 128, num_splits), q.device) if ws is None else ws
    rc = lib().mala_decode_fp8(_view(q, _TIn), _view8(kcache8), _view8(vcache8), kscale.data_ptr(), vscale.data_ptr(),
                               _view(o, _TOut), lse.data_ptr() if lse is not None else None,
                               ctypes.byref(st.c) if st else None, B, Hq, Hkv, Nk, d, scale, tau, num_splits,
                               ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_decode_fp8")
    return o, lse, st


def decode_fp8_multi(q, kcache8, vcache8, kscale, vscale, scale: float, tau: float, num_splits: int, stats: bool = False,
                     ws=None, out=None, want_lse: bool = True):
    """mala_decode_fp8_multi: q [B,Sq,Hq,d] bf16, the Sq new tokens of each sequence (their keys / values are the last
    Sq positions of the caches); caches and scales as for decode_fp8.  Returns (o [B,Sq,Hq,d] bf16, lse [B,Sq,Hq]
    fp32 or None, Stats or None)."""
    B, Sq, Hq, d = q.shape
    Nk, Hkv = kcache8.shape[1], kcache8.shape[2]
    assert kscale.dtype == torch.float32 and kscale.is_contiguous() and tuple(kscale.shape) == (B, Hkv, -(-Nk // 128))
    assert vscale.dtype == torch.float32 and vscale.is_contiguous() and tuple(vscale.shape) == (B, Hkv, -(-Nk // 128))
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Sq, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    tps = -(-(-(-Nk // num_splits)) // 128)
    st = Stats((B, Hkv, num_splits), -(-tps // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_DECODE, B * Sq, Hq, Hkv, Nk, 128, num_splits), q.device) if ws is None else ws
    rc = lib().mala_decode_fp8_multi(_view(q, _TIn), _view8(kcache8), _view8(vcache8), kscale.data_ptr(), vscale.data_ptr(),
                                     _view(o, _TOut), lse.data_ptr() if lse is not None else None,
                                     ctypes.byref(st.c) if st else None, B, Hq, Hkv, Nk, Sq, d, scale, tau, num_splits,
                                     ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_decode_fp8_multi")
    return o, lse, st


def decode_fp8_paged(q, kpages8, vpages8, kscale, vscale, block_table, seqlens, scale: float, tau: float, num_splits: int,
                     stats: bool = False, ws=None, out=None, want_lse: bool = True):
    """mala_decode_fp8_paged: q [B,1,Hq,d] bf16; kpages8, vpages8 e4m3 codes [num_pages, page_size, Hkv, d];
    kscale, vscale fp32 [num_pages, Hkv, max(1, page_size/128)]; block_table int32 [B, max_pages_per_seq]; seqlens int32 [B] or
    None.  Returns (o [B,1,Hq,d] bf16, lse [B,Hq] fp32 or None, Stats or None)."""
    B, one, Hq, d = q.shape
    assert one == 1
    num_pages, page_size, Hkv = kpages8.shape[0], kpages8.shape[1], kpages8.shape[2]
    assert block_table.dtype == torch.int32 and block_table.is_contiguous() and block_table.shape[0] == B
    assert seqlens is None or (seqlens.dtype == torch.int32 and seqlens.is_contiguous() and seqlens.shape == (B,))
    for t in (kscale, vscale):
        assert t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (num_pages, Hkv, max(1, page_size // 128))
    max_pages = block_table.shape[1]
    Nk = max_pages * page_size
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    tps = -(-(-(-Nk // num_splits)) // 128)
    st = Stats((B, Hkv, num_splits), -(-tps // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_DECODE, B, Hq, Hkv, Nk, 128, num_splits), q.device) if ws is None else ws
    rc = lib().mala_decode_fp8_paged(_view(q, _TIn), _view8(kpages8), _view8(vpages8), kscale.data_ptr(),
                                     vscale.data_ptr(), block_table.data_ptr(),
                                     seqlens.data_ptr() if seqlens is not None else None, _view(o, _TOut),
                                     lse.data_ptr() if lse is not None else None, ctypes.byref(st.c) if st else None,
                                     B, Hq, Hkv, num_pages, page_size, max_pages, d, scale, tau, num_splits,
                                     ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_decode_fp8_paged")
    return o, lse, st


def decode_multi(q, kcache, vcache, scale: float, tau: float, num_splits: int, stats: bool = False, ws=None, out=None,
                 want_lse: bool = True):
    """mala_decode_multi: q [B,Sq,Hq,d], the Sq new tokens of each sequence (their keys / values are the last Sq
    positions of the caches).  Returns (o [B,Sq,Hq,d] bf16, lse [B,Sq,Hq] fp32 or None, Stats or None)."""
    B, Sq, Hq, d = q.shape
    Nk, Hkv = kcache.shape[1], kcache.shape[2]
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Sq, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    tps = -(-(-(-Nk // num_splits)) // 128)
    st = Stats((B, Hkv, num_splits), -(-tps // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_DECODE, B * Sq, Hq, Hkv, Nk, d, num_splits), q.device) if ws is None else ws
    rc = lib().mala_decode_multi(_view(q, _TIn), _view(kcache, _TIn), _view(vcache, _TIn), _view(o, _TOut),
                                 lse.data_ptr() if lse is not None else None, ctypes.byref(st.c) if st else None,
                                 B, Hq, Hkv, Nk, Sq, d, scale, tau, num_splits, ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_decode_multi")
    return o, lse, st


def decode_paged(q, kpages, vpages, block_table, seqlens, scale: float, tau: float, num_splits: int,
                 stats: bool = False, ws=None, out=None, want_lse: bool = True):
    """mala_decode_paged: q [B,Sq,Hq,d] (Sq new tokens per sequence); kpages, vpages [num_pages, page_size, Hkv, d];
    block_table int32 [B, max_pages_per_seq]; seqlens int32 [B] or None.
    Returns (o [B,Sq,Hq,d], lse [B,Hq] (Sq = 1) or [B,Sq,Hq] or None, Stats or None)."""
    B, Sq, Hq, d = q.shape
    num_pages, page_size, Hkv = kpages.shape[0], kpages.shape[1], kpages.shape[2]
    assert block_table.dtype == torch.int32 and block_table.is_contiguous() and block_table.shape[0] == B
    assert seqlens is None or (seqlens.dtype == torch.int32 and seqlens.is_contiguous() and seqlens.shape == (B,))
    max_pages = block_table.shape[1]
    Nk = max_pages * page_size
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq) if Sq == 1 else (B, Sq, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    tps = -(-(-(-Nk // num_splits)) // 128)
    st = Stats((B, Hkv, num_splits), -(-tps // 32), q.device) if stats else None
    ws = _ws(workspace_bytes(OP_DECODE, B * Sq, Hq, Hkv, Nk, d, num_splits), q.device) if ws is None else ws
    rc = lib().mala_decode_paged(_view(q, _TIn), _view(kpages, _TIn), _view(vpages, _TIn), block_table.data_ptr(),
                                 seqlens.data_ptr() if seqlens is not None else None, _view(o, _TOut),
                                 lse.data_ptr() if lse is not None else None, ctypes.byref(st.c) if st else None,
                                 B, Hq, Hkv, num_pages, page_size, max_pages, Sq, d, scale, tau, num_splits,
                                 ws.data_ptr(), ws.numel(), _stream())
    if rc != 0:
        raise MalaError(rc, "mala_decode_paged")
    return o, lse, st


STATIC_SCRATCH_BYTES = 24 << 20


def decode_static(q, kcache, vcache, scale: float, tau: float, num_splits: int, out=None, want_lse: bool = True):
    """mala_decode_static: decode without any caller-provided scratch.

    For callers that cannot allocate device memory at the point of the call (a fixed memory plan, a plug-in
    that only receives its inputs and outputs, a path that must not touch the allocator).  The split partials
    live in a 24 MiB array inside the library image; calls on one device must not overlap on the GPU.  Only
    the output tensors are created here when the caller does not pass them.
    Returns (o [B,1,Hq,d] bf16, lse [B,Hq] fp32 or None)."""
    B, one, Hq, d = q.shape
    assert one == 1
    Nk, Hkv = kcache.shape[1], kcache.shape[2]
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if want_lse else None
    rc = lib().mala_decode_static(_view(q, _TIn), _view(kcache, _TIn), _view(vcache, _TIn), _view(o, _TOut),
                                  lse.data_ptr() if lse is not None else None, B, Hq, Hkv, Nk, d, scale, tau,
                                  num_splits, _stream())
    if rc != 0:
        raise MalaError(rc, "mala_decode_static")
    return o, lse
