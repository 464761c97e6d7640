"""ctypes front end of the fp64 MALA oracle (``mala_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module; the
product path never does.  The C functions work on ONE query head and its key/value head, exactly
as the paper's Methodology section writes the operator; this file adds nothing but the batch /
head loops (contiguous GQA groups: ``h_kv = h_q // (Hq // Hkv)``), the summation of dK, dV over
the query heads that share a KV head, and array marshalling.

Tensors are ``[B, N, H, d]`` (torch tensors of any float dtype, or numpy arrays); every head slice
is widened to float64 before it reaches C.  lse / D are ``[B, Hq, N]``.  Tile masks use the C
encoding: 0 = not legal, 1 = skipped, 2 = retained; ``crit`` is the tile criterion C (skip iff
C < 0), NaN where not legal.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mala_oracle.c")
_LIB = os.path.join(_HERE, "libmala_oracle.so")
_lib = None

ILLEGAL, SKIPPED, RETAINED = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.check_call(cmd)
    return _LIB


_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int)
_U8 = ctypes.POINTER(ctypes.c_uint8)
_ci, _cd = ctypes.c_int, ctypes.c_double


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.mala_oracle_threads.restype = _ci
        L.mala_oracle_dense_fwd.argtypes = [_D, _D, _D, _ci, _ci, _ci, _cd, _ci, _ci, _ci, _D, _D]
        L.mala_oracle_dense_bwd.argtypes = [_D, _D, _D, _D, _ci, _ci, _cd, _ci, _D, _D, _D]
        L.mala_oracle_fwd.argtypes = [_D, _D, _D, _ci, _ci, _ci, _cd, _cd, _ci, _ci, _ci, _ci, _I, _D, _D, _U8, _D]
        L.mala_oracle_fwd_split.argtypes = [_D, _D, _D, _ci, _ci, _ci, _cd, _cd, _ci, _ci, _ci, _ci, _ci, _ci, _I, _D, _D,
                                            _U8, _D]
        L.mala_oracle_bwd_D.argtypes = [_D, _D, _ci, _ci, _D]
        L.mala_oracle_bwd.argtypes = [_D, _D, _D, _D, _D, _D, _ci, _ci, _ci, _cd, _cd, _ci, _ci, _ci, _ci, _ci, _I,
                                      _D, _D, _D, _U8, _D]
        L.mala_oracle_bwd_dq.argtypes = [_D, _D, _D, _D, _D, _D, _ci, _ci, _ci, _cd, _cd, _ci, _ci, _ci, _ci, _ci, _I,
                                         _D]
        L.mala_oracle_decode_tiles_per_split.argtypes = [_ci, _ci, _ci]
        L.mala_oracle_decode_splits.argtypes = [_D, _D, _D, _ci, _ci, _ci, _cd, _cd, _ci, _ci, _D, _D, _U8, _D]
        L.mala_oracle_decode_splits_tps.argtypes = [_D, _D, _D, _ci, _ci, _ci, _cd, _cd, _ci, _ci, _ci, _D, _D, _U8, _D]
        L.mala_oracle_decode_splits_rows.argtypes = [_D, _D, _D, _ci, _ci, _ci, _cd, _cd, _ci, _ci, _ci, _I, _D, _D,
                                                     _U8, _D]
        L.mala_oracle_decode_merge.argtypes = [_D, _D, _ci, _ci, _ci, _D, _D]
        for f in ("mala_oracle_dense_fwd", "mala_oracle_dense_bwd", "mala_oracle_fwd", "mala_oracle_fwd_split",
                  "mala_oracle_bwd_D",
                  "mala_oracle_bwd", "mala_oracle_bwd_dq", "mala_oracle_decode_tiles_per_split",
                  "mala_oracle_decode_splits", "mala_oracle_decode_splits_tps", "mala_oracle_decode_splits_rows",
                  "mala_oracle_decode_merge"):
            getattr(L, f).restype = _ci
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().mala_oracle_threads())


def _np(x) -> np.ndarray:
    """float64 contiguous numpy copy of a torch tensor / numpy array (exact for bf16, fp32)."""
    if hasattr(x, "detach"):
        import torch
        x = x.detach().cpu().to(torch.float64).numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _head(x, b: int, h: int) -> np.ndarray:
    return _np(x[b, :, h, :])


def _p(a: np.ndarray):
    return a.ctypes.data_as(_D)


def _ip(a):
    return a.ctypes.data_as(_I) if a is not None else None


def _u8(a: np.ndarray):
    return a.ctypes.data_as(_U8)


def _ck(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what} rejected its arguments (rc={rc})")


def dense_fwd(q, k, v, scale: float, causal: bool = True):
    """FullAttn by its definition (causal with fewer queries than keys: the queries are the last positions).
    Returns o [B,N,Hq,d], lse [B,Hq,N]."""
    B, N, Hq, d = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    o = np.zeros((B, N, Hq, d))
    lse = np.zeros((B, Hq, N))
    for b in range(B):
        for h in range(Hq):
            Q, K, V = _head(q, b, h), _head(k, b, h // G), _head(v, b, h // G)
            O = np.zeros((N, d))
            _ck(lib().mala_oracle_dense_fwd(_p(Q), _p(K), _p(V), N, K.shape[0], d, scale, int(causal), 0, N,
                                            _p(O), _p(lse[b, h])), "dense_fwd")
            o[b, :, h, :] = O
    return o, lse


def dense_bwd(q, k, v, do, scale: float, causal: bool = True):
    """FullAttn gradients by the closed forms.  Returns dq [B,N,Hq,d], dk, dv [B,N,Hkv,d]."""
    B, N, Hq, d = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    dq = np.zeros((B, N, Hq, d))
    dk = np.zeros((B, N, Hkv, d))
    dv = np.zeros((B, N, Hkv, d))
    for b in range(B):
        for h in range(Hq):
            Q, K, V, dO = _head(q, b, h), _head(k, b, h // G), _head(v, b, h // G), _head(do, b, h)
            a, c, e = np.zeros((N, d)), np.zeros((N, d)), np.zeros((N, d))
            _ck(lib().mala_oracle_dense_bwd(_p(Q), _p(K), _p(V), _p(dO), N, d, scale, int(causal), _p(a), _p(c),
                                            _p(e)), "dense_bwd")
            dq[b, :, h, :] = a
            dk[b, :, h // G, :] += c
            dv[b, :, h // G, :] += e
    return dq, dk, dv


def fwd(q, k, v, scale: float, tau: float, Bq: int, Bk: int, causal: bool = True, units=None, num_splits: int = 1,
        q_shift: int = 0):
    """Algorithm 1.  ``units``: optional list of (b, h_q, i) query blocks; rows of other blocks stay NaN.
    ``num_splits`` > 1: the key blocks are cut into that many contiguous ranges of ceil(Tc / num_splits) blocks,
    each range runs the rule on its own state and the results are merged by their log-normalizers.
    ``q_shift`` (0 <= q_shift < Bq): the query blocks are laid out as if q_shift more rows preceded the first one
    (block i = rows q with i*Bq <= q + q_shift < (i+1)*Bq); with q_shift = (Nk - N) % Bq a chunk's blocks are the
    blocks its rows have in the equal-length problem over all Nk positions.

    q [B,N,Hq,d]; k, v [B,Nk,Hkv,d] with Nk >= N: the queries are the last N of the Nk positions (chunked
    prefill), query row q sees the keys 0 .. q + Nk - N and L_q = q + 1 + Nk - N.
    Returns dict(o [B,N,Hq,d], lse [B,Hq,N], mask [B,Hq,Tr,Tc] uint8, crit [B,Hq,Tr,Tc]).
    """
    B, N, Hq, d = q.shape
    Nk, Hkv = k.shape[1], k.shape[2]
    G = Hq // Hkv
    Tr, Tc = -(-(N + q_shift) // Bq), -(-Nk // Bk)
    o = np.full((B, N, Hq, d), np.nan)
    lse = np.full((B, Hq, N), np.nan)
    mask = np.zeros((B, Hq, Tr, Tc), dtype=np.uint8)
    crit = np.full((B, Hq, Tr, Tc), np.nan)
    heads = {}
    if units is None:
        for b in range(B):
            for h in range(Hq):
                heads[(b, h)] = None
    else:
        for (b, h, i) in units:
            heads.setdefault((b, h), []).append(int(i))
    for (b, h), blocks in heads.items():
        Q, K, V = _head(q, b, h), _head(k, b, h // G), _head(v, b, h // G)
        O = np.full((N, d), np.nan)
        l = np.full((N,), np.nan)
        m = np.zeros((Tr, Tc), dtype=np.uint8)
        c = np.full((Tr, Tc), np.nan)
        bl = np.asarray(blocks, dtype=np.int32) if blocks is not None else None
        _ck(lib().mala_oracle_fwd_split(_p(Q), _p(K), _p(V), N, Nk, d, scale, tau, Bq, Bk, int(causal), num_splits,
                                        q_shift, 0 if bl is None else len(bl), _ip(bl), _p(O), _p(l), _u8(m), _p(c)),
            "fwd")
        o[b, :, h, :] = O
        lse[b, h] = l
        mask[b, h] = m
        crit[b, h] = c
    return dict(o=o, lse=lse, mask=mask, crit=crit)


def bwd(q, k, v, o, do, lse, scale: float, tau: float, Bq: int, Bk: int, causal: bool = True,
        key_units=None, dq_units=None, q_shift: int = 0):
    """Algorithm 2 with the given forward output ``o`` and saved ``lse``.

    Full run (both unit lists None): dq, dk, dv complete.  With ``key_units`` = [(b, h_kv, j)] only
    those key blocks are run: their dK/dV rows (summed over the group's query heads) are exact and
    everything else is NaN.  With ``dq_units`` = [(b, h_q, i)] the dQ rows of those query blocks are
    computed from all their legal key blocks.  Fewer queries than keys and ``q_shift``: as in ``fwd``
    (query block i = rows q with i*Bq <= q + q_shift < (i+1)*Bq; Tr = ceil((N + q_shift)/Bq)).
    Returns dict(dq, dk, dv, mask [B,Hq,Tc,Tr], crit [B,Hq,Tc,Tr]).
    """
    B, N, Hq, d = q.shape
    Nk, Hkv = k.shape[1], k.shape[2]
    G = Hq // Hkv
    Tr, Tc = -(-(N + q_shift) // Bq), -(-Nk // Bk)
    full = key_units is None and dq_units is None
    dq = np.zeros((B, N, Hq, d)) if full else np.full((B, N, Hq, d), np.nan)
    dk = np.zeros((B, Nk, Hkv, d)) if full else np.full((B, Nk, Hkv, d), np.nan)
    dv = np.zeros((B, Nk, Hkv, d)) if full else np.full((B, Nk, Hkv, d), np.nan)
    mask = np.zeros((B, Hq, Tc, Tr), dtype=np.uint8)
    crit = np.full((B, Hq, Tc, Tr), np.nan)

    def head_inputs(b, h):
        Q, K, V, dO = _head(q, b, h), _head(k, b, h // G), _head(v, b, h // G), _head(do, b, h)
        O = _head(o, b, h)
        l = _np(lse[b, h])
        D = np.zeros((N,))
        lib().mala_oracle_bwd_D(_p(O), _p(dO), N, d, _p(D))
        return Q, K, V, dO, l, D

    groups = {}
    if full:
        for b in range(B):
            for g in range(Hkv):
                groups[(b, g)] = None
    elif key_units is not None:
        for (b, g, j) in key_units:
            groups.setdefault((b, g), []).append(int(j))
    for (b, g), blocks in groups.items():
        bl = np.asarray(blocks, dtype=np.int32) if blocks is not None else None
        rows = None
        if bl is not None:
            rows = np.concatenate([np.arange(j * Bk, min(Nk, (j + 1) * Bk)) for j in bl])
            dk[b, rows, g, :] = 0.0
            dv[b, rows, g, :] = 0.0
        for h in range(g * G, (g + 1) * G):
            Q, K, V, dO, l, D = head_inputs(b, h)
            a = np.zeros((N, d))
            c = np.zeros((Nk, d))
            e = np.zeros((Nk, d))
            m = np.zeros((Tc, Tr), dtype=np.uint8)
            cr = np.full((Tc, Tr), np.nan)
            _ck(lib().mala_oracle_bwd(_p(Q), _p(K), _p(V), _p(dO), _p(l), _p(D), N, Nk, d, scale, tau, Bq, Bk,
                                      int(causal), q_shift, 0 if bl is None else len(bl), _ip(bl),
                                      _p(a) if full else None, _p(c), _p(e), _u8(m), _p(cr)), "bwd")
            if full:
                dq[b, :, h, :] = a
                dk[b, :, g, :] += c
                dv[b, :, g, :] += e
                mask[b, h] = m
                crit[b, h] = cr
            else:
                dk[b, rows, g, :] += c[rows]
                dv[b, rows, g, :] += e[rows]
                mask[b, h, bl] = m[bl]
                crit[b, h, bl] = cr[bl]
    if dq_units is not None:
        heads = {}
        for (b, h, i) in dq_units:
            heads.setdefault((b, h), []).append(int(i))
        for (b, h), blocks in heads.items():
            bl = np.asarray(blocks, dtype=np.int32)
            Q, K, V, dO, l, D = head_inputs(b, h)
            a = np.full((N, d), np.nan)
            _ck(lib().mala_oracle_bwd_dq(_p(Q), _p(K), _p(V), _p(dO), _p(l), _p(D), N, Nk, d, scale, tau, Bq, Bk,
                                         int(causal), q_shift, len(bl), _ip(bl), _p(a)), "bwd_dq")
            rows = np.concatenate([np.arange(max(0, i * Bq - q_shift), min(N, (i + 1) * Bq - q_shift)) for i in bl])
            dq[b, rows, h, :] = a[rows]
    return dict(dq=dq, dk=dk, dv=dv, mask=mask, crit=crit)


def decode(q, kcache, vcache, scale: float, tau: float, num_splits: int, Bk: int, units=None,
           packed_rows: bool = True):
    """Split-KV decode of one new token per sequence.

    q [B,Hq,d] (or [B,1,Hq,d]); caches [B,Nk,Hkv,d].  ``units``: optional list of (b, h_kv); other
    entries stay NaN.  ``packed_rows``: the Hq/Hkv query heads of one KV head form the rows of one
    tile (one row that needs a tile retains it for all); False runs every query head alone.
    Returns dict(o [B,Hq,d], lse [B,Hq], mask [B,Hkv,S,tps] (packed) or [B,Hq,S,tps], crit, o_part, lse_part).
    """
    if len(q.shape) == 4:
        q = q[:, 0]
    B, Hq, d = q.shape
    Nk, Hkv = kcache.shape[1], kcache.shape[2]
    G = Hq // Hkv
    tps = int(lib().mala_oracle_decode_tiles_per_split(Nk, num_splits, Bk))
    o = np.full((B, Hq, d), np.nan)
    lse = np.full((B, Hq), np.nan)
    nm = Hkv if packed_rows else Hq
    mask = np.zeros((B, nm, num_splits, tps), dtype=np.uint8)
    crit = np.full((B, nm, num_splits, tps), np.nan)
    o_part = np.full((B, Hq, num_splits, d), np.nan)
    lse_part = np.full((B, Hq, num_splits), np.nan)
    if units is None:
        units = [(b, g) for b in range(B) for g in range(Hkv)]
    for (b, g) in units:
        K, V = _head(kcache, b, g), _head(vcache, b, g)
        row_sets = [list(range(g * G, (g + 1) * G))] if packed_rows else [[h] for h in range(g * G, (g + 1) * G)]
        for hs in row_sets:
            R = len(hs)
            Q = _np(q[b, hs[0]:hs[-1] + 1, :])
            op = np.zeros((num_splits, R, d))
            lp = np.zeros((num_splits, R))
            m = np.zeros((num_splits, tps), dtype=np.uint8)
            c = np.full((num_splits, tps), np.nan)
            _ck(lib().mala_oracle_decode_splits(_p(Q), _p(K), _p(V), R, Nk, d, scale, tau, num_splits, Bk, _p(op),
                                                _p(lp), _u8(m), _p(c)), "decode_splits")
            oo = np.zeros((R, d))
            ll = np.zeros((R,))
            _ck(lib().mala_oracle_decode_merge(_p(op), _p(lp), num_splits, R, d, _p(oo), _p(ll)), "decode_merge")
            o[b, hs[0]:hs[-1] + 1] = oo
            lse[b, hs[0]:hs[-1] + 1] = ll
            o_part[b, hs[0]:hs[-1] + 1] = op.transpose(1, 0, 2)
            lse_part[b, hs[0]:hs[-1] + 1] = lp.T
            mi = g if packed_rows else hs[0]
            mask[b, mi] = m
            crit[b, mi] = c
    return dict(o=o, lse=lse, mask=mask, crit=crit, o_part=o_part, lse_part=lse_part)


def decode_paged(q, kpages, vpages, block_table, seqlens, scale: float, tau: float, num_splits: int, Bk: int,
                 units=None):
    """Split-KV decode over a paged cache with one length per sequence.

    q [B,Hq,d] or [B,Sq,Hq,d] (Sq new tokens per sequence, whose keys are the last Sq of the sequence's keys);
    kpages, vpages [num_pages, page_size, Hkv, d]; block_table [B, max_pages] (page of the keys page_size*x ..);
    seqlens [B] (None: every sequence holds max_pages*page_size keys).
    The cache of sequence b is put together page by page and cut off at its length n; the decode rule then runs on
    it: token s sees the keys before position n - Sq + s + 1, which is also its L.  All sequences share one layout of
    splits over the key positions, the one ``decode`` derives for N_k = max_pages*page_size.  ``units``: optional
    list of (b, h_kv), other entries stay zero.
    Returns dict(o [B,Sq,Hq,d] ([B,Hq,d] for a 3-d q), lse, mask [B,Hkv,S,tps], crit, lse_part [B,Sq,Hq,S] / [B,Hq,S]).
    """
    squeeze = len(q.shape) == 3
    if squeeze:
        q = q[:, None]
    B, Sq, Hq, d = q.shape
    page_size, Hkv = kpages.shape[1], kpages.shape[2]
    G = Hq // Hkv
    R = Sq * G
    bt = np.asarray(block_table, dtype=np.int64)
    max_pages = bt.shape[1]
    Nmax = max_pages * page_size
    lens = np.full((B,), Nmax, dtype=np.int64) if seqlens is None else np.asarray(seqlens, dtype=np.int64)
    tps = int(lib().mala_oracle_decode_tiles_per_split(Nmax, num_splits, Bk))
    o = np.zeros((B, Sq, Hq, d))
    lse = np.zeros((B, Sq, Hq))
    mask = np.zeros((B, Hkv, num_splits, tps), dtype=np.uint8)
    crit = np.full((B, Hkv, num_splits, tps), np.nan)
    lse_part = np.zeros((B, Sq, Hq, num_splits))
    if units is None:
        units = [(b, g) for b in range(B) for g in range(Hkv)]
    for (b, g) in units:
        n = int(min(max(lens[b], 0), Nmax))
        npg = -(-n // page_size)
        K = np.concatenate([_np(kpages[int(bt[b, x]), :, g, :]) for x in range(npg)], axis=0)[:n] \
            if npg else np.zeros((1, d))
        V = np.concatenate([_np(vpages[int(bt[b, x]), :, g, :]) for x in range(npg)], axis=0)[:n] \
            if npg else np.zeros((1, d))
        K, V = np.ascontiguousarray(K), np.ascontiguousarray(V)
        Q = np.ascontiguousarray(_np(q[b, :, g * G:(g + 1) * G, :]).reshape(R, d))
        vis = np.ascontiguousarray(np.repeat(n - Sq + 1 + np.arange(Sq), G).astype(np.int32))
        op = np.zeros((num_splits, R, d))
        lp = np.zeros((num_splits, R))
        m = np.zeros((num_splits, tps), dtype=np.uint8)
        c = np.full((num_splits, tps), np.nan)
        _ck(lib().mala_oracle_decode_splits_rows(_p(Q), _p(K), _p(V), R, n, d, scale, tau, num_splits, tps, Bk,
                                                 _ip(vis), _p(op), _p(lp), _u8(m), _p(c)), "decode_splits_rows")
        oo = np.zeros((R, d))
        ll = np.zeros((R,))
        _ck(lib().mala_oracle_decode_merge(_p(op), _p(lp), num_splits, R, d, _p(oo), _p(ll)), "decode_merge")
        o[b, :, g * G:(g + 1) * G] = oo.reshape(Sq, G, d)
        lse[b, :, g * G:(g + 1) * G] = ll.reshape(Sq, G)
        lse_part[b, :, g * G:(g + 1) * G] = lp.T.reshape(Sq, G, num_splits)
        mask[b, g] = m
        crit[b, g] = c
    if squeeze:
        o, lse, lse_part = o[:, 0], lse[:, 0], lse_part[:, 0]
    return dict(o=o, lse=lse, mask=mask, crit=crit, lse_part=lse_part)


def decode_multi(q, kcache, vcache, scale: float, tau: float, num_splits: int, Bk: int, units=None):
    """Split-KV decode of Sq new tokens per sequence (their keys and values are the last Sq cache positions).

    q [B,Sq,Hq,d]; caches [B,Nk,Hkv,d].  Token s sits at position Nk - Sq + s, sees the keys up to its own position
    and has L = Nk - Sq + s + 1.  The Sq * Hq/Hkv rows of a KV head form one tile, row s * G + g.
    Returns dict(o [B,Sq,Hq,d], lse [B,Sq,Hq], mask [B,Hkv,S,tps], crit, lse_part [B,Sq,Hq,S]).
    """
    B, Sq, Hq, d = q.shape
    Nk, Hkv = kcache.shape[1], kcache.shape[2]
    G = Hq // Hkv
    R = Sq * G
    tps = int(lib().mala_oracle_decode_tiles_per_split(Nk, num_splits, Bk))
    o = np.zeros((B, Sq, Hq, d))
    lse = np.zeros((B, Sq, Hq))
    mask = np.zeros((B, Hkv, num_splits, tps), dtype=np.uint8)
    crit = np.full((B, Hkv, num_splits, tps), np.nan)
    lse_part = np.zeros((B, Sq, Hq, num_splits))
    vis = np.ascontiguousarray(np.repeat(Nk - Sq + 1 + np.arange(Sq), G).astype(np.int32))
    if units is None:
        units = [(b, g) for b in range(B) for g in range(Hkv)]
    for (b, g) in units:
        K, V = _head(kcache, b, g), _head(vcache, b, g)
        Q = np.ascontiguousarray(_np(q[b, :, g * G:(g + 1) * G, :]).reshape(R, d))
        op = np.zeros((num_splits, R, d))
        lp = np.zeros((num_splits, R))
        m = np.zeros((num_splits, tps), dtype=np.uint8)
        c = np.full((num_splits, tps), np.nan)
        _ck(lib().mala_oracle_decode_splits_rows(_p(Q), _p(K), _p(V), R, Nk, d, scale, tau, num_splits, tps, Bk,
                                                 _ip(vis), _p(op), _p(lp), _u8(m), _p(c)), "decode_splits_rows")
        oo = np.zeros((R, d))
        ll = np.zeros((R,))
        _ck(lib().mala_oracle_decode_merge(_p(op), _p(lp), num_splits, R, d, _p(oo), _p(ll)), "decode_merge")
        o[b, :, g * G:(g + 1) * G] = oo.reshape(Sq, G, d)
        lse[b, :, g * G:(g + 1) * G] = ll.reshape(Sq, G)
        lse_part[b, :, g * G:(g + 1) * G] = lp.T.reshape(Sq, G, num_splits)
        mask[b, g] = m
        crit[b, g] = c
    return dict(o=o, lse=lse, mask=mask, crit=crit, lse_part=lse_part)
