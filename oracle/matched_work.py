"""Matched-work diagnostics of the forward allocation (appendix "Normalized-Mass Allocation at Matched Work Setup")
-- TEST INFRASTRUCTURE / ANALYSIS ONLY, fp64 numpy on top of the oracle; the product path never imports it.

For every allocation decision (batch entry, query head, query block) the forward oracle retains some number of key
tiles.  The diagnostic controls spend tile budgets on the tiles that carry the most probability mass under the dense
(screening-disabled) softmax, ranked at the same granularity, and differ only in the budget each decision gets:

  per-instance   exactly the number of tiles MALA retained for that decision;
  static         MALA's count averaged over the batch entries, per (head, block position);
  position-only  MALA's count averaged over batch entries and heads, per block position.

Averages are turned into integer budgets by largest-remainder rounding inside each averaging group, so that all
policies spend exactly the same total number of tiles.  Omitted mass of a row = 1 - (dense probability mass of the
row's retained tiles) = 1 - exp(lse_screened - lse_reference).
"""
from __future__ import annotations

import numpy as np

from . import mala_oracle as orc


def dense_tile_mass(Q, K, scale: float, Bq: int, Bk: int, off: int):
    """Dense causal softmax of one head, summed per key tile: [N, Tc] (row q sees the keys 0 .. q + off)."""
    N, Nk = Q.shape[0], K.shape[0]
    S = scale * (Q @ K.T)
    S[np.arange(Nk)[None, :] > (np.arange(N)[:, None] + off)] = -np.inf
    P = np.exp(S - S.max(axis=1, keepdims=True))
    P /= P.sum(axis=1, keepdims=True)
    Tc = -(-Nk // Bk)
    return np.stack([P[:, j * Bk:(j + 1) * Bk].sum(axis=1) for j in range(Tc)], axis=1)


def _largest_remainder(avg: np.ndarray, total: int, cap: np.ndarray) -> np.ndarray:
    """Integers close to `avg` (same shape), none above `cap`, that sum to `total`."""
    base = np.minimum(np.floor(avg).astype(np.int64), cap)
    rest = int(total - base.sum())
    order = np.argsort(-(avg - np.floor(avg)).ravel(), kind="stable")
    flat, capf = base.ravel(), cap.ravel()
    while rest > 0:
        moved = False
        for x in order:
            if rest > 0 and flat[x] < capf[x]:
                flat[x] += 1
                rest -= 1
                moved = True
        if not moved:
            break
    return flat.reshape(avg.shape)


def _top_mass_omitted(block_mass: np.ndarray, row_mass: np.ndarray, budget: int, n_legal: int) -> np.ndarray:
    """Omitted mass per row when the `budget` legal tiles with the largest block mass are kept."""
    keep = np.argsort(-block_mass[:n_legal], kind="stable")[:budget]
    return 1.0 - row_mass[:, keep].sum(axis=1)


def matched_work(q, k, v, scale: float, tau: float, Bq: int, Bk: int):
    """q [B,N,Hq,d], k, v [B,Nk,Hkv,d] (causal, the queries the last N positions, N and Nk - N multiples of Bq).
    Returns dict(tiles = total retained tiles, and per policy the mean omitted mass over all rows:
    mala, per_instance, static, position_only) plus the per-decision arrays under '<policy>_per_block' [B,Hq,Tr]."""
    B, N, Hq, d = q.shape
    Nk, Hkv = k.shape[1], k.shape[2]
    G, off = Hq // Hkv, Nk - N
    assert N % Bq == 0 and off % Bq == 0
    Tr = N // Bq
    f = orc.fwd(q, k, v, scale, tau, Bq, Bk)
    counts = (f["mask"] == orc.RETAINED).sum(axis=3)                       # [B,Hq,Tr]
    legal = (f["mask"] != orc.ILLEGAL).sum(axis=3)                         # [B,Hq,Tr]
    static_avg = counts.mean(axis=0, keepdims=True).repeat(B, axis=0)
    pos_avg = counts.mean(axis=(0, 1), keepdims=True).repeat(B, axis=0).repeat(Hq, axis=1)
    budgets = {"per_instance": counts}
    st = np.zeros_like(counts)
    for h in range(Hq):
        for i in range(Tr):
            st[:, h, i] = _largest_remainder(static_avg[:, h, i], int(counts[:, h, i].sum()), legal[:, h, i])
    budgets["static"] = st
    po = np.zeros_like(counts)
    for i in range(Tr):
        po[:, :, i] = _largest_remainder(pos_avg[:, :, i], int(counts[:, :, i].sum()), legal[:, :, i])
    budgets["position_only"] = po
    out = {"tiles": int(counts.sum())}
    omitted = {p_: np.zeros((B, Hq, Tr)) for p_ in ("mala", "per_instance", "static", "position_only")}
    for b in range(B):
        for h in range(Hq):
            Q, K = orc._head(q, b, h), orc._head(k, b, h // G)
            M = dense_tile_mass(Q, K, scale, Bq, Bk, off)
            for i in range(Tr):
                rows = slice(i * Bq, (i + 1) * Bq)
                rm = M[rows]
                bm = rm.sum(axis=0)
                kept = f["mask"][b, h, i] == orc.RETAINED
                omitted["mala"][b, h, i] = (1.0 - rm[:, kept].sum(axis=1)).mean()
                for p_, bud in budgets.items():
                    omitted[p_][b, h, i] = _top_mass_omitted(bm, rm, int(bud[b, h, i]), int(legal[b, h, i])).mean()
    for p_, a in omitted.items():
        out[p_] = float(a.mean())
        out[p_ + "_per_block"] = a
    out["budgets"] = budgets
    return out
