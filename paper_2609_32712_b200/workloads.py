"""Seeded synthetic inputs for the MALA attention path (prefill fwd/bwd and split-KV decode).

This module only draws random tensors and plants structure in them; it holds none of the
method's arithmetic and imports neither the CUDA binding nor the oracle, so both sides can be
fed from it.  Everything is returned as bf16 tensors ``[B, N, H, d]`` (``q`` of decode:
``[B, 1, Hq, d]``).

Structure goes into Q only (K, V stay i.i.d. so that GQA sharing of K is unaffected), per query
head ``h`` with key head ``h // (Hq // Hkv)``:

  diffuse   q_i = q0_i
  planted   q_i = q0_i + 3 * sum_{j in P_i} k_j           P_i: up to P distinct keys drawn from [0, i)
  peaked    planted (P keys) + (4/sqrt(d)) * sum_{j=max(0,i-63)}^{i} k_j     (64-token local window, +4)
  sink      q_i = q0_i + (6/sqrt(d)) * sum_{j<min(4,i+1)} k_j              (first 4 keys, +6)
  decay     k_j[d-1] = j / 256, q_i[d-1] = rate * 256 * sqrt(d): score(i, j) = rate * j + noise, mass decaying smoothly
            toward earlier keys (rate = 1e-3 .. 3e-3 by head; one query head per KV head); for near-threshold tests

``q += c * k_j`` raises score (i, j) by ``c * |k_j|^2 / sqrt(d) ~= c * sqrt(d)``.

Preset ``"R"`` (paper-like regime; this repository's addition, the literal presets retain ~100 % of
tiles): every K row is rescaled to norm sqrt(d); non-diffuse heads use
``q_i = q0_i + 8 k_i + 8 (k_{j1(seg)} + k_{j2(seg)})`` with ``seg = i // 256`` and ``j1, j2`` uniform in
``[0, 256 seg)`` (none for seg 0): a self anchor plus two retrieval keys shared by 256 consecutive
queries.

Preset ``"S"`` (this repository's addition as well): preset "R" with EVERY head built that way, the diffuse ones
included -- no head retains everything, which puts the whole configuration at the sparsity the paper reports for
trained models (about 1000 retained key slots per query).

Preset ``"D"`` (decode): the last feature gates keys -- ``k_j[d-1] = 0`` for live keys and ``-19``
otherwise, ``q[d-1] = 19`` for non-diffuse KV groups; live keys are one 128-key tile per 1024-key
chunk (tile ``(5 * chunk + 3) mod 8``) plus the newest 128 keys.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import torch


@dataclass
class PrefillConfig:
    name: str
    B: int
    Hq: int
    Hkv: int
    N: int
    d: int
    head_types: List[str]          # one entry per query head
    planted: int = 8               # P for planted / peaked heads
    taus: List[float] = field(default_factory=lambda: [0.0, 1e-5, 1e-4, 1e-3])
    seed: int = 0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)


@dataclass
class DecodeConfig:
    name: str
    B: int
    Hq: int
    Hkv: int
    Nk: int
    d: int
    num_splits: int
    group_types: List[str]         # one entry per KV head (packed decode rows share a type)
    planted: int = 8
    taus: List[float] = field(default_factory=lambda: [0.0, 1e-4])
    seed: int = 0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)


def _mix4(n: int) -> List[str]:
    return [("diffuse", "sink", "peaked", "peaked")[h % 4] for h in range(n)]


def prefill_config(name: str) -> PrefillConfig:
    """The four prefill configurations of the benchmark definition, by name ``cfg1`` .. ``cfg4``, and ``tp8``."""
    if name == "cfg1":
        return PrefillConfig("cfg1", 1, 2, 2, 1024, 64, ["planted"] * 2, planted=4, seed=1)
    if name == "cfg2":
        return PrefillConfig("cfg2", 1, 16, 4, 8192, 128, ["diffuse"] * 8 + ["peaked"] * 8, seed=2)
    if name == "cfg3":
        return PrefillConfig("cfg3", 1, 32, 8, 32768, 128, _mix4(32), taus=[0.0, 1e-4], seed=3)
    if name == "cfg4":
        return PrefillConfig("cfg4", 1, 8, 2, 131072, 128, _mix4(8), taus=[0.0, 1e-4], seed=4)
    if name == "tp8":
        # one tensor-parallel rank's slice of the paper's operator benchmark (64 query / 8 KV heads over 8 ranks):
        # 8 query heads on 1 KV head, 131072 tokens, head size 128; the 32K configuration's head mix
        return PrefillConfig("tp8", 1, 8, 1, 131072, 128, _mix4(8), taus=[0.0, 1e-4, 1.0], seed=6)
    raise KeyError(name)


def decode_config(name: str = "cfg5") -> DecodeConfig:
    if name == "cfg5":
        return DecodeConfig("cfg5", 8, 32, 8, 131072, 128, 128, _mix4(8), seed=5)
    raise KeyError(name)


def _randn(shape, gen: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def _planted_sum(k_h: torch.Tensor, P: int, gen: torch.Generator, rows: Optional[torch.Tensor] = None):
    """sum over up to P distinct keys drawn uniformly from [0, i) for every row i (row 0: none).

    k_h: [N, d] fp32.  rows: optional 1-D tensor of row indices (default all rows)."""
    N, d = k_h.shape
    dev = k_h.device
    if rows is None:
        rows = torch.arange(N, device=dev)
    u = torch.rand((rows.numel(), P), generator=gen, device=dev, dtype=torch.float64)
    idx = torch.floor(u * rows.to(torch.float64)[:, None]).to(torch.int64)
    idx, _ = torch.sort(idx, dim=1)
    w = torch.ones_like(idx, dtype=torch.float32)
    w[:, 1:] = (idx[:, 1:] != idx[:, :-1]).to(torch.float32)     # drop duplicates
    w = w * (rows > 0).to(torch.float32)[:, None]
    out = torch.zeros((rows.numel(), d), device=dev, dtype=torch.float32)
    for p in range(P):
        out += k_h[idx[:, p]] * w[:, p:p + 1]
    return out


def _window_sum(k_h: torch.Tensor, width: int = 64) -> torch.Tensor:
    c = torch.cumsum(k_h.to(torch.float64), dim=0)
    lag = torch.zeros_like(c)
    lag[width:] = c[:-width]
    return (c - lag).to(torch.float32)


def _sink_sum(k_h: torch.Tensor, n_sink: int = 4) -> torch.Tensor:
    N = k_h.shape[0]
    c = torch.cumsum(k_h[:n_sink].to(torch.float64), dim=0).to(torch.float32)
    out = c[-1].expand(N, -1).clone()
    out[: min(n_sink, N)] = c[: min(n_sink, N)]
    return out


def make_prefill(cfg: PrefillConfig, preset: str = "literal", device="cpu", seed: Optional[int] = None):
    """Returns dict(q, k, v, do) bf16 ``[B, N, H, d]`` plus ``scale`` and the config."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed if seed is None else seed)
    B, Hq, Hkv, N, d = cfg.B, cfg.Hq, cfg.Hkv, cfg.N, cfg.d
    G = Hq // Hkv
    # fixed draw order: q0, k, v, dO, then index draws head by head
    q = _randn((B, N, Hq, d), gen, dev)
    k = _randn((B, N, Hkv, d), gen, dev)
    v = _randn((B, N, Hkv, d), gen, dev)
    do = _randn((B, N, Hq, d), gen, dev)
    if preset in ("R", "S"):
        k = k * (math.sqrt(d) / k.norm(dim=-1, keepdim=True))
    elif preset != "literal":
        raise KeyError(preset)
    rs = 1.0 / math.sqrt(d)
    for b in range(B):
        for h in range(Hq):
            kind = cfg.head_types[h]
            k_h = k[b, :, h // G, :]
            if kind == "diffuse" and preset != "S":
                continue
            if kind == "decay":
                # score(i, j) = rate * j + N(0, 1): the softmax mass of a row decays smoothly toward earlier keys (a
                # per-row shift does not change a softmax), so the tile criteria pass through zero with a small slope
                # per tile -- the inputs on which near-threshold decisions are tested.  Uses the last feature of the
                # head's KV head (meant for one query head per KV head).
                rate = 1e-3 * (1 + h % 3)
                k[b, :, h // G, d - 1] = torch.arange(N, device=dev, dtype=torch.float32) / 256.0
                q[b, :, h, d - 1] = rate * 256.0 * math.sqrt(d)
                continue
            if preset in ("R", "S"):
                nseg = -(-N // 256)
                u = torch.rand((nseg, 2), generator=gen, device=dev, dtype=torch.float64)
                seg = torch.arange(nseg, device=dev, dtype=torch.float64)
                j = torch.floor(u * (256.0 * seg)[:, None]).to(torch.int64)            # [nseg, 2]
                anchors = (k_h[j[:, 0]] + k_h[j[:, 1]]) * (seg > 0).to(torch.float32)[:, None]
                q[b, :, h, :] += 8.0 * k_h + 8.0 * anchors.repeat_interleave(256, dim=0)[:N]
                continue
            if kind in ("planted", "peaked"):
                q[b, :, h, :] += 3.0 * _planted_sum(k_h, cfg.planted, gen)
            if kind == "peaked":
                q[b, :, h, :] += (4.0 * rs) * _window_sum(k_h, 64)
            if kind == "sink":
                q[b, :, h, :] += (6.0 * rs) * _sink_sum(k_h, 4)
    bf = torch.bfloat16
    return dict(q=q.to(bf), k=k.to(bf), v=v.to(bf), do=do.to(bf), scale=cfg.scale, cfg=cfg, preset=preset)


def make_decode(cfg: DecodeConfig, preset: str = "literal", device="cpu", seed: Optional[int] = None):
    """Returns dict(q [B,1,Hq,d], kcache, vcache [B,Nk,Hkv,d]) bf16; the query is the newest token
    (position Nk-1, whose own key is the last cache entry)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed if seed is None else seed)
    B, Hq, Hkv, Nk, d = cfg.B, cfg.Hq, cfg.Hkv, cfg.Nk, cfg.d
    G = Hq // Hkv
    bf = torch.bfloat16
    q = _randn((B, 1, Hq, d), gen, dev)
    kc = torch.empty((B, Nk, Hkv, d), device=dev, dtype=bf)
    vc = torch.empty((B, Nk, Hkv, d), device=dev, dtype=bf)
    rs = 1.0 / math.sqrt(d)
    last = torch.tensor([Nk - 1], device=dev)
    for b in range(B):
        kb = _randn((Nk, Hkv, d), gen, dev)
        vb = _randn((Nk, Hkv, d), gen, dev)
        for g in range(Hkv):
            kind = cfg.group_types[g]
            k_h = kb[:, g, :]
            if preset == "D":
                tile = torch.arange(Nk, device=dev) // 128
                live = ((tile % 8) == ((5 * (tile // 8) + 3) % 8)) | (torch.arange(Nk, device=dev) >= Nk - 128)
                k_h[:, d - 1] = torch.where(live, 0.0, -19.0)
                if kind != "diffuse":
                    q[b, 0, g * G:(g + 1) * G, d - 1] = 19.0
                continue
            if preset != "literal":
                raise KeyError(preset)
            for h in range(g * G, (g + 1) * G):
                if kind == "peaked":
                    q[b, 0, h] += 3.0 * _planted_sum(k_h, cfg.planted, gen, rows=last)[0]
                    q[b, 0, h] += (4.0 * rs) * k_h[max(0, Nk - 64):].sum(dim=0)
                elif kind == "sink":
                    q[b, 0, h] += (6.0 * rs) * k_h[:4].sum(dim=0)
        kc[b] = kb.to(bf)
        vc[b] = vb.to(bf)
    return dict(q=q.to(bf), kcache=kc, vcache=vc, scale=cfg.scale, cfg=cfg, preset=preset)


def paginate(kcache: torch.Tensor, vcache: torch.Tensor, page_size: int, seqlens=None, seed: int = 0,
             spare_pages: int = 3):
    """Serving-side layout of a decode workload: the contiguous caches [B,Nk,Hkv,d] are cut into pages of
    ``page_size`` keys that are scattered over a shuffled pool of B*ceil(Nk/page_size) + spare_pages pages.
    Slots that no sequence uses (beyond ``seqlens[b]``, spare pages) hold finite junk, and block-table entries of
    pages a sequence does not reach point outside the pool.  Returns (kpages, vpages, block_table int32
    [B, max_pages], seqlens int32 [B])."""
    B, Nk, Hkv, d = kcache.shape
    dev = kcache.device
    mp = -(-Nk // page_size)
    pool = B * mp + spare_pages
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    perm = torch.randperm(pool, generator=gen)
    lens = [Nk] * B if seqlens is None else [int(x) for x in seqlens]
    # (one page of junk, repeated: the pool of a full-size cache has 10^9 slots)
    kp = (8.0 * torch.randn((page_size, Hkv, d), generator=gen)).to(kcache.dtype).to(dev).repeat(pool, 1, 1, 1)
    vp = (8.0 * torch.randn((page_size, Hkv, d), generator=gen)).to(vcache.dtype).to(dev).repeat(pool, 1, 1, 1)
    bt = torch.full((B, mp), pool + 5, dtype=torch.int32)
    for b in range(B):
        for x in range(-(-lens[b] // page_size)):
            n = min(page_size, lens[b] - x * page_size)
            pg = int(perm[b * mp + x])
            bt[b, x] = pg
            kp[pg, :n] = kcache[b, x * page_size:x * page_size + n]
            vp[pg, :n] = vcache[b, x * page_size:x * page_size + n]
    return kp, vp, bt.to(dev), torch.tensor(lens, dtype=torch.int32, device=dev)


def pack_sequences(ws):
    """Packed layout of several single-sequence prefill workloads (each B = 1, same heads): q, k, v, do
    concatenated along the rows as [1, total, H, d], and cu_seqlens int32 [len(ws) + 1]."""
    out = {x: torch.cat([w[x] for w in ws], dim=1).contiguous() for x in ("q", "k", "v", "do")}
    lens = [w["q"].shape[1] for w in ws]
    cu = [0]
    for n in lens:
        cu.append(cu[-1] + n)
    out.update(cu_seqlens=torch.tensor(cu, dtype=torch.int32, device=out["q"].device), lens=lens, scale=ws[0]["scale"])
    return out


def rademacher_like(t: torch.Tensor, seed: int) -> torch.Tensor:
    """Upstream gradient of +-1 entries (the Rademacher probe of the operator-fidelity protocol, Section 5.1)."""
    gen = torch.Generator(device=t.device)
    gen.manual_seed(seed)
    bits = torch.randint(0, 2, t.shape, generator=gen, device=t.device, dtype=torch.int8)
    return (bits * 2 - 1).to(t.dtype)


def custom_prefill(B, Hq, Hkv, N, d, head_types=None, planted=4, seed=0, preset="literal", device="cpu"):
    """Small / odd-shaped cases for tests (any N, including ragged tails)."""
    if head_types is None:
        head_types = [("diffuse", "planted", "peaked", "sink")[h % 4] for h in range(Hq)]
    cfg = PrefillConfig(f"custom_B{B}_H{Hq}_{Hkv}_N{N}_d{d}", B, Hq, Hkv, N, d, list(head_types), planted=planted,
                        seed=seed)
    return make_prefill(cfg, preset=preset, device=device)


def custom_decode(B, Hq, Hkv, Nk, d, num_splits, group_types=None, seed=0, preset="literal", device="cpu"):
    if group_types is None:
        group_types = _mix4(Hkv)
    cfg = DecodeConfig(f"custom_dec_B{B}_H{Hq}_{Hkv}_N{Nk}_d{d}", B, Hq, Hkv, Nk, d, num_splits, list(group_types),
                       seed=seed)
    return make_decode(cfg, preset=preset, device=device)


def paginate_scales(scales: torch.Tensor, block_table: torch.Tensor, page_size: int, tile: int = 128):
    """The per-tile scales [B, Hkv, nt] of a contiguous 8-bit cache in the layout of its paged copy made by
    ``paginate`` with the same ``page_size``: [num_pages, Hkv, page_size/tile], page block_table[b][x] holding the
    scales of tiles x*tpp .. of sequence b; pages no sequence uses get scale 1."""
    B, Hkv, nt = scales.shape
    tpp = page_size // tile
    mp = block_table.shape[1]
    pool = B * mp + 3 if int(block_table.max()) >= B * mp else int(block_table.max()) + 1
    pool = max(pool, int(block_table[block_table < B * mp + 3].max()) + 1)
    out = torch.ones((pool, Hkv, tpp), dtype=torch.float32, device=scales.device)
    pad = torch.ones((B, Hkv, mp * tpp), dtype=torch.float32, device=scales.device)
    pad[:, :, :nt] = scales
    bt = block_table.to(scales.device).long()
    for b in range(B):
        for x in range(mp):
            pg = int(bt[b, x])
            if 0 <= pg < pool:
                out[pg] = pad[b, :, x * tpp:(x + 1) * tpp]
    return out


def quantize_cache_e4m3(x: torch.Tensor, tile: int = 128):
    """8-bit storage of a KV cache [B, Nk, Hkv, d]: e4m3 values with one fp32 scale per (sequence, KV head, tile of
    128 keys), scale = largest magnitude of the tile / 448 (the largest e4m3 value).  Returns (codes uint8
    [B,Nk,Hkv,d], scales fp32 [B,Hkv,ceil(Nk/tile)], dequantised fp32 [B,Nk,Hkv,d] = scale * e4m3(code), the values an
    8-bit decode call works on and its oracle is given)."""
    B, Nk, Hkv, d = x.shape
    nt = -(-Nk // tile)
    xf = torch.zeros((B, nt * tile, Hkv, d), dtype=torch.float32, device=x.device)
    xf[:, :Nk] = x.float()
    t = xf.view(B, nt, tile, Hkv, d)
    amax = t.abs().amax(dim=(2, 4))                                   # [B, nt, Hkv]
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
    codes = (t / scale[:, :, None, :, None]).clamp(-448.0, 448.0).to(torch.float8_e4m3fn)
    deq = (codes.float() * scale[:, :, None, :, None]).view(B, nt * tile, Hkv, d)[:, :Nk].contiguous()
    codes = codes.view(B, nt * tile, Hkv, d)[:, :Nk].contiguous().view(torch.uint8)
    return codes, scale.permute(0, 2, 1).contiguous(), deq
