#!/usr/bin/env python
"""Benchmark of the MALA attention hot path on B200 (one process per GPU).

A step is one pass of the whole path -- mala_fwd then mala_bwd at tolerance tau -- over one batch of
seeded synthetic input of the benchmark definition's 32K configuration (cfg3; --workload selects
another).  `value` is dense-equivalent TFLOP/s of fwd+bwd (FullAttn FLOP model: 4*B*Hq*N^2*d/2 forward,
2.5x that backward) with inputs resident in HBM; `e2e` is the same metric with pinned-host inputs copied
in and results copied out every step.  The line also carries, under `detail`, fwd / bwd latency of the
MALA and dense kernels on cfg3 / cfg4 (literal and paper-regime "R" inputs), decode latency on cfg5
(literal and gated "D" inputs), the skipped-tile fractions, and for cfg3 R and cfg5 D the work / fidelity
figures (retained slots, omitted mass, relative L2 against the dense path) at tau = 1e-4, 1e-2 and 1.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
  python bench.py --only fwd|bwd|decode|decode8 --workload cfg2 --preset R --tau 1e-4 --iters 3
      (a few launches of one operator and nothing else: the small fixed command profiler captures are taken on)
  python bench.py --workload tp8 [--preset S --tau 1] (under torchrun --nproc-per-node 8: one tensor-parallel rank's
      head slice of the paper's 128K operator benchmark per GPU, timed as the synchronized wall clock of the group)
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

TILE = 128


def fwd_dense_equiv_flops(B, Hq, N, d):
    return 4.0 * B * Hq * N * N * d / 2.0


def bwd_dense_equiv_flops(B, Hq, N, d):
    return 2.5 * fwd_dense_equiv_flops(B, Hq, N, d)


def fwd_executed_flops(legal, retained, d):
    return (legal + retained) * 2.0 * TILE * TILE * d


def bwd_executed_flops(legal, retained, d):
    return (legal + 4.0 * retained) * 2.0 * TILE * TILE * d


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


def load_dram_traffic(workload, preset, tau):
    """DRAM bytes of the backward's main kernels for one call on (workload, preset, tau), from the table kept beside the
    ncu summaries it was read from (profiles/dram_traffic.txt); None where no capture exists."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None, None
    with open(path) as f:
        for line in f:
            t = line.split()
            if len(t) >= 6 and not line.startswith("#") and t[0] == workload and t[1] == preset and float(t[2]) == tau:
                return float(t[4]), t[5]
    return None, None


def clk_per_tile(mala_ms, dense_ms, retained, legal, sm_mhz, n_sm=148):
    """SM clocks one SM spends per retained and per skipped tile: the dense kernel's time over all legal tiles gives
    the retained figure, the MALA kernel's time minus the retained share of the dense time the skipped one."""
    if not sm_mhz or legal <= 0:
        return None, None
    per_ret = dense_ms * 1e-3 * sm_mhz * 1e6 * n_sm / legal
    skipped = legal - retained
    per_skip = ((mala_ms - retained / legal * dense_ms) * 1e-3 * sm_mhz * 1e6 * n_sm / skipped) if skipped > 0 else None
    return per_ret, per_skip


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        busy = [x for x in sm if x > 0.5 * max(sm)] if sm else []
        return dict(sm_mhz=statistics.median(busy) if busy else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def max_over_ranks(value: float, device) -> float:
    """Maximum of a per-rank scalar over all ranks of the default process group (identity if none)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(flops_per_rank_step: float, world: int, ms_per_step: float) -> float:
    """Aggregate TFLOP/s of `world` replicas that each process flops_per_rank_step in ms_per_step (max over ranks)."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def time_cuda(fn, warmup, iters):
    """Average milliseconds per call of fn(), CUDA events on the current stream."""
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def time_alternating(fns, warmup, iters, rounds=2, prep=None):
    """Average milliseconds per call of each function in `fns` (label -> callable).  The functions are measured in
    turn over several rounds, so that a clock that drifts under the power cap treats them alike (a kernel timed right
    after a long backward pass runs a few per cent slower than the same kernel timed first).  `prep` (label ->
    callable) runs untimed before each of the label's chunks, e.g. the forward pass whose output a backward needs."""
    import torch
    for k, f in fns.items():
        if prep:
            prep[k]()
        for _ in range(warmup):
            f()
    torch.cuda.synchronize()
    per = max(1, iters // rounds)
    tot = {k: 0.0 for k in fns}
    for _ in range(rounds):
        for k, f in fns.items():
            if prep:
                prep[k]()
            tot[k] += time_cuda(f, 0, per) * per
    return {k: v / (per * rounds) for k, v in tot.items()}


class PrefillCase:
    """Device-resident inputs, outputs and scratch of one prefill configuration."""

    def __init__(self, name, preset, device, seed_offset=0):
        import torch
        from paper_2609_32712_b200 import mala, workloads as W
        self.mala = mala
        self.cfg = W.prefill_config(name)
        self.preset = preset
        w = W.make_prefill(self.cfg, preset=preset, device=device, seed=self.cfg.seed + seed_offset)
        self.q, self.k, self.v, self.do = w["q"], w["k"], w["v"], w["do"]
        self.scale = w["scale"]
        c = self.cfg
        self.o = torch.empty_like(self.q)
        self.lse = torch.empty((c.B, c.Hq, c.N), dtype=torch.float32, device=device)
        self.dq, self.dk, self.dv = torch.empty_like(self.q), torch.empty_like(self.k), torch.empty_like(self.v)
        self.ws = torch.empty(mala.workspace_bytes(mala.OP_BWD, c.B, c.Hq, c.Hkv, c.N, c.d), dtype=torch.uint8,
                              device=device)
        self.fwd_de = fwd_dense_equiv_flops(c.B, c.Hq, c.N, c.d)
        self.bwd_de = bwd_dense_equiv_flops(c.B, c.Hq, c.N, c.d)

    def fwd(self, tau, stats=False):
        return self.mala.fwd(self.q, self.k, self.v, self.scale, tau, out=self.o, lse=self.lse, stats=stats, ws=self.ws)

    def bwd(self, tau, stats=False):
        return self.mala.bwd(self.q, self.k, self.v, self.o, self.do, self.lse, self.scale, tau, ws=self.ws,
                             dq=self.dq, dk=self.dk, dv=self.dv, stats=stats)

    def step(self, tau):
        self.fwd(tau)
        self.bwd(tau)

    def tile_stats(self, tau):
        import torch
        _, _, fs = self.fwd(tau, stats=True)
        _, _, _, bs = self.bwd(tau, stats=True)
        torch.cuda.synchronize()
        f, b = fs.totals.cpu().tolist(), bs.totals.cpu().tolist()
        return dict(fwd_retained=f[0], fwd_legal=f[1], bwd_retained=b[0], bwd_legal=b[1])

    def input_bytes(self):
        return sum(t.numel() * t.element_size() for t in (self.q, self.k, self.v, self.do))


def chunk_leg(cs, Nq, tau, it, peaks):
    """mala_fwd_chunk / mala_bwd_chunk on the last Nq queries of a prefill case (all keys): latency of the MALA and
    dense kernels and the tensor-pipe fraction on the tile FLOPs executed."""
    import torch
    mala, cc = cs.mala, cs.cfg
    off = cc.N - Nq
    q, do = cs.q[:, off:], cs.do[:, off:]
    o, lse = torch.empty_like(q), torch.empty((cc.B, cc.Hq, Nq), dtype=torch.float32, device=q.device)
    dq = torch.empty_like(q)
    row = {}
    taus = {"mala": tau, "dense": 0.0}
    fwd = {k: (lambda t_=t_: mala.fwd_chunk(q, cs.k, cs.v, cs.scale, t_, out=o, lse=lse)) for k, t_ in taus.items()}
    bwd = {k: (lambda t_=t_: mala.bwd_chunk(q, cs.k, cs.v, o, do, lse, cs.scale, t_, ws=cs.ws, dq=dq, dk=cs.dk, dv=cs.dv))
           for k, t_ in taus.items()}
    f_t, b_t = time_alternating(fwd, 3, it), time_alternating(bwd, 3, it, prep=fwd)
    for label in taus:
        row[label] = {"fwd_ms": f_t[label], "bwd_ms": b_t[label]}
    _, _, fs = mala.fwd_chunk(q, cs.k, cs.v, cs.scale, tau, out=o, lse=lse, stats=True)
    _, _, _, bs = mala.bwd_chunk(q, cs.k, cs.v, o, do, lse, cs.scale, tau, ws=cs.ws, dq=dq, dk=cs.dk, dv=cs.dv,
                                 stats=True)
    torch.cuda.synchronize()
    (fr, fl), (br, bl) = fs.totals.cpu().tolist(), bs.totals.cpu().tolist()
    row["fwd_retained_frac"], row["bwd_retained_frac"] = fr / fl, br / bl
    row["legal_tiles"] = fl
    row["fwd_tensor_frac_on_executed"] = (fwd_executed_flops(fl, fr, cc.d) / (row["mala"]["fwd_ms"] * 1e-3) / 1e12
                                          / peaks["tflops_sustained"])
    row["bwd_tensor_frac_on_executed"] = (bwd_executed_flops(bl, br, cc.d) / (row["mala"]["bwd_ms"] * 1e-3) / 1e12
                                          / peaks["tflops_sustained"])
    row["speedup_fwd"] = row["dense"]["fwd_ms"] / row["mala"]["fwd_ms"]
    row["speedup_bwd"] = row["dense"]["bwd_ms"] / row["mala"]["bwd_ms"]
    return row


def chunk_split_leg(cs, Nq, tau, it):
    """A short chunk of queries against a long context: mala_fwd_chunk (one CTA per pair of query blocks) against
    mala_fwd_chunk_split (the keys cut into ranges that run on different SMs), MALA and dense, with the retained
    fraction of each (the split-local test is the more conservative one)."""
    import torch
    mala, cc = cs.mala, cs.cfg
    q = cs.q[:, cc.N - Nq:]
    o, lse = torch.empty_like(q), torch.empty((cc.B, cc.Hq, Nq), dtype=torch.float32, device=q.device)
    row = {}
    for S in (1, 8, 16, 32):
        ws = torch.empty(max(256, mala.workspace_bytes(mala.OP_FWD, cc.B, cc.Hq, cc.Hkv, Nq, cc.d, S)), dtype=torch.uint8,
                         device=q.device)
        r = {}
        for label, t_ in (("mala", tau), ("dense", 0.0)):
            if S == 1:
                fn = lambda: mala.fwd_chunk(q, cs.k, cs.v, cs.scale, t_, out=o, lse=lse)
            else:
                fn = lambda: mala.fwd_chunk_split(q, cs.k, cs.v, cs.scale, t_, S, out=o, lse=lse, ws=ws)
            r[label + "_ms"] = time_cuda(fn, 3, it)
        if S == 1:
            _, _, st = mala.fwd_chunk(q, cs.k, cs.v, cs.scale, tau, out=o, lse=lse, stats=True)
        else:
            _, _, st = mala.fwd_chunk_split(q, cs.k, cs.v, cs.scale, tau, S, out=o, lse=lse, ws=ws, stats=True)
        ret, leg = st.totals.cpu().tolist()
        r["retained_frac"] = ret / leg
        row[f"splits={S}"] = r
        del ws
    return row


def varlen_leg(cfg, preset, lens, tau, it, peaks, dev):
    """mala_fwd_varlen / mala_bwd_varlen on packed sequences with the heads of a prefill configuration: latency of
    the MALA and dense kernels and the tensor-pipe fraction on the tile FLOPs executed."""
    import torch
    from paper_2609_32712_b200 import mala, workloads as W
    ws = [W.custom_prefill(1, cfg.Hq, cfg.Hkv, n, cfg.d, head_types=cfg.head_types, seed=cfg.seed + 31 * x,
                           preset=preset, device=dev) for x, n in enumerate(lens)]
    pk = W.pack_sequences(ws)
    q, k, v, do, cu = pk["q"], pk["k"], pk["v"], pk["do"], pk["cu_seqlens"]
    total, mx = sum(lens), max(lens)
    wsb = torch.empty(mala.workspace_bytes(mala.OP_BWD, 1, cfg.Hq, cfg.Hkv, total + 128 * len(lens), cfg.d),
                      dtype=torch.uint8, device=dev)
    row = {"lens": list(lens)}
    taus = {"mala": tau, "dense": 0.0}
    outs = {lab: mala.fwd_varlen(q, k, v, cu, mx, pk["scale"], t_)[:2] for lab, t_ in taus.items()}
    fwd = {lab: (lambda t_=t_: mala.fwd_varlen(q, k, v, cu, mx, pk["scale"], t_)) for lab, t_ in taus.items()}
    bwd = {lab: (lambda t_=t_, lab=lab: mala.bwd_varlen(q, k, v, outs[lab][0], do, outs[lab][1], cu, mx, pk["scale"], t_,
                                                         ws=wsb)) for lab, t_ in taus.items()}
    f_t, b_t = time_alternating(fwd, 3, it), time_alternating(bwd, 3, it)
    for label in taus:
        row[label] = {"fwd_ms": f_t[label], "bwd_ms": b_t[label]}
    o, lse, fs = mala.fwd_varlen(q, k, v, cu, mx, pk["scale"], tau, stats=True)
    _, _, _, bs = mala.bwd_varlen(q, k, v, o, do, lse, cu, mx, pk["scale"], tau, ws=wsb, stats=True)
    torch.cuda.synchronize()
    (fr, fl), (br, bl) = fs.totals.cpu().tolist(), bs.totals.cpu().tolist()
    row["legal_tiles"] = fl
    row["fwd_retained_frac"], row["bwd_retained_frac"] = fr / fl, br / bl
    row["fwd_tensor_frac_on_executed"] = (fwd_executed_flops(fl, fr, cfg.d) / (row["mala"]["fwd_ms"] * 1e-3) / 1e12
                                          / peaks["tflops_sustained"])
    row["bwd_tensor_frac_on_executed"] = (bwd_executed_flops(bl, br, cfg.d) / (row["mala"]["bwd_ms"] * 1e-3) / 1e12
                                          / peaks["tflops_sustained"])
    return row


def head_size_leg(cfg, preset, d, tau, it, peaks, dev):
    """The configuration's shapes with another head size (it runs on the next wider kernel, with zero-filled columns):
    latency of the MALA and dense kernels and the tensor-pipe fraction counted on the d columns that carry data."""
    import torch
    from paper_2609_32712_b200 import mala, workloads as W
    w = W.custom_prefill(cfg.B, cfg.Hq, cfg.Hkv, cfg.N, d, head_types=cfg.head_types, seed=cfg.seed, preset=preset, device=dev)
    q, k, v, do = w["q"], w["k"], w["v"], w["do"]
    wsb = torch.empty(mala.workspace_bytes(mala.OP_BWD, cfg.B, cfg.Hq, cfg.Hkv, cfg.N, d), dtype=torch.uint8, device=dev)
    taus = {"mala": tau, "dense": 0.0}
    outs = {lab: mala.fwd(q, k, v, w["scale"], t_)[:2] for lab, t_ in taus.items()}
    fwd = {lab: (lambda t_=t_: mala.fwd(q, k, v, w["scale"], t_)) for lab, t_ in taus.items()}
    bwd = {lab: (lambda t_=t_, lab=lab: mala.bwd(q, k, v, outs[lab][0], do, outs[lab][1], w["scale"], t_, ws=wsb))
           for lab, t_ in taus.items()}
    f_t, b_t = time_alternating(fwd, 3, it), time_alternating(bwd, 3, it)
    row = {"d": d}
    for label in taus:
        row[label] = {"fwd_ms": f_t[label], "bwd_ms": b_t[label]}
    _, _, fs = mala.fwd(q, k, v, w["scale"], tau, stats=True)
    torch.cuda.synchronize()
    fr, fl = fs.totals.cpu().tolist()
    row["fwd_retained_frac"] = fr / fl
    row["dense_fwd_tensor_frac_on_d_columns"] = (fwd_executed_flops(fl, fl, d) / (f_t["dense"] * 1e-3) / 1e12
                                                 / peaks["tflops_sustained"])
    row["dense_bwd_tensor_frac_on_d_columns"] = (bwd_executed_flops(fl, fl, d) / (b_t["dense"] * 1e-3) / 1e12
                                                 / peaks["tflops_sustained"])
    return row


def head_size_256_fwd_leg(cfg, preset, tau, it, peaks, dev):
    """The configuration's shapes with half the heads of twice the size (d = 256: the same FLOPs and bytes), forward only
    (one query block per CTA; the backward stops at 128 columns)."""
    import torch
    from paper_2609_32712_b200 import mala, workloads as W
    Hq, Hkv, d = cfg.Hq // 2, cfg.Hkv // 2, 256
    w = W.custom_prefill(cfg.B, Hq, Hkv, cfg.N, d, head_types=cfg.head_types[:cfg.Hq // 2], seed=cfg.seed, preset=preset, device=dev)
    q, k, v = w["q"], w["k"], w["v"]
    o = torch.empty_like(q)
    taus = {"mala": tau, "dense": 0.0}
    f_t = time_alternating({lab: (lambda t_=t_: mala.fwd(q, k, v, w["scale"], t_, out=o)) for lab, t_ in taus.items()}, 3, it)
    _, _, fs = mala.fwd(q, k, v, w["scale"], tau, stats=True)
    torch.cuda.synchronize()
    fr, fl = fs.totals.cpu().tolist()
    return {"d": d, "Hq": Hq, "Hkv": Hkv, "mala": {"fwd_ms": f_t["mala"]}, "dense": {"fwd_ms": f_t["dense"]},
            "fwd_retained_frac": fr / fl,
            "dense_fwd_tensor_frac": fwd_executed_flops(fl, fl, d) / (f_t["dense"] * 1e-3) / 1e12 / peaks["tflops_sustained"]}


def serving_prefill_leg(cfg, preset, tau, it, peaks, dev):
    """A serving-style prefill batch with the heads of a prefill configuration: eight sequences, a 2048-token chunk each
    behind prefixes of 0 ... 30720 tokens, packed (mala_fwd_varlen_prefix) and against a paged cache (mala_fwd_paged,
    256-key and 16-key pages in a shuffled pool): latency of the MALA and dense kernels, tensor-pipe fraction on executed work."""
    import torch
    from paper_2609_32712_b200 import mala, workloads as W
    prefixes, chunk = (30720, 16384, 8192, 4096, 2048, 1000, 300, 0), 2048
    nk = [p_ + chunk for p_ in prefixes]
    ws = [W.custom_prefill(1, cfg.Hq, cfg.Hkv, n, cfg.d, head_types=cfg.head_types, seed=cfg.seed + 17 * x, preset=preset,
                           device=dev) for x, n in enumerate(nk)]
    q = torch.cat([w["q"][:, n - chunk:] for w, n in zip(ws, nk)], dim=1).contiguous()
    k = torch.cat([w["k"] for w in ws], dim=1).contiguous()
    v = torch.cat([w["v"] for w in ws], dim=1).contiguous()
    cq = torch.tensor([chunk * x for x in range(len(nk) + 1)], dtype=torch.int32, device=dev)
    ck = torch.tensor([0] + list(torch.tensor(nk).cumsum(0)), dtype=torch.int32, device=dev)
    scale = ws[0]["scale"]
    Nmax = -(-max(nk) // 256) * 256
    kc = torch.zeros((len(nk), Nmax, cfg.Hkv, cfg.d), dtype=torch.bfloat16, device=dev)
    vc = torch.zeros_like(kc)
    for b, (w, n) in enumerate(zip(ws, nk)):
        kc[b, :n], vc[b, :n] = w["k"][0], w["v"][0]
    kp, vp, bt, sl = W.paginate(kc, vc, 256, seqlens=nk, seed=11)
    kp16, vp16, bt16, sl16 = W.paginate(kc, vc, 16, seqlens=nk, seed=12)
    del kc, vc, ws
    row = {"prefixes": list(prefixes), "chunk": chunk}
    taus = {"mala": tau, "dense": 0.0}
    packed = time_alternating({lab: (lambda t_=t_: mala.fwd_varlen_prefix(q, k, v, cq, ck, chunk, max(nk), scale, t_))
                               for lab, t_ in taus.items()}, 3, it)
    paged = time_alternating({lab: (lambda t_=t_: mala.fwd_paged(q, kp, vp, cq, bt, sl, chunk, scale, t_))
                              for lab, t_ in taus.items()}, 3, it)
    paged16 = time_alternating({lab: (lambda t_=t_: mala.fwd_paged(q, kp16, vp16, cq, bt16, sl16, chunk, scale, t_))
                                for lab, t_ in taus.items()}, 3, it)
    _, _, st = mala.fwd_varlen_prefix(q, k, v, cq, ck, chunk, max(nk), scale, tau, stats=True)
    torch.cuda.synchronize()
    ret, leg = st.totals.cpu().tolist()
    for lab in taus:
        row[lab] = {"packed_ms": packed[lab], "paged_ms": paged[lab], "paged_16key_pages_ms": paged16[lab]}
    row["legal_tiles"], row["retained_frac"] = leg, ret / leg
    row["tensor_frac_on_executed"] = (fwd_executed_flops(leg, ret, cfg.d) / (packed["mala"] * 1e-3) / 1e12
                                      / peaks["tflops_sustained"])
    row["dense_tensor_frac"] = (fwd_executed_flops(leg, leg, cfg.d) / (packed["dense"] * 1e-3) / 1e12
                                / peaks["tflops_sustained"])
    return row


def head_type_leg(cs, tau, it):
    """Per head type of a prefill case (one query head of each KV group, run as a multi-head call on strided views):
    retained fraction and latency of the MALA and dense kernels, so that the skip path's throughput can be read for
    the sparse head types alone."""
    import torch
    mala, cc = cs.mala, cs.cfg
    G = cc.Hq // cc.Hkv
    rows = {}
    for t in range(G):
        q, do = cs.q[:, :, t::G], cs.do[:, :, t::G]                 # head h = G g + t of every group g: its own KV head
        o, dq = torch.empty_like(q), torch.empty_like(q)
        lse = torch.empty((cc.B, cc.Hkv, cc.N), dtype=torch.float32, device=q.device)
        taus = {"mala": tau, "dense": 0.0}
        fwd = {k_: (lambda t_=t_: mala.fwd(q, cs.k, cs.v, cs.scale, t_, out=o, lse=lse)) for k_, t_ in taus.items()}
        bwd = {k_: (lambda t_=t_: mala.bwd(q, cs.k, cs.v, o, do, lse, cs.scale, t_, ws=cs.ws, dq=dq, dk=cs.dk, dv=cs.dv))
               for k_, t_ in taus.items()}
        f_t, b_t = time_alternating(fwd, 3, it), time_alternating(bwd, 3, it, prep=fwd)
        _, _, fs = mala.fwd(q, cs.k, cs.v, cs.scale, tau, out=o, lse=lse, stats=True)
        _, _, _, bs = mala.bwd(q, cs.k, cs.v, o, do, lse, cs.scale, tau, ws=cs.ws, dq=dq, dk=cs.dk, dv=cs.dv, stats=True)
        torch.cuda.synchronize()
        (fr, fl), (br, bl) = fs.totals.cpu().tolist(), bs.totals.cpu().tolist()
        kind = cc.head_types[t] if cs.preset == "literal" else ("diffuse" if (cc.head_types[t] == "diffuse" and cs.preset == "R") else "anchor+retrieval")
        rows[f"type{t}:{kind}"] = {"heads": cc.Hkv, "fwd_retained_frac": fr / fl, "bwd_retained_frac": br / bl,
                                   "fwd_ms": f_t["mala"], "bwd_ms": b_t["mala"], "dense_fwd_ms": f_t["dense"],
                                   "dense_bwd_ms": b_t["dense"], "speedup_fwd": f_t["dense"] / f_t["mala"],
                                   "speedup_bwd": b_t["dense"] / b_t["mala"]}
    return rows


def fidelity(cs, taus, it):
    """Work and operator fidelity of MALA against the in-library dense path on one configuration (the protocol
    of Section 5.1 on synthetic states): retained slots per query in forward and backward, omitted softmax mass
    eps = 1 - exp(lse_tau - lse_0) (bounded by tau / (1 + tau), Proposition 1), and relative L2 distance of O
    and of dQ, dK, dV under a Rademacher upstream gradient."""
    import torch
    from paper_2609_32712_b200 import workloads as W
    cc = cs.cfg
    do_saved = cs.do
    cs.do = W.rademacher_like(cs.q, seed=1000 + cc.seed)
    cs.fwd(0.0)
    cs.bwd(0.0)
    ref = {n: getattr(cs, n).float() for n in ("o", "dq", "dk", "dv")}
    nrm = {n: float(t.norm()) for n, t in ref.items()}
    lse0 = cs.lse.clone()
    dense_ms = (time_cuda(lambda: cs.fwd(0.0), 3, it), time_cuda(lambda: cs.bwd(0.0), 3, it))
    rows = {}
    for t_ in taus:
        st = cs.tile_stats(t_)                      # leaves the MALA o, lse and gradients in the case's buffers
        eps = 1.0 - torch.exp(cs.lse - lse0)
        row = {"fwd_slots_per_query": st["fwd_retained"] * TILE * TILE / (cc.B * cc.Hq * cc.N),
               "bwd_slots_per_query": st["bwd_retained"] * TILE * TILE / (cc.B * cc.Hq * cc.N),
               "fwd_retained_frac": st["fwd_retained"] / st["fwd_legal"],
               "bwd_retained_frac": st["bwd_retained"] / st["bwd_legal"],
               "omitted_mass_max": float(eps.max()), "omitted_mass_mean": float(eps.mean()),
               "omitted_mass_bound": t_ / (1.0 + t_)}
        for n in ("o", "dq", "dk", "dv"):
            row[f"rel_l2_{n}"] = float((getattr(cs, n).float() - ref[n]).norm()) / nrm[n]
        f_ms, b_ms = time_cuda(lambda: cs.fwd(t_), 3, it), time_cuda(lambda: cs.bwd(t_), 3, it)
        row.update(fwd_ms=f_ms, bwd_ms=b_ms, speedup_fwd=dense_ms[0] / f_ms, speedup_bwd=dense_ms[1] / b_ms)
        rows[f"tau={t_:g}"] = row
    cs.do = do_saved
    return rows


def oracle_sample(case, tau, o_gpu, lse_gpu):
    """Times the fp64 oracle on a bounded sample of the case's tiles (forward: some query blocks,
    backward: some key blocks).  Returns (dense-equivalent FLOPs of the sample, seconds, description)."""
    from oracle import mala_oracle as orc
    c = case.cfg
    T = -(-c.N // TILE)
    G = c.Hq // c.Hkv
    nb = min(16, T)
    fwd_blocks = sorted({max(0, T * (x + 1) // nb - 1) for x in range(nb)})
    fwd_units = [(0, h, i) for h in sorted({0, c.Hq - 1}) for i in fwd_blocks]
    bwd_blocks = sorted({min(T - 1, T // 2 + T * x // (2 * nb)) for x in range(nb)})
    bwd_units = [(0, 0, j) for j in bwd_blocks]
    tile_flops = 2.0 * TILE * TILE * c.d
    flops = sum((i + 1) * 2 * tile_flops for (_, _, i) in fwd_units)
    flops += sum(G * (T - j) * 5 * tile_flops for (_, _, j) in bwd_units)
    t0 = time.perf_counter()
    orc.fwd(case.q, case.k, case.v, case.scale, tau, TILE, TILE, units=fwd_units)
    orc.bwd(case.q, case.k, case.v, o_gpu, case.do, lse_gpu.cpu().numpy(), case.scale, tau, TILE, TILE,
            key_units=bwd_units)
    dt = time.perf_counter() - t0
    what = (f"{c.name} {case.preset}: oracle fwd on {len(fwd_blocks)} query blocks (every T/{nb}-th) of heads 0 and "
            f"{c.Hq - 1} + oracle bwd on {len(bwd_blocks)} key blocks of the upper half of KV head 0 "
            f"({flops / 1e9:.1f} dense-equivalent GFLOP of fp64 work)")
    return flops, dt, what


def run_reference(args, rank):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample of the same workload per step."""
    if rank != 0:
        return
    import torch
    from oracle import mala_oracle as orc
    from paper_2609_32712_b200 import workloads as W

    class Host:
        pass
    cfg = W.prefill_config(args.workload)
    # the inputs of the GPU arm: drawn by the same generator on the same kind of device (a CUDA generator where the
    # box has a GPU, which it does wherever the GPU arm runs), then moved to the host
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = W.make_prefill(cfg, preset=args.preset, device=gen_dev)
    case = Host()
    case.cfg, case.preset, case.scale = cfg, args.preset, w["scale"]
    case.q, case.k, case.v, case.do = (w[x].cpu() for x in ("q", "k", "v", "do"))
    T = -(-cfg.N // TILE)
    # the sampled backward needs o and lse of the sampled rows only through D and lse; use the oracle's own forward
    # on the rows that the sampled key blocks touch (the query blocks of the upper half)
    units = [(0, h, i) for h in range(cfg.Hq // cfg.Hkv) for i in range(T // 2, T)]
    f = orc.fwd(case.q, case.k, case.v, case.scale, args.tau, TILE, TILE, units=units)
    o = torch.from_numpy(f["o"]).nan_to_num(0.0)
    lse = torch.from_numpy(f["lse"]).nan_to_num(0.0)
    times, flops = [], 0.0
    what = ""
    for s in range(args.warmup + args.steps):
        fl, dt, what = oracle_sample(case, args.tau, o, lse)
        if s >= args.warmup:
            times.append(dt)
            flops = fl
    sec = sum(times) / len(times)
    val = flops / sec / 1e12
    print(json.dumps({
        "impl": "reference", "metric": "mala_fwd_bwd_dense_equiv_tflops", "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload} {args.preset} tau={args.tau}", "sample": what,
                   "inputs": f"seeded generator on {gen_dev} (the GPU arm's tensors), moved to the host"},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle", "sample": what},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_only(args, dev):
    """--only: a few launches of one operator on one synthetic configuration, nothing else."""
    import dataclasses
    import torch
    from paper_2609_32712_b200 import mala, workloads as W
    if args.only in ("decode", "decode8"):
        cfg = dataclasses.replace(W.decode_config("cfg5"), B=args.decode_batch)
        w = W.make_decode(cfg, preset=args.preset if args.preset in ("literal", "D") else "literal", device=dev)
        if args.only == "decode8":
            k8, ks8, _ = W.quantize_cache_e4m3(w["kcache"])
            v8, vs8, _ = W.quantize_cache_e4m3(w["vcache"])
        for _ in range(args.iters):
            if args.only == "decode8":
                mala.decode_fp8(w["q"], k8, v8, ks8, vs8, w["scale"], args.tau, cfg.num_splits)
            else:
                mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], args.tau, cfg.num_splits)
    else:
        cfg = W.prefill_config(args.workload)
        w = W.make_prefill(cfg, preset=args.preset, device=dev)
        o, lse, _ = mala.fwd(w["q"], w["k"], w["v"], w["scale"], args.tau)
        for _ in range(args.iters):
            if args.only == "fwd":
                mala.fwd(w["q"], w["k"], w["v"], w["scale"], args.tau, out=o, lse=lse)
            else:
                mala.bwd(w["q"], w["k"], w["v"], o, w["do"], lse, w["scale"], args.tau)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    print("ok")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="mala", choices=["mala", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg1", "cfg2", "cfg3", "cfg4", "tp8"])
    ap.add_argument("--preset", default="literal", choices=["literal", "R", "S", "D"])
    ap.add_argument("--only", default=None, choices=["fwd", "bwd", "decode", "decode8"],
                    help="run a few launches of one operator on --workload / --preset / --tau and exit (no timing table, "
                         "no CPU leg): the command that profiler captures are taken on")
    ap.add_argument("--iters", type=int, default=3, help="launches of --only")
    ap.add_argument("--decode-batch", type=int, default=2, help="batch size of --only decode (cfg5 shapes otherwise)")
    ap.add_argument("--tau", type=float, default=1e-4)
    ap.add_argument("--detail-iters", type=int, default=None,
                    help="timed iterations of every prefill detail measurement, after 3 warm-up iterations.  Default: the "
                         "MALA / dense rows of cfg3 and cfg4 use the paper's protocol (25 warm-up + 100 timed iterations, "
                         "as the decode rows always do) and the secondary rows (chunks, packed sequences, head types "
                         "...) 3 + 20; config.protocol in the output says which")
    ap.add_argument("--no-detail", action="store_true", help="skip the per-config detail table")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_32712_b200 import mala, workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    mala.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    warmup = max(args.warmup, 3)
    peaks = load_peaks()

    if args.only:
        run_only(args, dev)
        return

    # ---------------------------------------------------------------- main timed region (inputs in HBM)
    case = PrefillCase(args.workload, args.preset, dev, seed_offset=rank)
    c = case.cfg
    tau = args.tau
    for _ in range(warmup):
        case.step(tau)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    # timing hygiene: inputs larger than L2 need no flush; smaller ones (cfg1, cfg2) get L2 overwritten between steps,
    # outside the per-step events
    L2_BYTES = 126 << 20
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if case.input_bytes() <= L2_BYTES else None
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    for s in range(args.steps):
        if flush_buf is not None:
            flush_buf.fill_(s & 0xff)
        ev[s][0].record()
        case.fwd(tau)
        ev[s][1].record()
        case.bwd(tau)
        ev[s][2].record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    fwd_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    bwd_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps
    # the K steps run back to back on one stream: without a flush this is the elapsed time of the whole region
    total_ms = ev[0][0].elapsed_time(ev[-1][2]) if flush_buf is None else sum(e[0].elapsed_time(e[2]) for e in ev)
    total_ms = max_over_ranks(total_ms, dev)
    assert mala.device_status() == 0, "a device-side wait expired"
    ms_per_step = total_ms / args.steps
    step_flops = case.fwd_de + case.bwd_de
    value = whole_job_value(step_flops, world, ms_per_step)

    # The paper's operator benchmark: one tensor-parallel rank's head slice per GPU, timed as the synchronized wall
    # clock of the group (the slowest rank), the dense kernels on the same inputs beside it
    tp8 = None
    if args.workload == "tp8":
        def group_ms(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            t = time_cuda(fn, 0, max(args.steps, 5))
            return max_over_ranks(t, dev)
        case.fwd(0.0)
        d_f, d_b = group_ms(lambda: case.fwd(0.0)), group_ms(lambda: case.bwd(0.0))
        case.fwd(tau)
        m_f, m_b = group_ms(lambda: case.fwd(tau)), group_ms(lambda: case.bwd(tau))
        tp8 = {"ranks": world, "slice": f"Hq={c.Hq} Hkv={c.Hkv} N={c.N} d={c.d} per rank, preset {args.preset}, tau={tau}",
               "timing": "synchronized wall clock of the group: CUDA events per rank, maximum over the ranks",
               "mala": {"fwd_ms": m_f, "bwd_ms": m_b}, "dense": {"fwd_ms": d_f, "bwd_ms": d_b},
               "speedup_fwd": d_f / m_f, "speedup_bwd": d_b / m_b,
               "paper_context": "8 x H100, TP = 8, tau = 1, about 1024 retained slots per query on the authors' model: "
                                "forward 2.2x, backward 3.0x, decode 1.6x over FullAttn (other hardware and inputs; "
                                "context, not a target)"}

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    ts = case.tile_stats(tau)
    # roofline of the dominant kernel (the backward main kernel): executed tile FLOPs / launch duration
    bwd_exec = bwd_executed_flops(ts["bwd_legal"], ts["bwd_retained"], c.d)
    fwd_exec = fwd_executed_flops(ts["fwd_legal"], ts["fwd_retained"], c.d)
    ach = bwd_exec / (bwd_ms * 1e-3) / 1e12
    # DRAM bytes of the main kernels of one mala_bwd call (at tau > 0: first pass, list pass, one-pass kernel on the rows
    # left to it): from the table of committed ncu captures, null where none exists
    traffic, traffic_src = load_dram_traffic(args.workload, args.preset, tau)
    roofline = {"bound": "tensor", "kernel": "mala_bwd_kernel", "achieved": ach, "peak": peaks["tflops_sustained"],
                "unit": "TFLOP/s", "frac": ach / peaks["tflops_sustained"], "traffic": traffic,
                "traffic_source": traffic_src,
                "peak_source": f"{peaks['source']} (bf16 matmul, sustained)",
                "note": "duration = whole mala_bwd call (preprocess + main kernels + dQ convert; at tau > 0 the main "
                        "kernels are the first pass that tests every legal tile, the pass over its retained tiles and "
                        "the one-pass kernel on the rows left to it), so frac is a lower bound",
                "fwd": {"kernel": "mala_fwd_kernel", "achieved": fwd_exec / (fwd_ms * 1e-3) / 1e12,
                        "frac": fwd_exec / (fwd_ms * 1e-3) / 1e12 / peaks["tflops_sustained"]}}

    # ---------------------------------------------------------------- end to end: host buffers, copies timed
    # The step's inputs lie in pinned host memory, one contiguous block per KV-head group (the unit the path shards
    # by), and its results go back to pinned host memory.  The groups are independent, so the step is pipelined over
    # them through the library's own calls: group g + 1 is copied in and group g - 1 copied out while group g runs
    # forward and backward (three streams; the calls are asynchronous on the stream they are given).  A group's
    # forward waits only for its q, k, v (dO follows behind them) and its output goes back while its backward runs,
    # which shortens the pipeline's fill and drain.
    G = c.Hq // c.Hkv
    groups = []
    for g in range(c.Hkv):
        qs, ks, vs, dos = (case.q[:, :, g * G:(g + 1) * G], case.k[:, :, g:g + 1], case.v[:, :, g:g + 1],
                           case.do[:, :, g * G:(g + 1) * G])
        d_in = [t.contiguous() for t in (qs, ks, vs, dos)]
        d_out = [torch.empty_like(d_in[0]), torch.empty_like(d_in[0]), torch.empty_like(d_in[1]), torch.empty_like(d_in[2])]
        groups.append({"d_in": d_in, "d_out": d_out, "h_in": [t.cpu().pin_memory() for t in d_in],
                       "h_out": [torch.empty_like(t, device="cpu").pin_memory() for t in d_out]})
    g_lse = torch.empty((c.B, G, c.N), dtype=torch.float32, device=dev)
    g_ws = torch.empty(mala.workspace_bytes(mala.OP_BWD, c.B, G, 1, c.N, c.d), dtype=torch.uint8, device=dev)
    cin, cout = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def e2e_step():
        main = torch.cuda.current_stream()
        start = main.record_event()
        ready = []
        with torch.cuda.stream(cin):
            cin.wait_event(start)                       # the previous step has read these buffers
            for gr in groups:
                for d_, h_ in zip(gr["d_in"][:3], gr["h_in"][:3]):
                    d_.copy_(h_, non_blocking=True)
                ev_qkv = cin.record_event()
                gr["d_in"][3].copy_(gr["h_in"][3], non_blocking=True)
                ready.append((ev_qkv, cin.record_event()))
        cout.wait_event(start)
        for gr, (ev_qkv, ev_do) in zip(groups, ready):
            q_, k_, v_, do_ = gr["d_in"]
            o_, dq_, dk_, dv_ = gr["d_out"]
            main.wait_event(ev_qkv)
            mala.fwd(q_, k_, v_, case.scale, tau, out=o_, lse=g_lse, ws=g_ws)
            fwd_done = main.record_event()
            with torch.cuda.stream(cout):
                cout.wait_event(fwd_done)
                gr["h_out"][0].copy_(o_, non_blocking=True)
            main.wait_event(ev_do)
            mala.bwd(q_, k_, v_, o_, do_, g_lse, case.scale, tau, ws=g_ws, dq=dq_, dk=dk_, dv=dv_)
            done = main.record_event()
            with torch.cuda.stream(cout):
                cout.wait_event(done)
                for h_, d_ in zip(gr["h_out"][1:], gr["d_out"][1:]):
                    h_.copy_(d_, non_blocking=True)
        main.wait_stream(cout)
        main.wait_stream(cin)

    e2e_iters = max(1, min(args.steps, 5))
    e2e_ms = time_cuda(e2e_step, 1, e2e_iters)
    h2d = sum(t.numel() * t.element_size() for gr in groups for t in gr["h_in"])
    d2h = sum(t.numel() * t.element_size() for gr in groups for t in gr["h_out"])
    e2e = {"value": step_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "how": f"pipelined over the {c.Hkv} KV-head groups: copy-in, forward + backward, copy-out on three streams"}
    # the pipelined step computes what the single call computes
    torch.cuda.synchronize()
    case.step(tau)
    torch.cuda.synchronize()
    g_last = groups[-1]
    assert torch.equal(g_last["h_out"][0].to(dev), case.o[:, :, (c.Hkv - 1) * G:]), "e2e path: output mismatch"
    del groups, g_lse, g_ws

    # ---------------------------------------------------------------- CPU baseline: the oracle on a bounded sample
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import mala_oracle as orc
        case.fwd(tau)
        torch.cuda.synchronize()
        fl, dt, what = oracle_sample(case, tau, case.o.float().cpu(), case.lse)
        cpu_baseline = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle",
                        "sample": what, "seconds": dt}

    # ---------------------------------------------------------------- detail: MALA vs dense, per config
    detail = {}
    if world == 1 and not args.no_detail:
        it = args.detail_iters if args.detail_iters else 20                    # secondary rows
        main_w, main_it = (3, args.detail_iters) if args.detail_iters else (25, 100)   # MALA / dense rows
        for name in ("cfg3", "cfg4"):
            for preset in ("literal", "R", "S"):
                cs = case if (name == args.workload and preset == args.preset) else PrefillCase(name, preset, dev)
                cc = cs.cfg
                row = {}
                taus = {"mala": tau, "dense": 0.0}
                smp = ClockSampler(local_rank)
                smp.start()
                f_t = time_alternating({k: (lambda t_=t_: cs.fwd(t_)) for k, t_ in taus.items()}, main_w, main_it)
                b_t = time_alternating({k: (lambda t_=t_: cs.bwd(t_)) for k, t_ in taus.items()}, main_w, main_it,
                                       prep={k: (lambda t_=t_: cs.fwd(t_)) for k, t_ in taus.items()})
                mhz = smp.stop().get("sm_mhz")
                for label in taus:
                    f_ms, b_ms = f_t[label], b_t[label]
                    row[label] = {"fwd_ms": f_ms, "bwd_ms": b_ms,
                                  "fwd_dense_equiv_tflops": cs.fwd_de / f_ms / 1e9,
                                  "bwd_dense_equiv_tflops": cs.bwd_de / b_ms / 1e9}
                st = cs.tile_stats(tau)
                row["fwd_retained_frac"] = st["fwd_retained"] / st["fwd_legal"]
                row["bwd_retained_frac"] = st["bwd_retained"] / st["bwd_legal"]
                row["fwd_slots_per_query"] = st["fwd_retained"] * TILE * TILE / (cc.B * cc.Hq * cc.N)
                row["bwd_slots_per_query"] = st["bwd_retained"] * TILE * TILE / (cc.B * cc.Hq * cc.N)
                row["fwd_tensor_frac_on_executed"] = (fwd_executed_flops(st["fwd_legal"], st["fwd_retained"], cc.d)
                                                      / (row["mala"]["fwd_ms"] * 1e-3) / 1e12 / peaks["tflops_sustained"])
                row["bwd_tensor_frac_on_executed"] = (bwd_executed_flops(st["bwd_legal"], st["bwd_retained"], cc.d)
                                                      / (row["mala"]["bwd_ms"] * 1e-3) / 1e12 / peaks["tflops_sustained"])
                row["speedup_fwd"] = row["dense"]["fwd_ms"] / row["mala"]["fwd_ms"]
                row["speedup_bwd"] = row["dense"]["bwd_ms"] / row["mala"]["bwd_ms"]
                # SM clocks per tile and SM (time x sampled median SM clock / tiles): a retained tile from the dense
                # kernel, a skipped one from what the MALA kernel takes beyond the retained share of the dense time
                n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
                fr, fs_ = clk_per_tile(f_t["mala"], f_t["dense"], st["fwd_retained"], st["fwd_legal"], mhz, n_sm)
                br, bs_ = clk_per_tile(b_t["mala"], b_t["dense"], st["bwd_retained"], st["bwd_legal"], mhz, n_sm)
                row["clk_per_retained_tile"] = {"fwd": fr, "bwd": br}
                row["clk_per_skipped_tile"] = {"fwd": fs_, "bwd": bs_}
                row["sm_mhz_during_row"] = mhz
                if preset in ("R", "S"):             # per head type: where the retained tiles are, and what each type costs
                    row["by_head_type"] = head_type_leg(cs, tau, it)
                if preset == "S":                    # (this repository's addition, like R: every head sparse)
                    detail[f"{name}_{preset}"] = row
                    del cs
                    torch.cuda.empty_cache()
                    continue
                if name == "cfg4":                  # a 1024-query chunk against the 128K context, unsplit and split
                    row["chunk_last_1024"] = chunk_split_leg(cs, 1024, tau, it)
                if name == "cfg3":                  # chunked prefill: the last 8192 queries against all 32768 keys
                    row["chunk_last_8192"] = chunk_leg(cs, 8192, tau, it, peaks)
                if name == "cfg3":                  # the same heads on packed sequences of 16K + 8K + 5000 + 3192 rows
                    row["varlen_4seq_32768"] = varlen_leg(cc, preset, (16384, 8192, 5000, 3192), tau, it, peaks, dev)
                if name == "cfg3":                  # a serving-style batch of prefill chunks behind cached prefixes
                    row["serving_prefill_8x2048"] = serving_prefill_leg(cc, preset, tau, it, peaks, dev)
                if name == "cfg3":                  # the same shapes with 96-column heads (run on the 128-column kernels)
                    row["head_size_96"] = head_size_leg(cc, preset, 96, tau, it, peaks, dev)
                if name == "cfg3":                  # half the heads, 256 columns each: the forward's one-block-per-CTA kernel
                    row["head_size_256_fwd"] = head_size_256_fwd_leg(cc, preset, tau, it, peaks, dev)
                if name == "cfg3" and preset == "R":
                    row["fidelity_vs_dense"] = fidelity(cs, (1e-4, 1e-2, 1.0), it)
                detail[f"{name}_{preset}"] = row
                if cs is not case:
                    del cs
                    torch.cuda.empty_cache()
        # decode (cfg5): HBM roofline = bytes that must be read (K always, V of retained tiles) / time
        dcfg = W.decode_config("cfg5")
        for preset in ("literal", "D"):
            wd = W.make_decode(dcfg, preset=preset, device=dev)
            qd, kc, vc = wd["q"], wd["kcache"], wd["vcache"]
            wsd = torch.empty(mala.workspace_bytes(mala.OP_DECODE, dcfg.B, dcfg.Hq, dcfg.Hkv, dcfg.Nk, dcfg.d,
                                                   dcfg.num_splits), dtype=torch.uint8, device=dev)
            od = torch.empty_like(qd)
            row = {}
            for label, t_ in (("mala", tau), ("dense", 0.0)):
                us = 1e3 * time_cuda(lambda: mala.decode(qd, kc, vc, wd["scale"], t_, dcfg.num_splits, ws=wsd, out=od,
                                                          want_lse=False), 25, 100)
                _, _, st = mala.decode(qd, kc, vc, wd["scale"], t_, dcfg.num_splits, ws=wsd, out=od, stats=True)
                torch.cuda.synchronize()
                ret, leg = st.totals.cpu().tolist()
                need = (leg + ret) * TILE * dcfg.d * 2          # K tiles always, V tiles if retained
                row[label] = {"us": us, "retained_frac": ret / leg, "needed_gb": need / 1e9,
                              "achieved_gbs": need / (us * 1e-6) / 1e9,
                              "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
            row["speedup"] = row["dense"]["us"] / row["mala"]["us"]
            # the same cache stored as e4m3 with one scale per 128-key tile (mala_decode_fp8): half the bytes.  Two
            # layouts of the same [B,Nk,Hkv,d] view: key-major (a key's heads adjacent, the layout of the bf16 rows) and
            # head-major (a head's keys adjacent: a tile is then one contiguous 16 KB run instead of 128-byte pieces)
            k8, ks8, _ = W.quantize_cache_e4m3(kc)
            v8, vs8, _ = W.quantize_cache_e4m3(vc)
            head_major = lambda x: x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            f8 = {}
            for layout, (ka, va) in (("key_major", (k8, v8)), ("head_major", (head_major(k8), head_major(v8)))):
                lay = {}
                for label, t_ in (("mala", tau), ("dense", 0.0)):
                    us = 1e3 * time_cuda(lambda: mala.decode_fp8(qd, ka, va, ks8, vs8, wd["scale"], t_, dcfg.num_splits,
                                                                  ws=wsd, out=od, want_lse=False), 25, 100)
                    o8, _, st = mala.decode_fp8(qd, ka, va, ks8, vs8, wd["scale"], t_, dcfg.num_splits, ws=wsd, stats=True)
                    torch.cuda.synchronize()
                    ret, leg = st.totals.cpu().tolist()
                    need = (leg + ret) * TILE * dcfg.d              # one byte per element
                    o16, _, _ = mala.decode(qd, kc, vc, wd["scale"], t_, dcfg.num_splits)
                    lay[label] = {"us": us, "retained_frac": ret / leg, "needed_gb": need / 1e9,
                                  "achieved_gbs": need / (us * 1e-6) / 1e9,
                                  "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                                  "speedup_vs_bf16_cache": row[label]["us"] / us,
                                  "rel_l2_o_vs_bf16_cache": float((o8.float() - o16.float()).norm() / o16.float().norm())}
                f8[layout] = lay
                del ka, va
            # ... and in 256-key pages scattered over a shuffled pool (mala_decode_fp8_paged; scales per tile of a page)
            kp8, vp8, bt8, _ = W.paginate(k8, v8, 256, seed=7)
            sp = lambda sc: W.paginate_scales(sc, bt8, 256)
            ksp, vsp = sp(ks8), sp(vs8)
            pg8 = {}
            for label, t_ in (("mala", tau), ("dense", 0.0)):
                us = 1e3 * time_cuda(lambda: mala.decode_fp8_paged(qd, kp8, vp8, ksp, vsp, bt8, None, wd["scale"], t_,
                                                                    dcfg.num_splits, ws=wsd, out=od, want_lse=False), 25, 100)
                need = f8["key_major"][label]["needed_gb"] * 1e9
                pg8[label] = {"us": us, "achieved_gbs": need / (us * 1e-6) / 1e9,
                              "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
            f8["paged_256"] = pg8
            del kp8, vp8, bt8, ksp, vsp
            # ... and in 16-key pages (eight copies per tile; one scale per page, quantised page by page)
            kp, vp, bt16, _ = W.paginate(kc, vc, 16, seed=7)
            kp8, ksp, _ = W.quantize_cache_e4m3(kp, tile=16)
            vp8, vsp, _ = W.quantize_cache_e4m3(vp, tile=16)
            del kp, vp
            pg8 = {}
            for label, t_ in (("mala", tau), ("dense", 0.0)):
                us = 1e3 * time_cuda(lambda: mala.decode_fp8_paged(qd, kp8, vp8, ksp, vsp, bt16, None, wd["scale"], t_,
                                                                    dcfg.num_splits, ws=wsd, out=od, want_lse=False), 25, 100)
                need = f8["key_major"][label]["needed_gb"] * 1e9
                pg8[label] = {"us": us, "achieved_gbs": need / (us * 1e-6) / 1e9,
                              "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
            f8["paged_16"] = pg8
            del kp8, vp8, bt16, ksp, vsp
            # ... and with eight query heads per KV head (64 query heads on the same cache: two threads per key)
            q64 = qd.view(dcfg.B, 1, dcfg.Hkv, dcfg.Hq // dcfg.Hkv, dcfg.d)      # every group's heads, twice
            q64 = torch.cat([q64, q64], dim=3).reshape(dcfg.B, 1, 2 * dcfg.Hq, dcfg.d).contiguous()
            o64 = torch.empty_like(q64)
            ws64 = torch.empty(mala.workspace_bytes(mala.OP_DECODE, dcfg.B, 2 * dcfg.Hq, dcfg.Hkv, dcfg.Nk, dcfg.d,
                                                    dcfg.num_splits), dtype=torch.uint8, device=dev)
            g8 = {}
            for label, t_ in (("mala", tau), ("dense", 0.0)):
                us = 1e3 * time_cuda(lambda: mala.decode_fp8(q64, k8, v8, ks8, vs8, wd["scale"], t_, dcfg.num_splits,
                                                              ws=ws64, out=o64, want_lse=False), 25, 100)
                us16 = 1e3 * time_cuda(lambda: mala.decode(q64, kc, vc, wd["scale"], t_, dcfg.num_splits, ws=ws64,
                                                            out=o64, want_lse=False), 25, 100)
                need = f8["key_major"][label]["needed_gb"] * 1e9
                g8[label] = {"us": us, "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"], "bf16_cache_us": us16}
            f8["eight_heads_per_kv_head"] = g8
            del q64, o64, ws64
            # ... and two new tokens per sequence in one step (mala_decode_fp8_multi: eight rows per KV head, the same bytes)
            q2 = qd.repeat(1, 2, 1, 1).contiguous()
            o2t = torch.empty_like(q2)
            ws2 = torch.empty(mala.workspace_bytes(mala.OP_DECODE, dcfg.B * 2, dcfg.Hq, dcfg.Hkv, dcfg.Nk, dcfg.d,
                                                   dcfg.num_splits), dtype=torch.uint8, device=dev)
            m2 = {}
            for label, t_ in (("mala", tau), ("dense", 0.0)):
                us = 1e3 * time_cuda(lambda: mala.decode_fp8_multi(q2, k8, v8, ks8, vs8, wd["scale"], t_, dcfg.num_splits,
                                                                    ws=ws2, out=o2t, want_lse=False), 25, 100)
                _, _, st = mala.decode_fp8_multi(q2, k8, v8, ks8, vs8, wd["scale"], t_, dcfg.num_splits, ws=ws2, stats=True)
                ret, leg = st.totals.cpu().tolist()
                need = (leg + ret) * TILE * dcfg.d
                m2[label] = {"us": us, "retained_frac": ret / leg, "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                             "two_single_steps_us": 2 * f8["key_major"][label]["us"]}
            f8["multi_token_2"] = m2
            del q2, o2t, ws2
            row["e4m3_cache"] = f8
            del k8, v8, ks8, vs8
            # half the KV heads with 256 columns each (the same bytes per key): 64 KB tiles, two output accumulators
            w2 = W.custom_decode(dcfg.B, dcfg.Hq // 2, dcfg.Hkv // 2, dcfg.Nk, 256, dcfg.num_splits,
                                 group_types=dcfg.group_types[:dcfg.Hkv // 2], seed=dcfg.seed, preset=preset, device=dev)
            o2 = torch.empty_like(w2["q"])
            h256 = {"d": 256, "Hq": dcfg.Hq // 2, "Hkv": dcfg.Hkv // 2}
            for label, t_ in (("mala", tau), ("dense", 0.0)):
                us = 1e3 * time_cuda(lambda: mala.decode(w2["q"], w2["kcache"], w2["vcache"], w2["scale"], t_, dcfg.num_splits,
                                                          ws=wsd, out=o2, want_lse=False), 25, 100)
                _, _, st = mala.decode(w2["q"], w2["kcache"], w2["vcache"], w2["scale"], t_, dcfg.num_splits, ws=wsd, stats=True)
                torch.cuda.synchronize()
                ret, leg = st.totals.cpu().tolist()
                need = (leg + ret) * TILE * 256 * 2
                h256[label] = {"us": us, "retained_frac": ret / leg, "needed_gb": need / 1e9,
                               "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
            row["head_size_256"] = h256
            del w2, o2
            if preset == "D":                       # work and fidelity against the dense decode, tau up to 1
                o0, lse0, _ = mala.decode(qd, kc, vc, wd["scale"], 0.0, dcfg.num_splits, ws=wsd)
                o0, fid = o0.float(), {}
                for t_ in (1e-4, 1e-2, 1.0):
                    ot, lset, st = mala.decode(qd, kc, vc, wd["scale"], t_, dcfg.num_splits, ws=wsd, stats=True)
                    ret, leg = st.totals.cpu().tolist()
                    us = 1e3 * time_cuda(lambda: mala.decode(qd, kc, vc, wd["scale"], t_, dcfg.num_splits, ws=wsd,
                                                              out=od, want_lse=False), 25, 100)
                    fid[f"tau={t_:g}"] = {"us": us, "retained_frac": ret / leg,
                                          "rel_l2_o": float((ot.float() - o0).norm() / o0.norm()),
                                          "omitted_mass_max": float((1.0 - torch.exp(lset - lse0)).max()),
                                          "speedup": row["dense"]["us"] / us}
                row["fidelity_vs_dense"] = fid
                # fewer, longer splits: a split's normalizer grows with its length, so more of its tiles fall under the
                # threshold ("Fused decoding execution": the split-local test is the conservative one)
                sweep = {}
                S_auto = mala.decode_suggest_splits(dcfg.B, dcfg.Hkv, dcfg.Nk)
                for S in sorted({128, 64, 32, 16, S_auto}, reverse=True):
                    _, _, st = mala.decode(qd, kc, vc, wd["scale"], tau, S, ws=wsd, out=od, stats=True)
                    ret, leg = st.totals.cpu().tolist()
                    us = 1e3 * time_cuda(lambda: mala.decode(qd, kc, vc, wd["scale"], tau, S, ws=wsd, out=od,
                                                              want_lse=False), 25, 100)
                    need = (leg + ret) * TILE * dcfg.d * 2
                    sweep[f"splits={S}" + (" (suggested)" if S == S_auto else "")] = {"us": us, "retained_frac": ret / leg,
                                            "rel_l2_o": float((od.float() - o0).norm() / o0.norm()),
                                            "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                                            "speedup": row["dense"]["us"] / us}
                row["splits_sweep"] = sweep
                # four new tokens per sequence in one step (mala_decode_multi): 16 rows per KV head, the same bytes
                q4 = qd.repeat(1, 4, 1, 1).contiguous()
                o4 = torch.empty_like(q4)
                ws4 = torch.empty(mala.workspace_bytes(mala.OP_DECODE, dcfg.B * 4, dcfg.Hq, dcfg.Hkv, dcfg.Nk, dcfg.d,
                                                       dcfg.num_splits), dtype=torch.uint8, device=dev)
                mt = {}
                for label, t_ in (("mala", tau), ("dense", 0.0)):
                    _, _, st = mala.decode_multi(q4, kc, vc, wd["scale"], t_, dcfg.num_splits, ws=ws4, out=o4, stats=True)
                    ret, leg = st.totals.cpu().tolist()
                    us = 1e3 * time_cuda(lambda: mala.decode_multi(q4, kc, vc, wd["scale"], t_, dcfg.num_splits, ws=ws4,
                                                                    out=o4, want_lse=False), 25, 100)
                    need = (leg + ret) * TILE * dcfg.d * 2
                    mt[label] = {"us": us, "retained_frac": ret / leg,
                                 "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
                row["multi_token_4"] = mt
                del q4, o4, ws4
                # the same cache in 256-key pages scattered over a shuffled pool (mala_decode_paged)
                kp, vp, bt, _ = W.paginate(kc, vc, 256, seed=7)
                pg = {}
                for label, t_ in (("mala", tau), ("dense", 0.0)):
                    us = 1e3 * time_cuda(lambda: mala.decode_paged(qd, kp, vp, bt, None, wd["scale"], t_, dcfg.num_splits,
                                                                    ws=wsd, out=od, want_lse=False), 25, 100)
                    need = row[label]["needed_gb"] * 1e9
                    pg[label] = {"us": us, "achieved_gbs": need / (us * 1e-6) / 1e9,
                                 "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
                row["paged_256"] = pg
                del kp, vp, bt
                # ... and in 16-key pages (a tile is then put together from eight pages)
                kp, vp, bt, _ = W.paginate(kc, vc, 16, seed=7)
                pg = {}
                for label, t_ in (("mala", tau), ("dense", 0.0)):
                    us = 1e3 * time_cuda(lambda: mala.decode_paged(qd, kp, vp, bt, None, wd["scale"], t_, dcfg.num_splits,
                                                                    ws=wsd, out=od, want_lse=False), 25, 100)
                    need = row[label]["needed_gb"] * 1e9
                    pg[label] = {"us": us, "achieved_gbs": need / (us * 1e-6) / 1e9,
                                 "hbm_frac": need / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
                row["paged_16"] = pg
                del kp, vp, bt
            detail[f"cfg5_{preset}"] = row
            del wd, qd, kc, vc, wsd
            torch.cuda.empty_cache()

    out = {
        "metric": "mala_fwd_bwd_dense_equiv_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{c.name} {args.preset}: causal GQA B={c.B} Hq={c.Hq} Hkv={c.Hkv} N={c.N} d={c.d}, "
                               f"tau={tau}, fwd+bwd per step",
                   "l2": (f"inputs {case.input_bytes() / 1e6:.0f} MB per step exceed the 126 MB L2 (no flush needed)"
                          if flush_buf is None else
                          f"inputs {case.input_bytes() / 1e6:.0f} MB per step fit in L2: a 252 MB buffer is written between "
                          f"steps, outside the timed events"),
                   "protocol": ("main timed region: --warmup / --steps; detail rows: cfg3 / cfg4 MALA and dense kernels "
                                + ("25 warm-up + 100 timed iterations" if not args.detail_iters else
                                   f"3 warm-up + {args.detail_iters} timed iterations")
                                + ", in turn over two rounds; secondary rows (chunks, packed sequences, serving batch, "
                                  "head sizes, head types, fidelity) 3 + "
                                + str(args.detail_iters if args.detail_iters else 20) + "; decode rows 25 + 100"),
                   "parallelism": "replicas (one head slice per GPU, no collective)" if world > 1 else "single GPU"},
        "fwd_ms": fwd_ms, "bwd_ms": bwd_ms,
        "fwd_retained_frac": ts["fwd_retained"] / ts["fwd_legal"], "bwd_retained_frac": ts["bwd_retained"] / ts["bwd_legal"],
        "clocks": clocks, "e2e": e2e, "gpu_launches": (6 if tau > 0 else 4) * args.steps,   # (timed region per step: fwd + preprocess, main kernel(s) -- three at tau > 0 -- and dQ convert of the backward)
        "roofline": roofline, "cpu_baseline": cpu_baseline, "detail": detail,
    }
    if tp8 is not None:
        out["tp8"] = tp8
    print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
