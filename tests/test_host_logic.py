"""CPU-only checks of the boundary and the host logic: the C-ABI library loads and exports every symbol
the header declares, argument validation returns the documented codes without touching a GPU, the seeded
generators are deterministic and shaped as documented, and the benchmark's accounting and multi-rank
aggregation (gloo, world size 2) behave."""
import ctypes
import json
import math
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mala():
    from paper_2609_32712_b200 import build, mala as m
    build.build()
    m.lib()
    return m


def test_library_exports_every_declared_symbol(mala):
    hdr = open(os.path.join(ROOT, "include", "mala.h")).read()
    names = sorted(set(re.findall(r"\b(mala_[a-z_]+)\s*\(", hdr)))
    assert {"mala_fwd", "mala_bwd", "mala_decode", "mala_workspace_bytes", "mala_tile_shape", "mala_device_status",
            "mala_strerror", "mala_version"} <= set(names)
    L = mala.lib()
    for n in names:
        assert hasattr(L, n), f"libmala.so does not export {n}"


def test_host_only_queries(mala):
    assert mala.lib().mala_version() >= 100
    assert mala.tile_shape(mala.OP_FWD, 128) == (128, 128)
    assert mala.tile_shape(mala.OP_BWD, 64) == (128, 128)
    assert mala.tile_shape(mala.OP_DECODE, 128) == (0, 128)
    assert mala.tile_shape(mala.OP_FWD, 256) == (128, 128) and mala.tile_shape(mala.OP_DECODE, 200) == (0, 128)
    for op, d in ((mala.OP_FWD, 264), (mala.OP_BWD, 256), (mala.OP_BWD, 136), (mala.OP_DECODE, 512)):
        with pytest.raises(mala.MalaError):   # the forward and the decode step take up to 256 columns, the backward 128
            mala.tile_shape(op, d)
    # backward scratch: fp32 dQ accumulator + three fp32 per-row vectors, rows padded to whole tiles
    assert mala.workspace_bytes(mala.OP_BWD, 1, 2, 2, 1000, 64) == 2 * 1024 * 64 * 4 + 3 * 2 * 1024 * 4 + 256 + 256
    # (head sizes between the two kernel widths take the wider one's scratch)
    assert mala.workspace_bytes(mala.OP_BWD, 1, 2, 2, 1000, 96) == mala.workspace_bytes(mala.OP_BWD, 1, 2, 2, 1000, 128)
    assert mala.workspace_bytes(mala.OP_DECODE, 2, 8, 2, 4096, 40, 8) == mala.workspace_bytes(mala.OP_DECODE, 2, 8, 2, 4096, 64, 8)
    assert mala.workspace_bytes(mala.OP_DECODE, 8, 32, 8, 131072, 128, 128) == 8 * 32 * 128 * 128 * 4 + 8 * 32 * 128 * 4
    assert mala.workspace_bytes(mala.OP_DECODE, 8, 32, 8, 131072, 128, 0) == 0
    assert mala.workspace_bytes(mala.OP_DECODE, 8, 16, 4, 131072, 256, 128) == 8 * 16 * 128 * 256 * 4 + 8 * 16 * 128 * 4
    assert mala.workspace_bytes(mala.OP_DECODE, 2, 8, 2, 4096, 136, 8) == mala.workspace_bytes(mala.OP_DECODE, 2, 8, 2, 4096, 256, 8)
    assert mala.workspace_bytes(mala.OP_BWD, 1, 2, 2, 1000, 256) == 0     # (no backward above 128 columns)
    assert mala.lib().mala_strerror(-4).decode() == "workspace too small"
    # split count for decode: the smallest one that fills the SMs evenly (queue = items per SM x tiles per item)
    # with at least six items per SM and two tiles per split
    T = 1024
    queue = lambda S, groups=64, sms=148: -(-groups * S // sms) * -(-T // S)
    S = mala.decode_suggest_splits(8, 8, 131072, 148)
    lo = -(-6 * 148 // 64)
    best = min(queue(x) for x in range(lo, T // 2 + 1))
    assert S >= lo and queue(S) * 100 <= best * 104 and all(queue(x) * 100 > best * 104 for x in range(lo, S))
    assert S == 16                                                        # 1024 items: seven per SM, 64 tiles each
    assert mala.decode_suggest_splits(1024, 8, 4096, 148) == 1            # enough sequences: no split needed
    assert mala.decode_suggest_splits(1, 1, 100, 148) == 1                # one tile cannot be split
    assert mala.decode_suggest_splits(1, 1, 131072, 148) in range(128, 149)   # one head: about one split per SM
    assert mala.decode_suggest_splits(2, 8, 1024, 148) <= 4               # short cache: two tiles per split at least
    with pytest.raises(mala.MalaError):
        mala.decode_suggest_splits(0, 8, 4096, 148)


def test_argument_validation_codes(mala):
    L = mala.lib()
    buf = ctypes.create_string_buffer(4096)
    base = (ctypes.addressof(buf) + 255) & ~255
    tin = lambda off=0, sn=256: mala._TIn(base + off, 0, sn, 128)
    tout = lambda off=0, sn=256: mala._TOut(base + off, 0, sn, 128)
    f = lambda **kw: L.mala_fwd(kw.get("q", tin()), tin(), tin(), tout(), kw.get("lse", base), None, kw.get("B", 1),
                                kw.get("Hq", 2), kw.get("Hkv", 2), kw.get("N", 4), kw.get("d", 128), 1,
                                kw.get("scale", 0.1), kw.get("tau", 1e-4), None, 0, None)
    assert f(B=0) == -1 and f(N=-3) == -1
    assert f(tau=-1.0) == -1 and f(tau=float("nan")) == -1 and f(scale=0.0) == -1 and f(scale=float("inf")) == -1
    assert f(lse=None) == -1
    assert f(d=264) == -2 and f(d=512) == -2 and f(d=100) == -2 and f(d=0) == -2 and f(Hq=3, Hkv=2) == -2
    assert f(q=tin(off=2)) == -3 and f(q=tin(sn=130)) == -3
    # decode: too many packed heads, bad split count
    g = lambda **kw: L.mala_decode(tin(), tin(), tin(), tout(), None, None, 1, kw.get("Hq", 4), kw.get("Hkv", 1), 256,
                                   128, 0.1, 1e-4, kw.get("S", 2), kw.get("ws", base), 1 << 20, None)
    assert g(S=0) == -1 and g(ws=None) == -1 and g(Hq=32, Hkv=1) == -2
    # backward: workspace too small / misaligned
    h = lambda ws, n: L.mala_bwd(tin(), tin(), tin(), tin(), tin(), base, tout(), tout(), tout(), None, 1, 2, 2, 4, 128,
                                 1, 0.1, 1e-4, ws, n, None)
    assert h(base, 16) == -4 and h(base + 16, 1 << 20) == -3
    h256 = L.mala_bwd(tin(), tin(), tin(), tin(), tin(), base, tout(), tout(), tout(), None, 1, 2, 2, 4, 256, 1, 0.1,
                      1e-4, base, 1 << 20, None)
    assert h256 == -2                                                    # the backward stops at 128 columns
    if not torch.cuda.is_available():
        # valid arguments on a machine without a GPU: a loud CUDA error, never a silent fallback
        assert f() in (-5, -6)


def test_argument_validation_codes_of_the_general_shape_calls(mala):
    L = mala.lib()
    buf = ctypes.create_string_buffer(4096)
    base = (ctypes.addressof(buf) + 255) & ~255
    tin = lambda: mala._TIn(base, 0, 256, 128)
    tout = lambda: mala._TOut(base, 0, 256, 128)
    # chunked prefill: a causal chunk has no more queries than keys and may start anywhere
    fc = lambda Nq, Nk, causal=1: L.mala_fwd_chunk(tin(), tin(), tin(), tout(), base, None, 1, 2, 2, Nq, Nk, 128, causal,
                                                   0.1, 1e-4, None, 0, None)
    assert fc(512, 256) == -2 and fc(0, 256) == -1 and fc(100, 300) != -2
    bc = lambda Nq, Nk: L.mala_bwd_chunk(tin(), tin(), tin(), tin(), tin(), base, tout(), tout(), tout(), None, 1, 2, 2,
                                         Nq, Nk, 128, 1, 0.1, 1e-4, base, 1 << 20, None)
    assert bc(512, 256) == -2 and bc(128, 0) == -1 and bc(100, 300) != -2
    # key ranges: a positive count, scratch that is large enough and aligned
    fs = lambda S, ws=base, n=1 << 20: L.mala_fwd_chunk_split(tin(), tin(), tin(), tout(), base, None, 1, 2, 2, 128, 512, 128,
                                                              1, 0.1, 1e-4, S, ws, n, None)
    assert fs(0) == -1 and fs(4, ws=None) == -1 and fs(4, ws=base + 16) == -3 and fs(4, n=64) == -4
    assert mala.workspace_bytes(mala.OP_FWD, 1, 2, 2, 128, 128, 4) == 2 * 4 * 128 * 128 * 4 + 2 * 4 * 128 * 4
    assert mala.workspace_bytes(mala.OP_FWD, 1, 2, 2, 128, 128) == 256
    # packed sequences: cu_seqlens required, longest sequence within the total
    fv = lambda cu, total, mx: L.mala_fwd_varlen(tin(), tin(), tin(), cu, tout(), base, None, 2, 2, 2, total, mx, 128, 1,
                                                 0.1, 1e-4, None, 0, None)
    assert fv(None, 256, 128) == -1 and fv(base, 0, 128) == -1 and fv(base, 256, 512) == -2 and fv(base + 2, 256, 128) == -3
    fp = lambda cq, ck, mq=128, mk=256: L.mala_fwd_varlen_prefix(tin(), tin(), tin(), cq, ck, tout(), base, None, 2, 2, 2, 256,
                                                                 512, mq, mk, 128, 1, 0.1, 1e-4, None, 0, None)
    assert fp(None, base) == -1 and fp(base, None) == -1 and fp(base, base, mq=256, mk=128) == -2
    bp = lambda cq, ck, mq=128, mk=256, n=1 << 30: L.mala_bwd_varlen_prefix(
        tin(), tin(), tin(), tin(), tin(), base, cq, ck, tout(), tout(), tout(), None, 2, 2, 2, 256, 512, mq, mk, 128, 1, 0.1,
        1e-4, base, n, None)
    assert bp(None, base) == -1 and bp(base, None) == -1 and bp(base, base, mq=256, mk=128) == -2
    assert bp(base, base, n=1024) == -4        # scratch for total_q + 384 B rows
    fg = lambda page=128, bt=base, sl=base: L.mala_fwd_paged(tin(), tin(), tin(), base, bt, sl, tout(), base, None, 2, 2, 2, 256,
                                                             128, 8, page, 4, 128, 1, 0.1, 1e-4, None, 0, None)
    assert fg(page=48) == -2 and fg(page=4) == -2 and fg(bt=None) == -1 and fg(sl=None) == -1 and fg(bt=base + 2) == -3
    # several tokens per decode step: at most 16 rows per KV head, no more new tokens than keys
    dm = lambda Sq, Hq=4, Nk=256: L.mala_decode_multi(tin(), tin(), tin(), tout(), None, None, 1, Hq, 1, Nk, Sq, 128, 0.1,
                                                      1e-4, 2, base, 1 << 20, None)
    assert dm(0) == -1 and dm(5) == -2 and dm(2, Hq=16) == -2 and dm(4, Nk=3) == -2
    # paged decode: pages of whole tiles or of 8, 16, 32, 64 keys, a block table
    dp = lambda page, bt=base, Sq=1: L.mala_decode_paged(tin(), tin(), tin(), bt, None, tout(), None, None, 1, 4, 1, 8,
                                                         page, 4, Sq, 128, 0.1, 1e-4, 2, base, 1 << 20, None)
    assert dp(48) == -2 and dp(200) == -2 and dp(4) == -2 and dp(0) == -1 and dp(128, bt=None) == -1
    assert dp(128, bt=base + 1) == -3 and dp(16, bt=base + 1) == -3
    assert dp(128, Sq=0) == -1 and dp(128, Sq=5) == -2
    # workspace of a decode step with several tokens: as for that many more sequences
    assert mala.workspace_bytes(mala.OP_DECODE, 8 * 4, 32, 8, 131072, 128, 128) == 4 * mala.workspace_bytes(
        mala.OP_DECODE, 8, 32, 8, 131072, 128, 128)


def test_binding_has_no_cpu_fallback(mala):
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    q = torch.zeros(1, 128, 1, 128, dtype=torch.bfloat16)
    with pytest.raises(Exception):
        mala.fwd(q, q, q, 0.1, 0.0)


def test_generators_are_seeded_and_shaped():
    from paper_2609_32712_b200 import workloads as W
    c = W.prefill_config("cfg1")
    a, b = W.make_prefill(c), W.make_prefill(c)
    assert all(torch.equal(a[x], b[x]) for x in ("q", "k", "v", "do"))
    assert a["q"].shape == (1, 1024, 2, 64) and a["q"].dtype == torch.bfloat16 and a["scale"] == 1 / 8
    assert not torch.equal(W.make_prefill(c, seed=9)["q"], a["q"])
    for name, shp in (("cfg2", (1, 8192, 16, 4, 128)), ("cfg3", (1, 32768, 32, 8, 128)), ("cfg4", (1, 131072, 8, 2, 128))):
        cc = W.prefill_config(name)
        assert (cc.B, cc.N, cc.Hq, cc.Hkv, cc.d) == shp and len(cc.head_types) == cc.Hq
    d5 = W.decode_config("cfg5")
    assert (d5.B, d5.Hq, d5.Hkv, d5.Nk, d5.d, d5.num_splits) == (8, 32, 8, 131072, 128, 128)
    w = W.custom_decode(2, 8, 2, 1024, 128, 4, preset="D", group_types=["diffuse", "peaked"], seed=3)
    assert w["q"].shape == (2, 1, 8, 128) and w["kcache"].shape == (2, 1024, 2, 128)
    gate = w["kcache"][0, :, 0, 127].float()
    assert set(gate.unique().tolist()) == {0.0, -19.0} and (gate[-128:] == 0).all()
    assert (w["q"][0, 0, 4:, 127] == 19).all() and (w["q"][0, 0, :4, 127] != 19).all()


def test_planted_keys_raise_their_scores():
    from paper_2609_32712_b200 import workloads as W
    w = W.custom_prefill(1, 1, 1, 512, 64, head_types=["planted"], planted=4, seed=4)
    s = (w["q"][0, :, 0].float() @ w["k"][0, :, 0].float().T) * w["scale"]
    s = s.masked_fill(torch.triu(torch.ones(512, 512, dtype=torch.bool), 1), -1e9)
    top = s[64:].topk(4, dim=1).values.mean()
    assert top > 12.0            # about 3*sqrt(d) = 24 above the N(0, ~37) noise floor on the planted keys
    r = W.custom_prefill(1, 2, 1, 512, 128, head_types=["diffuse", "peaked"], seed=4, preset="R")
    assert torch.allclose(r["k"].float().norm(dim=-1), torch.full((1, 512, 1), math.sqrt(128)), rtol=1e-2)


def test_flop_model_matches_the_papers_accounting():
    sys.path.insert(0, ROOT)
    import bench
    # per token and layer: C_FullAttn = 8 a_n h d_qk + 6 a_n h d_v with a_n = (n + 1) / 2: 4 a_n h d of it forward
    n, h, d = 32768, 32, 128
    a_n = (n + 1) / 2
    assert abs(bench.fwd_dense_equiv_flops(1, h, n, d) / (n * 4 * a_n * h * d) - 1) < 1e-4
    assert abs((bench.fwd_dense_equiv_flops(1, h, n, d) + bench.bwd_dense_equiv_flops(1, h, n, d))
               / (n * (8 * a_n * h * d + 6 * a_n * h * d)) - 1) < 1e-4
    # C_MALA = 4 a_n h d (QK fwd + recompute) + 4 s_b h d + 2 s_f h d + 4 s_b h d, in tiles
    legal, rf, rb = 1000, 300, 200
    tile = 2 * 128 * 128 * d
    assert bench.fwd_executed_flops(legal, rf, d) + bench.bwd_executed_flops(legal, rb, d) == \
        2 * legal * tile + rf * tile + 4 * rb * tile
    assert bench.whole_job_value(1e12, 4, 1000.0) == pytest.approx(4.0)


def _gloo_worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
    dist.barrier()
    q.put((rank, ms, bench.whole_job_value(2e12, world, ms)))
    dist.destroy_process_group()


def test_multi_rank_timing_is_max_over_ranks_gloo():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 500)
    ps = [ctx.Process(target=_gloo_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    got = sorted(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]                 # both ranks see the slowest rank's time
    assert got[0][2] == pytest.approx(2 * 2e12 / 15e-3 / 1e12)  # whole-job value: all ranks' work / max time


def test_reference_arm_runs_the_oracle_on_cpu():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["dtype"] == "f64"
