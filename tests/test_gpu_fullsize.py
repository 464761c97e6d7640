"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot run 32K / 128K attention in full, so forward query blocks, backward key blocks / dQ
query blocks and decode (batch, KV head) units are sampled and computed one by one; properties that hold
at any size (nesting, tau = 0 retains everything, omitted-mass bound from the two normalizers) are checked
over the whole output."""
import numpy as np
import pytest
import torch

from paper_2609_32712_b200 import workloads as W
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mala():
    from paper_2609_32712_b200 import mala as m
    m.lib()
    return m


def _prefill_sampled(mala, oracle, name, preset, tau, fwd_units, key_units, dq_units):
    cfg = W.prefill_config(name)
    w = W.make_prefill(cfg, preset=preset, device="cuda")
    q, k, v, do = w["q"], w["k"], w["v"], w["do"]
    B, N, Hq, d = q.shape
    T = -(-N // 128)
    o, lse, fst = mala.fwd(q, k, v, w["scale"], tau, stats=True)
    dq, dk, dv, bst = mala.bwd(q, k, v, o, do, lse, w["scale"], tau, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    fm = fst.mask(T)
    bm = bst.mask(T)
    # properties over the whole problem
    assert (bm.transpose(2, 3) <= fm).all(), "backward support must be nested in forward support"
    tri = torch.tril(torch.ones(T, T, dtype=torch.bool, device=fm.device))
    assert not (fm & ~tri).any() and fm.diagonal(dim1=2, dim2=3).all()
    if tau == 0.0:
        assert (fm == tri).all() and (bm.transpose(2, 3) == tri).all()
    else:
        o_d, lse_d, _ = mala.fwd(q, k, v, w["scale"], 0.0)
        eps = 1.0 - torch.exp(lse - lse_d)
        assert eps.max() <= tau / (1 + tau) + 1e-3 and eps.min() >= -1e-3      # Proposition 1 (fp32 normalizers)
    assert torch.isfinite(o.float()).all() and torch.isfinite(dq.float()).all()
    assert torch.isfinite(dk.float()).all() and torch.isfinite(dv.float()).all()

    # sampled forward blocks
    ref = oracle.fwd(q, k, v, w["scale"], tau, 128, 128, units=fwd_units)
    fmc = fm.cpu().numpy()
    for (b, h, i) in fwd_units:
        rows = slice(i * 128, min(N, (i + 1) * 128))
        parity.check_mask(fmc[b, h, i], ref["mask"][b, h, i], ref["crit"][b, h, i], list(range(i, -1, -1)), tau,
                          i * 128 + 1)
        parity.check_output(o[b, rows, h].float().cpu().numpy(), ref["o"][b, rows, h])
        assert np.abs(lse[b, h, rows].cpu().numpy() - ref["lse"][b, h, rows]).max() <= parity.LSE_ABS
    # sampled backward blocks, fed with the same o / lse the GPU backward saw
    g = oracle.bwd(q, k, v, o, do, lse.cpu().numpy(), w["scale"], tau, 128, 128, key_units=key_units,
                   dq_units=dq_units)
    bmc = bm.cpu().numpy()
    G = Hq // k.shape[2]
    for (b, hk, j) in key_units:
        rows = slice(j * 128, min(N, (j + 1) * 128))
        parity.check_grad(dk[b, rows, hk].float().cpu().numpy(), g["dk"][b, rows, hk], f"dk block {j}")
        parity.check_grad(dv[b, rows, hk].float().cpu().numpy(), g["dv"][b, rows, hk], f"dv block {j}")
        for h in range(hk * G, (hk + 1) * G):
            om, oc = g["mask"][b, h, j], g["crit"][b, h, j]
            for i in range(T):
                if bool(bmc[b, h, j, i]) != (om[i] == 2):
                    assert om[i] != 0 and abs(oc[i]) <= parity.MASK_BAND, (h, j, i, oc[i])
    for (b, h, i) in dq_units:
        rows = slice(i * 128, min(N, (i + 1) * 128))
        parity.check_grad(dq[b, rows, h].float().cpu().numpy(), g["dq"][b, rows, h], f"dq block {i}")
    return float(fm.sum()) / float(tri.sum() * B * Hq)


@pytest.mark.parametrize("preset", ["literal", "R"])
@pytest.mark.parametrize("tau", [0.0, 1e-5, 1e-4, 1e-3])
def test_cfg2_8k(mala, oracle, preset, tau):
    T = 64
    fwd_units = [(0, 0, 0), (0, 3, 17), (0, 9, T - 1), (0, 15, 40)]
    key_units = [(0, 0, T - 1), (0, 2, 50), (0, 3, 30)]
    dq_units = [(0, 1, 5), (0, 12, T - 1)]
    frac = _prefill_sampled(mala, oracle, "cfg2", preset, tau, fwd_units, key_units, dq_units)
    if preset == "R" and tau > 0:
        assert frac < 0.8


@pytest.mark.parametrize("preset,tau", [("literal", 1e-4), ("R", 1e-4), ("literal", 0.0)])
def test_cfg3_32k(mala, oracle, preset, tau):
    T = 256
    fwd_units = [(0, 0, T - 1), (0, 1, 100), (0, 2, 200), (0, 31, 7)]
    key_units = [(0, 0, T - 2), (0, 5, 200)]
    dq_units = [(0, 6, 130)]
    _prefill_sampled(mala, oracle, "cfg3", preset, tau, fwd_units, key_units, dq_units)


@pytest.mark.parametrize("preset,tau", [("literal", 1e-4), ("R", 1e-4), ("literal", 0.0)])
def test_cfg4_128k(mala, oracle, preset, tau):
    T = 1024
    fwd_units = [(0, 1, T - 1), (0, 2, 300), (0, 4, 3)]
    key_units = [(0, 1, T - 3), (0, 0, 900)]
    dq_units = [(0, 7, 257)]
    _prefill_sampled(mala, oracle, "cfg4", preset, tau, fwd_units, key_units, dq_units)


@pytest.mark.parametrize("preset,tau", [("literal", 0.0), ("literal", 1e-4), ("D", 1e-4)])
def test_cfg5_decode_128k(mala, oracle, preset, tau):
    cfg = W.decode_config("cfg5")
    w = W.make_decode(cfg, preset=preset, device="cuda")
    q, kc, vc = w["q"], w["kcache"], w["vcache"]
    o, lse, st = mala.decode(q, kc, vc, w["scale"], tau, cfg.num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert torch.isfinite(o.float()).all()
    units = [(0, 0), (3, 1), (5, 2), (7, 7)]
    ref = oracle.decode(q, kc, vc, w["scale"], tau, cfg.num_splits, 128, units=units)
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    G = cfg.Hq // cfg.Hkv
    for (b, g) in units:
        for s in range(cfg.num_splits):
            parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                              tau, cfg.Nk)
        hs = slice(g * G, (g + 1) * G)
        parity.check_output(o[b, 0, hs].float().cpu().numpy(), ref["o"][b, hs])
        assert np.abs(lse[b, hs].cpu().numpy() - ref["lse"][b, hs]).max() <= parity.LSE_ABS
    if preset == "D":
        tot = st.totals.cpu().numpy()
        assert tot[0] < tot[1]
    if tau == 0.0:
        assert gm.all()


@pytest.mark.parametrize("tau", [0.0, 1e-4])
def test_cfg5_decode_128k_paged_variable_lengths(mala, oracle, tau):
    """cfg5 D held in 256-key pages scattered over a shuffled pool, the eight sequences of different lengths
    (one key, lengths that end inside a tile, inside a page and inside a split)."""
    cfg = W.decode_config("cfg5")
    w = W.make_decode(cfg, preset="D", device="cuda")
    lens = [131072, 100000, 65536 + 5, 131072, 1, 77777, 131072, 4097]
    kp, vp, bt, sl = W.paginate(w["kcache"], w["vcache"], 256, seqlens=lens, seed=3)
    del w["kcache"], w["vcache"]
    o, lse, st = mala.decode_paged(w["q"], kp, vp, bt, sl, w["scale"], tau, cfg.num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert torch.isfinite(o.float()).all()
    units = [(0, 0), (1, 3), (2, 5), (4, 2), (7, 7)]
    ref = oracle.decode_paged(w["q"][:, 0], kp, vp, bt.cpu().numpy(), lens, w["scale"], tau, cfg.num_splits, 128,
                              units=units)
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    G = cfg.Hq // cfg.Hkv
    for (b, g) in units:
        for s in range(cfg.num_splits):
            parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                              tau, lens[b])
        hs = slice(g * G, (g + 1) * G)
        parity.check_output(o[b, 0, hs].float().cpu().numpy(), ref["o"][b, hs])
        assert np.abs(lse[b, hs].cpu().numpy() - ref["lse"][b, hs]).max() <= parity.LSE_ABS
    legal = sum(-(-n // 128) for n in lens) * cfg.Hkv
    tot = st.totals.cpu().numpy()
    assert tot[1] == legal and (tot[0] == legal if tau == 0.0 else tot[0] < legal)


@pytest.mark.parametrize("preset,tau", [("R", 1e-4), ("literal", 0.0)])
def test_cfg3_32k_chunk_of_the_last_8192_queries(mala, oracle, preset, tau):
    """Chunked prefill at the benchmark's size: the last 8192 queries of cfg3 against all 32768 keys, sampled blocks
    against the oracle; the forward must also reproduce the rows of the equal-length call bit for bit."""
    cfg = W.prefill_config("cfg3")
    w = W.make_prefill(cfg, preset=preset, device="cuda")
    Nq, off = 8192, cfg.N - 8192
    q, k, v, do = w["q"][:, off:], w["k"], w["v"], w["do"][:, off:]
    Tq, Tk, a = Nq // 128, cfg.N // 128, off // 128
    o, lse, fst = mala.fwd_chunk(q, k, v, w["scale"], tau, stats=True)
    dq, dk, dv, bst = mala.bwd_chunk(q, k, v, o, do, lse, w["scale"], tau, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    o_full, lse_full, _ = mala.fwd(w["q"], k, v, w["scale"], tau)
    assert torch.equal(o_full[:, off:], o) and torch.equal(lse_full[:, :, off:], lse)
    fm, bm = fst.mask(Tk), bst.mask(Tq)
    assert (bm.transpose(2, 3) <= fm).all(), "backward support must be nested in forward support"
    legal = torch.tril(torch.ones(Tq, Tk, dtype=torch.bool, device=fm.device), diagonal=a)
    assert not (fm & ~legal).any()
    if tau == 0.0:
        assert (fm == legal).all() and (bm.transpose(2, 3) == legal).all()
    for t in (dq, dk, dv):
        assert torch.isfinite(t.float()).all()
    fwd_units = [(0, 0, Tq - 1), (0, 1, 0), (0, 2, 33), (0, 31, 7)]
    ref = oracle.fwd(q, k, v, w["scale"], tau, 128, 128, units=fwd_units)
    fmc = fm.cpu().numpy()
    for (b, h, i) in fwd_units:
        rows = slice(i * 128, (i + 1) * 128)
        parity.check_mask(fmc[b, h, i], ref["mask"][b, h, i], ref["crit"][b, h, i], list(range(i + a, -1, -1)), tau,
                          i * 128 + 1 + off)
        parity.check_output(o[b, rows, h].float().cpu().numpy(), ref["o"][b, rows, h])
        assert np.abs(lse[b, h, rows].cpu().numpy() - ref["lse"][b, h, rows]).max() <= parity.LSE_ABS
    key_units = [(0, 0, Tk - 2), (0, 5, 100), (0, 3, a + 10)]     # after, before and inside the chunk's own positions
    dq_units = [(0, 6, 40)]
    g = oracle.bwd(q, k, v, o, do, lse.cpu().numpy(), w["scale"], tau, 128, 128, key_units=key_units,
                   dq_units=dq_units)
    bmc = bm.cpu().numpy()
    G = cfg.Hq // cfg.Hkv
    for (b, hk, j) in key_units:
        rows = slice(j * 128, (j + 1) * 128)
        parity.check_grad(dk[b, rows, hk].float().cpu().numpy(), g["dk"][b, rows, hk], f"dk block {j}")
        parity.check_grad(dv[b, rows, hk].float().cpu().numpy(), g["dv"][b, rows, hk], f"dv block {j}")
        for h in range(hk * G, (hk + 1) * G):
            om, oc = g["mask"][b, h, j], g["crit"][b, h, j]
            for i in range(Tq):
                if bool(bmc[b, h, j, i]) != (om[i] == 2):
                    assert om[i] != 0 and abs(oc[i]) <= parity.MASK_BAND, (h, j, i, oc[i])
    for (b, h, i) in dq_units:
        rows = slice(i * 128, (i + 1) * 128)
        parity.check_grad(dq[b, rows, h].float().cpu().numpy(), g["dq"][b, rows, h], f"dq block {i}")


def _check_decode_units(oracle, q, kd, vd, scale, tau, S, units, G, o, lse, gm):
    """Sampled (sequence, KV head) units of a decode call, each against the oracle on its own slice of the cache
    (kd, vd: the values the call works on, fp32 or bf16, on the GPU; only the slices travel to the host)."""
    for (b, g) in units:
        hs = slice(g * G, (g + 1) * G)
        n = kd.shape[1]
        qs, ks, vs = q[b:b + 1, :, hs].cpu(), kd[b:b + 1, :, g:g + 1].cpu(), vd[b:b + 1, :, g:g + 1].cpu()
        ref = oracle.decode(qs, ks, vs, scale, tau, S, 128)
        ref_abs = oracle.decode(qs, ks, vs.abs(), scale, tau, S, 128)
        tps = ref["mask"].shape[-1]
        for s in range(S):
            parity.check_mask(gm[b, g, s], ref["mask"][0, 0, s], ref["crit"][0, 0, s], list(range(tps - 1, -1, -1)), tau, n)
        parity.check_output(o[b, 0, hs].float().cpu().numpy(), ref["o"][0], a_ref=ref_abs["o"][0])
        assert np.abs(lse[b, hs].cpu().numpy() - ref["lse"][0]).max() <= parity.LSE_ABS


@pytest.mark.parametrize("heads", [32, 64])
@pytest.mark.parametrize("preset,tau", [("literal", 0.0), ("D", 1e-4)])
def test_cfg5_decode_128k_over_an_e4m3_cache(mala, oracle, preset, tau, heads):
    """The bench's e4m3 rows: cfg5 with the cache stored as e4m3 codes and a scale per tile, with cfg5's four and with
    eight query heads per KV head (every group's heads twice)."""
    cfg = W.decode_config("cfg5")
    w = W.make_decode(cfg, preset=preset, device="cuda")
    G0 = cfg.Hq // cfg.Hkv
    q = w["q"]
    if heads == 64:
        q = q.view(cfg.B, 1, cfg.Hkv, G0, cfg.d)
        q = torch.cat([q, q], dim=3).reshape(cfg.B, 1, 2 * cfg.Hq, cfg.d).contiguous()
    k8, ks, kd = W.quantize_cache_e4m3(w["kcache"])
    del w["kcache"]
    v8, vs, vd = W.quantize_cache_e4m3(w["vcache"])
    del w["vcache"]
    o, lse, st = mala.decode_fp8(q, k8, v8, ks, vs, w["scale"], tau, cfg.num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert torch.isfinite(o.float()).all()
    tps = -(-(-(-cfg.Nk // cfg.num_splits)) // 128)
    gm = st.mask(tps).cpu().numpy()
    _check_decode_units(oracle, q, kd, vd, w["scale"], tau, cfg.num_splits, [(0, 0), (5, 2), (7, 7)], heads // cfg.Hkv,
                        o, lse, gm)
    tot = st.totals.cpu().numpy()
    assert tot[1] == cfg.B * cfg.Hkv * (cfg.Nk // 128) and (tot[0] == tot[1] if tau == 0.0 else tot[0] < tot[1])


@pytest.mark.parametrize("preset,tau", [("literal", 0.0), ("D", 1e-4)])
def test_cfg5_decode_128k_with_256_column_heads(mala, oracle, preset, tau):
    """The bench's 256-column decode row: cfg5's bytes per key on half the heads of twice the size."""
    cfg = W.decode_config("cfg5")
    Hq, Hkv = cfg.Hq // 2, cfg.Hkv // 2
    w = W.custom_decode(cfg.B, Hq, Hkv, cfg.Nk, 256, cfg.num_splits, group_types=cfg.group_types[:Hkv], seed=cfg.seed,
                        preset=preset, device="cuda")
    o, lse, st = mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], tau, cfg.num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert torch.isfinite(o.float()).all()
    tps = -(-(-(-cfg.Nk // cfg.num_splits)) // 128)
    gm = st.mask(tps).cpu().numpy()
    _check_decode_units(oracle, w["q"], w["kcache"], w["vcache"], w["scale"], tau, cfg.num_splits, [(0, 0), (6, 3)],
                        Hq // Hkv, o, lse, gm)
    if tau == 0.0:
        assert gm.all()


@pytest.mark.parametrize("preset,tau", [("literal", 0.0), ("R", 1e-4)])
def test_cfg3_32k_forward_with_256_column_heads(mala, oracle, preset, tau):
    """The bench's 256-column forward row: cfg3's shape with half the heads of twice the size (one query block per CTA)."""
    cfg = W.prefill_config("cfg3")
    Hq, Hkv = cfg.Hq // 2, cfg.Hkv // 2
    w = W.custom_prefill(cfg.B, Hq, Hkv, cfg.N, 256, head_types=cfg.head_types[:Hq], seed=cfg.seed, preset=preset,
                         device="cuda")
    q, k, v = w["q"], w["k"], w["v"]
    T = cfg.N // 128
    o, lse, st = mala.fwd(q, k, v, w["scale"], tau, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert torch.isfinite(o.float()).all()
    fm = st.mask(T)
    tri = torch.tril(torch.ones(T, T, dtype=torch.bool, device=fm.device))
    assert not (fm & ~tri).any() and fm.diagonal(dim1=2, dim2=3).all()
    if tau == 0.0:
        assert (fm == tri).all()
    else:
        _, lse_d, _ = mala.fwd(q, k, v, w["scale"], 0.0)
        eps = 1.0 - torch.exp(lse - lse_d)
        assert eps.max() <= tau / (1 + tau) + 1e-3 and eps.min() >= -1e-3      # Proposition 1 (fp32 normalizers)
        assert fm.sum() < tri.sum() * Hq
    units = [(0, 1, T - 1), (0, 2, 100), (0, 5, 3), (0, 15, 200)]
    ref = oracle.fwd(q, k, v, w["scale"], tau, 128, 128, units=units)
    ref_abs = oracle.fwd(q, k, v.abs(), w["scale"], tau, 128, 128, units=units)
    fmc = fm.cpu().numpy()
    for (b, h, i) in units:
        rows = slice(i * 128, (i + 1) * 128)
        parity.check_mask(fmc[b, h, i], ref["mask"][b, h, i], ref["crit"][b, h, i], list(range(i, -1, -1)), tau, i * 128 + 1)
        parity.check_output(o[b, rows, h].float().cpu().numpy(), ref["o"][b, rows, h], a_ref=ref_abs["o"][b, rows, h])
        assert np.abs(lse[b, h, rows].cpu().numpy() - ref["lse"][b, h, rows]).max() <= parity.LSE_ABS
