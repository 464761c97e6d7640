"""GPU parity of mala_decode (split-KV decode through the C ABI) against the fp64 oracle."""
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


def _run_and_check(mala, oracle, w, tau, num_splits, units=None, rounding_bound=False):
    q, kc, vc = (w[x].cuda() for x in ("q", "kcache", "vcache"))
    B, _, Hq, d = q.shape
    Nk, Hkv = kc.shape[1], kc.shape[2]
    G = Hq // Hkv
    o, lse, st = mala.decode(q, kc, vc, w["scale"], tau, num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    _, Bk = mala.tile_shape(mala.OP_DECODE, d)
    ref = oracle.decode(w["q"], w["kcache"], w["vcache"], w["scale"], tau, num_splits, Bk, units=units)
    ref_abs = (oracle.decode(w["q"], w["kcache"], w["vcache"].abs(), w["scale"], tau, num_splits, Bk, units=units)
               if rounding_bound else None)          # a = sum_k p_k |v_k| for parity.check_output's rounding bound
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()                    # [B,Hkv,S,tps]
    if units is None:
        units = [(b, g) for b in range(B) for g in range(Hkv)]
    o_c, lse_c = o.float().cpu().numpy()[:, 0], lse.cpu().numpy()
    skipped = retained = flips = 0
    for (b, g) in units:
        for s in range(num_splits):
            flips += parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s],
                                       list(range(tps - 1, -1, -1)), tau, Nk, Bk)
            assert int(st.retained[b, g, s]) == int(gm[b, g, s].sum())
        hs = slice(g * G, (g + 1) * G)
        parity.check_output(o_c[b, hs], ref["o"][b, hs], a_ref=ref_abs["o"][b, hs] if rounding_bound else None)
        assert np.abs(lse_c[b, hs] - ref["lse"][b, hs]).max() <= parity.LSE_ABS
        skipped += int((ref["mask"][b, g] == 1).sum())
        retained += int((ref["mask"][b, g] == 2).sum())
    return dict(skipped=skipped, retained=retained, flips=flips, totals=st.totals.cpu().numpy())


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv", [(128, 1, 4, 1), (1024, 4, 8, 2), (1000, 3, 4, 4), (4096, 8, 16, 2),
                                          (700, 8, 2, 1)])
def test_decode_literal(mala, oracle, Nk, S, Hq, Hkv, tau):
    w = W.custom_decode(2, Hq, Hkv, Nk, 128, S, seed=Nk + S)
    _run_and_check(mala, oracle, w, tau, S)


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv", [(300, 2, 6, 2), (2048, 16, 16, 1), (8192, 64, 10, 2), (1536, 4, 3, 1)])
def test_decode_group_sizes_and_short_items(mala, oracle, Nk, S, Hq, Hkv, tau):
    """Group sizes that are not powers of two (3, 5), the largest one (16), and more work items than SMs with one or
    two tiles each (the partial output of an item is then written at the end of the next item)."""
    w = W.custom_decode(2, Hq, Hkv, Nk, 128, S, seed=Nk + S + Hq)
    _run_and_check(mala, oracle, w, tau, S)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("Nk,S", [(8192, 8), (8192, 2), (5000, 4)])
def test_decode_gated_keys_skip_value_tiles(mala, oracle, Nk, S, tau):
    w = W.custom_decode(2, 8, 2, Nk, 128, S, group_types=["diffuse", "peaked"], seed=3, preset="D")
    res = _run_and_check(mala, oracle, w, tau, S)
    assert res["skipped"] > 0, "workload must exercise skipping"
    assert res["totals"][1] == res["retained"] + res["skipped"]


def test_decode_with_the_suggested_split_count(mala, oracle):
    w = W.custom_decode(2, 8, 2, 20000, 128, 1, group_types=["diffuse", "peaked"], seed=77, preset="D")
    S = mala.decode_suggest_splits(2, 2, 20000)              # SM count of the current device
    assert 1 <= S <= 157 // 2
    assert S == mala.decode_suggest_splits(2, 2, 20000, torch.cuda.get_device_properties(0).multi_processor_count)
    _run_and_check(mala, oracle, w, 1e-4, S)


def test_decode_tau_zero_is_split_invariant(mala):
    w = W.custom_decode(1, 8, 2, 4096, 128, 4, seed=11)
    q, kc, vc = (w[x].cuda() for x in ("q", "kcache", "vcache"))
    o1, l1, _ = mala.decode(q, kc, vc, w["scale"], 0.0, 1)
    o2, l2, _ = mala.decode(q, kc, vc, w["scale"], 0.0, 16)
    assert (o1.float() - o2.float()).abs().max() <= 1e-2
    assert (l1 - l2).abs().max() <= 1e-4


def test_decode_strided_cache_view(mala, oracle):
    # caches stored [B, Hkv, Nk, d] and passed as a permuted view
    w = W.custom_decode(1, 4, 2, 1024, 128, 4, seed=13)
    q = w["q"].cuda()
    kc = w["kcache"].cuda().permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vc = w["vcache"].cuda().permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    o, lse, _ = mala.decode(q, kc, vc, w["scale"], 0.0, 4)
    ref = oracle.decode(w["q"], w["kcache"], w["vcache"], w["scale"], 0.0, 4, 128)
    parity.check_output(o.float().cpu().numpy()[:, 0], ref["o"])


def _run_paged(mala, oracle, w, tau, num_splits, page_size, seqlens, seed=0, rounding_bound=False):
    kp, vp, bt, lens = W.paginate(w["kcache"], w["vcache"], page_size, seqlens=seqlens, seed=seed)
    q = w["q"].cuda()
    B, _, Hq, d = q.shape
    Hkv = kp.shape[2]
    G = Hq // Hkv
    o, lse, st = mala.decode_paged(q, kp.cuda(), vp.cuda(), bt.cuda(), lens.cuda() if seqlens is not None else None,
                                   w["scale"], tau, num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    _, Bk = mala.tile_shape(mala.OP_DECODE, d)
    ref = oracle.decode_paged(w["q"][:, 0], kp, vp, bt.numpy(), lens.numpy() if seqlens is not None else None,
                              w["scale"], tau, num_splits, Bk)
    ref_abs = (oracle.decode_paged(w["q"][:, 0], kp, vp.abs(), bt.numpy(), lens.numpy() if seqlens is not None else None,
                                   w["scale"], tau, num_splits, Bk) if rounding_bound else None)
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy()[:, 0], lse.cpu().numpy()
    skipped = retained = 0
    for b in range(B):
        n = int(lens[b])
        for g in range(Hkv):
            for s in range(num_splits):
                parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                                  tau, max(n, 1), Bk)
                assert int(st.retained[b, g, s]) == int(gm[b, g, s].sum())
            hs = slice(g * G, (g + 1) * G)
            parity.check_output(o_c[b, hs], ref["o"][b, hs], a_ref=ref_abs["o"][b, hs] if rounding_bound else None)
            if n > 0:
                assert np.abs(lse_c[b, hs] - ref["lse"][b, hs]).max() <= parity.LSE_ABS
            else:
                assert np.isneginf(lse_c[b, hs]).all() and (o_c[b, hs] == 0).all()
            skipped += int((ref["mask"][b, g] == 1).sum())
            retained += int((ref["mask"][b, g] == 2).sum())
    tot = st.totals.cpu().numpy()
    assert tot[1] == retained + skipped
    return dict(skipped=skipped, retained=retained)


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv,page,lens", [
    (1024, 4, 8, 2, 128, None),                        # one tile per page, every sequence full
    (2048, 4, 4, 1, 256, [2048, 1000, 129]),           # two tiles per page, ragged lengths, empty trailing splits
    (1536, 3, 6, 2, 512, [1, 1536, 0, 700]),           # a split per page; one key; no key at all
    (8192, 64, 8, 2, 128, [8192, 5000, 128, 3333]),    # more work items than SMs, one tile each
])
def test_decode_paged_literal(mala, oracle, Nk, S, Hq, Hkv, page, lens, tau):
    B = 2 if lens is None else len(lens)
    w = W.custom_decode(B, Hq, Hkv, Nk, 128, S, seed=Nk + S + page)
    _run_paged(mala, oracle, w, tau, S, page, lens, seed=page)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
def test_decode_paged_gated_keys_skip_value_tiles(mala, oracle, tau):
    w = W.custom_decode(3, 8, 2, 8192, 128, 8, group_types=["diffuse", "peaked"], seed=5, preset="D")
    res = _run_paged(mala, oracle, w, tau, 8, 256, [8192, 4096 + 77, 2500], seed=9)
    assert res["skipped"] > 0, "workload must exercise skipping"


def test_decode_paged_identity_table_equals_contiguous_call(mala):
    # pages laid out in order are the contiguous cache: both entry points must give the same bits
    w = W.custom_decode(2, 8, 2, 4096, 128, 8, group_types=["diffuse", "peaked"], seed=21, preset="D")
    q, kc, vc = (w[x].cuda() for x in ("q", "kcache", "vcache"))
    bt = torch.arange(2 * 16, dtype=torch.int32, device="cuda").reshape(2, 16)
    for tau in (0.0, 1e-4):
        o1, l1, s1 = mala.decode(q, kc, vc, w["scale"], tau, 8, stats=True)
        o2, l2, s2 = mala.decode_paged(q, kc.reshape(32, 256, 2, 128), vc.reshape(32, 256, 2, 128), bt, None,
                                       w["scale"], tau, 8, stats=True)
        assert torch.equal(o1, o2) and torch.equal(l1, l2)
        assert torch.equal(s1.retained, s2.retained)


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv,page,lens", [
    (1024, 4, 8, 2, 16, [1024, 500, 17]),              # 16-key pages: eight copies per tile
    (2048, 4, 4, 1, 64, [2048, 1000, 129, 0]),
    (1520, 3, 4, 2, 32, [1520, 33]),                   # the positions end inside a tile: table entries past the last page
    (4096, 16, 16, 2, 8, [4096, 2047]),
])
def test_decode_paged_with_pages_smaller_than_a_tile(mala, oracle, Nk, S, Hq, Hkv, page, lens, tau):
    w = W.custom_decode(len(lens), Hq, Hkv, Nk, 128, S, group_types=["diffuse", "peaked"], seed=Nk + page, preset="D")
    _run_paged(mala, oracle, w, tau, S, page, lens, seed=page)


def test_decode_paged_rejects_pages_that_do_not_tile(mala):
    q = torch.zeros((1, 1, 4, 128), dtype=torch.bfloat16, device="cuda")
    pages = torch.zeros((4, 48, 1, 128), dtype=torch.bfloat16, device="cuda")
    bt = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(mala.MalaError) as e:
        mala.decode_paged(q, pages, pages, bt, None, 0.1, 0.0, 1)
    assert e.value.code < 0


def _run_multi(mala, oracle, w, Sq, tau, num_splits, seed=0):
    """The decode workload's cache with Sq new tokens: their queries are drawn like the workload's one query."""
    kc, vc = w["kcache"], w["vcache"]
    B, Nk, Hkv, d = kc.shape
    Hq = w["q"].shape[2]
    G = Hq // Hkv
    gen = torch.Generator(device="cpu")
    gen.manual_seed(1000 + seed)
    q = w["q"].float().repeat(1, Sq, 1, 1)
    q[..., : d - 1] += 0.5 * torch.randn((B, Sq, Hq, d - 1), generator=gen)   # (the last feature keeps the key gate)
    q = q.to(torch.bfloat16)
    o, lse, st = mala.decode_multi(q.cuda(), kc.cuda(), vc.cuda(), w["scale"], tau, num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ref = oracle.decode_multi(q, kc, vc, w["scale"], tau, num_splits, 128)
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy(), lse.cpu().numpy()
    for b in range(B):
        for g in range(Hkv):
            for s in range(num_splits):
                parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                                  tau, Nk - Sq + 1, 128)
                assert int(st.retained[b, g, s]) == int(gm[b, g, s].sum())
    parity.check_output(o_c, ref["o"])
    assert np.abs(lse_c - ref["lse"]).max() <= parity.LSE_ABS
    return int((ref["mask"] == 1).sum())


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv,Sq", [(1024, 4, 8, 2, 4), (1000, 3, 4, 4, 16), (2050, 4, 4, 2, 5),
                                             (1027, 2, 6, 2, 4), (640, 5, 2, 1, 8), (4096, 8, 16, 2, 2)])
def test_decode_multi_literal(mala, oracle, Nk, S, Hq, Hkv, Sq, tau):
    """Several new tokens per step; (2050, 5) and (1027, 4): the newest key block holds fewer keys than there are
    new tokens, so its first rows see none of it."""
    w = W.custom_decode(2, Hq, Hkv, Nk, 128, S, seed=Nk + S + Sq)
    _run_multi(mala, oracle, w, Sq, tau, S, seed=Sq)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
def test_decode_multi_gated_keys_skip_value_tiles(mala, oracle, tau):
    w = W.custom_decode(2, 8, 2, 8192, 128, 8, group_types=["diffuse", "peaked"], seed=3, preset="D")
    assert _run_multi(mala, oracle, w, 4, tau, 8) > 0, "workload must exercise skipping"


def test_decode_multi_of_one_token_equals_decode(mala):
    w = W.custom_decode(2, 8, 2, 4096, 128, 8, group_types=["diffuse", "peaked"], seed=21, preset="D")
    q, kc, vc = (w[x].cuda() for x in ("q", "kcache", "vcache"))
    for tau in (0.0, 1e-4):
        o1, l1, _ = mala.decode(q, kc, vc, w["scale"], tau, 8)
        o2, l2, _ = mala.decode_multi(q, kc, vc, w["scale"], tau, 8)
        assert torch.equal(o1, o2) and torch.equal(l1, l2.reshape(l1.shape))


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv,page,Sq,lens", [
    (2048, 4, 8, 2, 256, 4, [2048, 1000, 129, 3]),     # 16 rows; the last sequence holds fewer keys than new tokens
    (1536, 3, 4, 2, 128, 3, [1536, 1, 700]),
])
def test_decode_paged_with_several_new_tokens(mala, oracle, Nk, S, Hq, Hkv, page, Sq, lens, tau):
    B = len(lens)
    w = W.custom_decode(B, Hq, Hkv, Nk, 128, S, group_types=["diffuse", "peaked"], seed=Nk + Sq, preset="D")
    kp, vp, bt, sl = W.paginate(w["kcache"], w["vcache"], page, seqlens=lens, seed=Sq)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(77)
    q = w["q"].float().repeat(1, Sq, 1, 1)
    q[..., :127] += 0.5 * torch.randn((B, Sq, Hq, 127), generator=gen)
    q = q.to(torch.bfloat16)
    o, lse, st = mala.decode_paged(q.cuda(), kp.cuda(), vp.cuda(), bt.cuda(), sl.cuda(), w["scale"], tau, S, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ref = oracle.decode_paged(q, kp, vp, bt.numpy(), lens, w["scale"], tau, S, 128)
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    for b in range(B):
        for g in range(Hkv):
            for s in range(S):
                parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                                  tau, max(lens[b] - Sq + 1, 1), 128)
    o_c, lse_c = o.float().cpu().numpy(), lse.cpu().numpy()
    parity.check_output(o_c, ref["o"])
    fin = np.isfinite(ref["lse"])
    assert np.abs(lse_c[fin] - ref["lse"][fin]).max() <= parity.LSE_ABS
    assert np.isneginf(lse_c[~fin]).all() and (o_c[~fin] == 0).all()


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv", [(1024, 4, 8, 2), (1000, 3, 4, 4), (4096, 8, 16, 1), (300, 2, 6, 2)])
def test_decode_head_size_64(mala, oracle, Nk, S, Hq, Hkv, tau):
    w = W.custom_decode(2, Hq, Hkv, Nk, 64, S, seed=Nk + S)
    _run_and_check(mala, oracle, w, tau, S)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
def test_decode_head_size_64_gated_paged_several_tokens(mala, oracle, tau):
    w = W.custom_decode(2, 8, 2, 8192, 64, 8, group_types=["diffuse", "peaked"], seed=3, preset="D")
    res = _run_and_check(mala, oracle, w, tau, 8)
    assert res["skipped"] > 0, "workload must exercise skipping"
    _run_paged(mala, oracle, w, tau, 8, 256, [8192, 4096 + 77], seed=9)
    assert _run_multi(mala, oracle, w, 3, tau, 8) > 0


def _run_fp8(mala, oracle, w, tau, num_splits, rounding_bound=False):
    """mala_decode_fp8 on the e4m3 codes of a cache against the oracle on the dequantised values (the oracle has no
    8-bit arithmetic of its own: it is handed scale * e4m3(code) as fp32).  rounding_bound: outputs are compared by
    parity.check_output's rounding model (a probability enters the PV product with a relative error of 2^-9, as in the
    bf16 kernels, here as the sum of two e4m3 numbers; the output is cast to bf16)."""
    k8, ks, kd = W.quantize_cache_e4m3(w["kcache"])
    v8, vs, vd = W.quantize_cache_e4m3(w["vcache"])
    q = w["q"].cuda()
    B, _, Hq, d = q.shape
    Nk, Hkv = k8.shape[1], k8.shape[2]
    G = Hq // Hkv
    o, lse, st = mala.decode_fp8(q, k8.cuda(), v8.cuda(), ks.cuda(), vs.cuda(), w["scale"], tau, num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ref = oracle.decode(w["q"], kd, vd, w["scale"], tau, num_splits, 128)
    ref_abs = oracle.decode(w["q"], kd, vd.abs(), w["scale"], tau, num_splits, 128) if rounding_bound else None
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy()[:, 0], lse.cpu().numpy()
    skipped = retained = 0
    for b in range(B):
        for g in range(Hkv):
            for s in range(num_splits):
                parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                                  tau, Nk, 128)
                assert int(st.retained[b, g, s]) == int(gm[b, g, s].sum())
            hs = slice(g * G, (g + 1) * G)
            parity.check_output(o_c[b, hs], ref["o"][b, hs], a_ref=ref_abs["o"][b, hs] if rounding_bound else None)
            assert np.abs(lse_c[b, hs] - ref["lse"][b, hs]).max() <= parity.LSE_ABS
            skipped += int((ref["mask"][b, g] == 1).sum())
            retained += int((ref["mask"][b, g] == 2).sum())
    return dict(skipped=skipped, retained=retained, totals=st.totals.cpu().numpy())


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv,d", [(128, 1, 4, 1, 128), (1024, 4, 8, 2, 128), (1000, 3, 4, 4, 128), (4096, 8, 2, 1, 128),
                                            (700, 8, 2, 1, 64), (2100, 5, 6, 2, 96), (8192, 64, 8, 2, 128),
                                            (1024, 4, 8, 1, 128), (3000, 5, 16, 2, 128), (2100, 3, 6, 1, 64), (900, 2, 14, 2, 80)])
def test_decode_fp8_cache_literal(mala, oracle, Nk, S, Hq, Hkv, d, tau):
    w = W.custom_decode(2, Hq, Hkv, Nk, d, S, seed=Nk + S)
    _run_fp8(mala, oracle, w, tau, S)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("Nk,S,Hq", [(8192, 8, 8), (5000, 4, 8), (8192, 8, 16)])
def test_decode_fp8_cache_skips_value_tiles(mala, oracle, Nk, S, Hq, tau):
    w = W.custom_decode(2, Hq, 2, Nk, 128, S, group_types=["diffuse", "peaked"], seed=3, preset="D")
    res = _run_fp8(mala, oracle, w, tau, S)
    assert res["skipped"] > 0, "workload must exercise skipping"
    assert res["totals"][1] == res["retained"] + res["skipped"]


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("B,Nk,S,Hq,Hkv", [(40, 3000, 5, 8, 8), (24, 1500, 7, 16, 4), (64, 700, 3, 4, 2)])
def test_decode_fp8_cache_many_work_items_per_cta(mala, oracle, B, Nk, S, Hq, Hkv, tau):
    """More (sequence, KV head, split) items than SMs, with one to five tiles each: every CTA walks several items, the
    softmax groups change places from item to item and the state slots and accumulators are handed back and reused."""
    w = W.custom_decode(B, Hq, Hkv, Nk, 128, S, seed=B + Nk, preset="D" if tau > 0 else "literal")
    res = _run_fp8(mala, oracle, w, tau, S, rounding_bound=True)
    assert res["totals"][1] == res["retained"] + res["skipped"]


@pytest.mark.parametrize("tau", [0.0, 1e-4])
def test_decode_fp8_repeated_launches_give_identical_bits(mala, tau):
    """Several work items per CTA, eight tiles each, launched many times: the result does not depend on how the groups
    of a CTA happen to interleave (no atomics on the data path, every hand-over through a barrier)."""
    w = W.custom_decode(8, 32, 8, 16384, 128, 16, seed=9, preset="D", device="cuda")
    k8, ks, _ = W.quantize_cache_e4m3(w["kcache"])
    v8, vs, _ = W.quantize_cache_e4m3(w["vcache"])
    first = None
    for _ in range(40):
        o, lse, _ = mala.decode_fp8(w["q"], k8, v8, ks, vs, w["scale"], tau, 16)
        if first is None:
            first = (o.clone(), lse.clone())
            assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
        else:
            assert torch.equal(o, first[0]) and torch.equal(lse, first[1])
    assert mala.device_status() == 0


@pytest.mark.parametrize("tau", [0.0, 1e-4])
def test_decode_fp8_head_major_cache_view(mala, tau):
    """The cache views are strided: a head-major [B,Hkv,Nk,d] cache passed as its [B,Nk,Hkv,d] view gives the bits of
    the key-major one."""
    w = W.custom_decode(2, 8, 2, 3000, 128, 5, seed=4, preset="D", device="cuda")
    k8, ks, _ = W.quantize_cache_e4m3(w["kcache"])
    v8, vs, _ = W.quantize_cache_e4m3(w["vcache"])
    hm = lambda x: x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    o0, l0, _ = mala.decode_fp8(w["q"], k8, v8, ks, vs, w["scale"], tau, 5)
    o1, l1, _ = mala.decode_fp8(w["q"], hm(k8), hm(v8), ks, vs, w["scale"], tau, 5)
    assert torch.equal(o0, o1) and torch.equal(l0, l1)


def test_decode_fp8_refuses_what_it_does_not_support(mala):
    w = W.custom_decode(1, 16, 1, 256, 128, 1, seed=1)
    k8, ks, _ = W.quantize_cache_e4m3(w["kcache"])
    with pytest.raises(mala.MalaError) as e:     # sixteen query heads per KV head
        mala.decode_fp8(w["q"].cuda(), k8.cuda(), k8.cuda(), ks.cuda(), ks.cuda(), w["scale"], 0.0, 1)
    assert e.value.code == -2


def _run_fp8_paged(mala, oracle, w, tau, num_splits, page_size, seqlens, seed=0):
    """mala_decode_fp8_paged against the paged oracle on the dequantised pages: the contiguous bf16 workload is cut
    into pages of a shuffled pool (junk in unused slots, table entries outside the pool), the pool is quantised page by
    page (one scale per 128-key tile of a page), and the oracle is handed scale * e4m3(code)."""
    kp, vp, bt, lens = W.paginate(w["kcache"], w["vcache"], page_size, seqlens=seqlens, seed=seed)
    # (a pool [num_pages, page_size, Hkv, d] has the shape of a cache; pages smaller than a tile: one scale per page)
    k8, ks, kd = W.quantize_cache_e4m3(kp, tile=min(128, page_size))
    v8, vs, vd = W.quantize_cache_e4m3(vp, tile=min(128, page_size))
    q = w["q"].cuda()
    B, _, Hq, d = q.shape
    Hkv = kp.shape[2]
    G = Hq // Hkv
    o, lse, st = mala.decode_fp8_paged(q, k8.cuda(), v8.cuda(), ks.cuda(), vs.cuda(), bt.cuda(),
                                       lens.cuda() if seqlens is not None else None, w["scale"], tau, num_splits, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ln = lens.numpy() if seqlens is not None else None
    ref = oracle.decode_paged(w["q"][:, 0], kd, vd, bt.numpy(), ln, w["scale"], tau, num_splits, 128)
    ref_abs = oracle.decode_paged(w["q"][:, 0], kd, vd.abs(), bt.numpy(), ln, w["scale"], tau, num_splits, 128)
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy()[:, 0], lse.cpu().numpy()
    skipped = retained = 0
    for b in range(B):
        n = int(lens[b])
        for g in range(Hkv):
            for s in range(num_splits):
                parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                                  tau, max(n, 1), 128)
                assert int(st.retained[b, g, s]) == int(gm[b, g, s].sum())
            hs = slice(g * G, (g + 1) * G)
            parity.check_output(o_c[b, hs], ref["o"][b, hs], a_ref=ref_abs["o"][b, hs])
            if n > 0:
                assert np.abs(lse_c[b, hs] - ref["lse"][b, hs]).max() <= parity.LSE_ABS
            else:
                assert np.isneginf(lse_c[b, hs]).all() and (o_c[b, hs] == 0).all()
            skipped += int((ref["mask"][b, g] == 1).sum())
            retained += int((ref["mask"][b, g] == 2).sum())
    tot = st.totals.cpu().numpy()
    assert tot[1] == retained + skipped
    return dict(skipped=skipped, retained=retained)


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv,page,lens", [
    (1024, 4, 8, 2, 128, None),                        # one tile per page, every sequence full
    (2048, 4, 4, 1, 256, [2048, 1000, 129]),           # two tiles per page, ragged lengths, empty trailing splits
    (1536, 3, 4, 2, 512, [1, 1536, 0, 700]),           # a split per page; one key; no key at all
    (8192, 64, 8, 2, 128, [8192, 5000, 128, 3333]),    # more work items than SMs, one tile each
    (6144, 6, 4, 4, 384, [6144, 6000, 385, 3000, 17]), # three tiles per page, one head per KV head
    (4096, 8, 16, 2, 256, [4096, 2049, 300]),          # eight heads per KV head
    (2048, 4, 8, 2, 16, [2048, 1000, 129, 5]),         # pages of 16 keys: eight per tile, a scale per page
    (1536, 3, 4, 1, 32, [1, 1536, 0, 700]),            # pages of 32 keys
    (4096, 16, 16, 2, 64, [4096, 2049, 300]),          # pages of 64 keys, eight heads per KV head
    (1040, 2, 6, 2, 16, [1040, 1025, 17]),             # a table whose last tile is partly past the row's end
])
def test_decode_fp8_paged_literal(mala, oracle, Nk, S, Hq, Hkv, page, lens, tau):
    B = 2 if lens is None else len(lens)
    w = W.custom_decode(B, Hq, Hkv, Nk, 128, S, seed=Nk + S + page)
    _run_fp8_paged(mala, oracle, w, tau, S, page, lens, seed=page)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
def test_decode_fp8_paged_gated_keys_skip_value_tiles(mala, oracle, tau):
    w = W.custom_decode(3, 8, 2, 8192, 128, 8, group_types=["diffuse", "peaked"], seed=5, preset="D")
    res = _run_fp8_paged(mala, oracle, w, tau, 8, 256, [8192, 4096 + 77, 2500], seed=9)
    assert res["skipped"] > 0, "workload must exercise skipping"


def test_decode_fp8_paged_identity_table_equals_contiguous_call(mala):
    # pages laid out in order are the contiguous cache: both entry points must give the same bits
    w = W.custom_decode(2, 8, 2, 4096, 128, 8, group_types=["diffuse", "peaked"], seed=21, preset="D", device="cuda")
    k8, ks, _ = W.quantize_cache_e4m3(w["kcache"])
    v8, vs, _ = W.quantize_cache_e4m3(w["vcache"])
    page = 512
    npg = 4096 // page
    kp = k8.view(2 * npg, page, 2, 128)
    vp = v8.view(2 * npg, page, 2, 128)
    # scales [B, Hkv, nt] -> [num_pages, Hkv, tiles per page]
    to_pages = lambda sc: sc.view(2, 2, npg, page // 128).permute(0, 2, 1, 3).reshape(2 * npg, 2, page // 128).contiguous()
    bt = torch.arange(2 * npg, dtype=torch.int32, device="cuda").view(2, npg)
    for tau in (0.0, 1e-4):
        o0, l0, _ = mala.decode_fp8(w["q"], k8, v8, ks, vs, w["scale"], tau, 8)
        o1, l1, _ = mala.decode_fp8_paged(w["q"], kp, vp, to_pages(ks), to_pages(vs), bt, None, w["scale"], tau, 8)
        assert torch.equal(o0, o1) and torch.equal(l0, l1)


def test_decode_fp8_paged_rejects_page_sizes_it_does_not_support(mala):
    w = W.custom_decode(1, 4, 1, 512, 128, 1, seed=1, device="cuda")
    for page in (8, 48, 192):          # (pages of whole tiles, or of 16, 32 or 64 keys)
        k8 = torch.zeros((8, page, 1, 128), dtype=torch.uint8, device="cuda")
        sc = torch.ones((8, 1, max(1, page // 128)), dtype=torch.float32, device="cuda")
        bt = torch.arange(8, dtype=torch.int32, device="cuda").view(1, 8)
        with pytest.raises(mala.MalaError) as e:
            mala.decode_fp8_paged(w["q"], k8, k8, sc, sc, bt, None, w["scale"], 0.0, 1)
        assert e.value.code == -2


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("page", [16, 64])
def test_decode_fp8_small_pages_gated_keys_skip_value_tiles(mala, oracle, page, tau):
    w = W.custom_decode(3, 8, 2, 8192, 128, 8, group_types=["diffuse", "peaked"], seed=5, preset="D")
    res = _run_fp8_paged(mala, oracle, w, tau, 8, page, [8192, 4096 + 77, 2500], seed=9)
    assert res["skipped"] > 0, "workload must exercise skipping"


def test_decode_fp8_small_pages_with_scales_far_apart(mala, oracle):
    # the pages of a tile get V (and K) magnitudes a factor 2^10 apart: a key's probability is scaled by its own page's
    # V scale while the 8-bit reference follows the tile's largest one
    w = W.custom_decode(2, 4, 2, 2048, 128, 4, seed=77)
    for name in ("kcache", "vcache"):
        c = w[name].float()
        f = torch.tensor([1.0, 2.0 ** -10, 2.0 ** -2, 2.0 ** -6])[(torch.arange(2048) // 16) % 4]
        w[name] = (c * f[None, :, None, None] * (0.25 if name == "kcache" else 1.0)).to(torch.bfloat16)
    for tau in (0.0, 1e-4):
        _run_fp8_paged(mala, oracle, w, tau, 4, 16, [2048, 1500], seed=3)


def _run_fp8_multi(mala, oracle, w, Sq, tau, num_splits, seed=0):
    """mala_decode_fp8_multi against the oracle's several-token decode on the dequantised cache (queries drawn as in
    _run_multi)."""
    k8, ks, kd = W.quantize_cache_e4m3(w["kcache"])
    v8, vs, vd = W.quantize_cache_e4m3(w["vcache"])
    B, Nk, Hkv, d = k8.shape
    Hq = w["q"].shape[2]
    gen = torch.Generator(device="cpu")
    gen.manual_seed(1000 + seed)
    q = w["q"].float().repeat(1, Sq, 1, 1)
    q[..., : d - 1] += 0.5 * torch.randn((B, Sq, Hq, d - 1), generator=gen)   # (the last feature keeps the key gate)
    q = q.to(torch.bfloat16)
    o, lse, st = mala.decode_fp8_multi(q.cuda(), k8.cuda(), v8.cuda(), ks.cuda(), vs.cuda(), w["scale"], tau, num_splits,
                                       stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ref = oracle.decode_multi(q, kd, vd, w["scale"], tau, num_splits, 128)
    ref_abs = oracle.decode_multi(q, kd, vd.abs(), w["scale"], tau, num_splits, 128)
    tps = ref["mask"].shape[-1]
    gm = st.mask(tps).cpu().numpy()
    for b in range(B):
        for g in range(Hkv):
            for s in range(num_splits):
                parity.check_mask(gm[b, g, s], ref["mask"][b, g, s], ref["crit"][b, g, s], list(range(tps - 1, -1, -1)),
                                  tau, Nk - Sq + 1, 128)
                assert int(st.retained[b, g, s]) == int(gm[b, g, s].sum())
    parity.check_output(o.float().cpu().numpy(), ref["o"], a_ref=ref_abs["o"])
    assert np.abs(lse.cpu().numpy() - ref["lse"]).max() <= parity.LSE_ABS
    return int((ref["mask"] == 1).sum())


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,S,Hq,Hkv,Sq", [(1024, 4, 8, 2, 2), (1000, 3, 4, 4, 8), (2050, 4, 4, 2, 4), (1027, 2, 6, 2, 2),
                                             (640, 5, 2, 1, 3), (4096, 8, 2, 2, 5), (1026, 2, 1, 1, 7)])
def test_decode_fp8_multi_literal(mala, oracle, Nk, S, Hq, Hkv, Sq, tau):
    """Several new tokens per step over an e4m3 cache, up to eight rows per KV head; (2050, 4), (1027, 2), (1026, 7): the
    newest key block holds fewer keys than there are new tokens, so its first rows see none of it."""
    w = W.custom_decode(2, Hq, Hkv, Nk, 128, S, seed=Nk + S + Sq)
    _run_fp8_multi(mala, oracle, w, Sq, tau, S, seed=Sq)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
def test_decode_fp8_multi_gated_keys_skip_value_tiles(mala, oracle, tau):
    w = W.custom_decode(2, 8, 2, 8192, 128, 8, group_types=["diffuse", "peaked"], seed=3, preset="D")
    assert _run_fp8_multi(mala, oracle, w, 2, tau, 8) > 0, "workload must exercise skipping"


def test_decode_fp8_multi_of_one_token_equals_decode_fp8(mala):
    w = W.custom_decode(2, 8, 2, 4096, 128, 8, group_types=["diffuse", "peaked"], seed=21, preset="D", device="cuda")
    k8, ks, _ = W.quantize_cache_e4m3(w["kcache"])
    v8, vs, _ = W.quantize_cache_e4m3(w["vcache"])
    for tau in (0.0, 1e-4):
        o0, l0, _ = mala.decode_fp8(w["q"], k8, v8, ks, vs, w["scale"], tau, 8)
        o1, l1, _ = mala.decode_fp8_multi(w["q"], k8, v8, ks, vs, w["scale"], tau, 8)
        assert torch.equal(o0, o1) and torch.equal(l0, l1.view_as(l0))
    q3 = w["q"].repeat(1, 3, 1, 1)                      # (twelve rows per KV head: more than the kernel packs)
    with pytest.raises(mala.MalaError) as e:
        mala.decode_fp8_multi(q3, k8, v8, ks, vs, w["scale"], 0.0, 8)
    assert e.value.code == -2


@pytest.mark.parametrize("page", [16, 32])
def test_decode_fp8_small_pages_absent_pages_do_not_set_the_reference(mala, oracle, page):
    """Sequences that end inside a tile, with table entries outside the pool behind them, and values 2^-6 small: the
    pages that are not there (scale 1) or lie past the sequence's end must not set the reference of the 8-bit
    probabilities, or every real key's probability would fall into e4m3's subnormals."""
    w = W.custom_decode(3, 8, 2, 4096, 64, 2, seed=462)
    w["vcache"] = (w["vcache"].float() * 2.0 ** -6).to(torch.bfloat16)
    for tau in (0.0, 1.0):
        _run_fp8_paged(mala, oracle, w, tau, 2, page, [4096, 1497, 48 + page // 2], seed=3)
