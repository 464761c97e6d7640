"""GPU parity of mala_fwd (through the C ABI) against the fp64 oracle."""
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


def _run_and_check(mala, oracle, w, tau, causal=True, units=None, rounding_bound=False):
    dev = "cuda"
    q, k, v = (w[x].to(dev) for x in ("q", "k", "v"))
    B, N, Hq, d = q.shape
    o, lse, st = mala.fwd(q, k, v, w["scale"], tau, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    Bq, Bk = mala.tile_shape(mala.OP_FWD, d)
    ref = oracle.fwd(w["q"], w["k"], w["v"], w["scale"], tau, Bq, Bk, causal=causal, units=units)
    # (the same call on |V|: a = sum_k p_k |v_k| over the retained keys, for the rounding bound of parity.check_output)
    ref_abs = oracle.fwd(w["q"], w["k"], w["v"].abs(), w["scale"], tau, Bq, Bk, causal=causal, units=units) if rounding_bound else None
    T = -(-N // Bq)
    gm = st.mask(T).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy(), lse.cpu().numpy()
    if units is None:
        units = [(b, h, i) for b in range(B) for h in range(Hq) for i in range(T)]
    flips = 0
    retained = skipped = 0
    worst = 0.0
    for (b, h, i) in units:
        order = list(range(i, -1, -1)) if causal else list(range(T - 1, -1, -1))
        rows = slice(i * Bq, min(N, (i + 1) * Bq))
        flips += parity.check_mask(gm[b, h, i], ref["mask"][b, h, i], ref["crit"][b, h, i], order, tau,
                                   i * Bq + 1 if causal else N, Bk)
        err = parity.check_output(o_c[b, rows, h], ref["o"][b, rows, h],
                                  a_ref=ref_abs["o"][b, rows, h] if rounding_bound else None)
        worst = max(worst, err[0])
        assert np.abs(lse_c[b, h, rows] - ref["lse"][b, h, rows]).max() <= parity.LSE_ABS
        retained += int((ref["mask"][b, h, i] == 2).sum())
        skipped += int((ref["mask"][b, h, i] == 1).sum())
        assert int(st.retained[b, h, i]) == int(gm[b, h, i].sum())
    crit = np.abs(ref["crit"][ref["mask"] > 0])
    return dict(flips=flips, retained=retained, skipped=skipped, totals=st.totals.cpu().numpy(), max_err=worst,
                near=int((crit < 1e-2).sum()), band=int((crit <= parity.MASK_BAND).sum()),
                o_absmax=float(np.abs(ref["o"][np.isfinite(ref["o"])]).max()))


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("N,d,Hq,Hkv", [(128, 128, 1, 1), (384, 128, 2, 1), (333, 128, 2, 2), (512, 64, 2, 2),
                                        (200, 64, 1, 1)])
def test_fwd_small_shapes_literal(mala, oracle, N, d, Hq, Hkv, tau):
    w = W.custom_prefill(2, Hq, Hkv, N, d, seed=N + d)
    _run_and_check(mala, oracle, w, tau)


@pytest.mark.parametrize("tau", [1e-5, 1e-4, 1e-3, 1.0])
@pytest.mark.parametrize("N,d", [(1024, 128), (1000, 128), (1024, 64)])
def test_fwd_skipping_regime(mala, oracle, N, d, tau):
    w = W.custom_prefill(1, 4, 2, N, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=7, preset="R")
    res = _run_and_check(mala, oracle, w, tau)
    assert res["skipped"] > 0, "workload must exercise skipping"
    assert res["totals"][0] == res["retained"] + 0 or res["flips"] > 0
    assert res["totals"][1] == res["retained"] + res["skipped"]


@pytest.mark.parametrize("tau", [0.0, 1e-4, 1e-3])
def test_fwd_cfg1(mala, oracle, tau):
    w = W.make_prefill(W.prefill_config("cfg1"))
    _run_and_check(mala, oracle, w, tau)


@pytest.mark.parametrize("tau", [0.0, 1e-2])
def test_fwd_non_causal(mala, oracle, tau):
    w = W.custom_prefill(1, 2, 1, 300, 128, head_types=["peaked", "diffuse"], seed=5, preset="R")
    _run_and_check(mala, oracle, w, tau, causal=False)


def test_fwd_tau_zero_equals_dense_kernel_bitwise_mask(mala, oracle):
    w = W.custom_prefill(1, 2, 1, 640, 128, seed=9, preset="R")
    q, k, v = (w[x].cuda() for x in ("q", "k", "v"))
    _, _, st = mala.fwd(q, k, v, w["scale"], 0.0, stats=True)
    T = 5
    m = st.mask(T).cpu().numpy()
    for i in range(T):
        assert m[0, :, i, :i + 1].all() and not m[0, :, i, i + 1:].any()


def test_fwd_near_threshold_decisions(mala, oracle, capsys):
    """Inputs whose tile criteria pass through zero with a small slope per tile (softmax mass decaying smoothly toward
    earlier keys): a visible number of tiles has |C| < 1e-2 and some lie inside the 1e-3 band in which the fp32 / log2
    evaluation of Eq. 3 may decide differently from the fp64 oracle.  Every decision outside the band must be the
    oracle's (parity.check_mask); the number of exempted flips is reported."""
    near = band = flips = 0
    for seed in (5, 6, 7, 8):
        w = W.custom_prefill(2, 6, 6, 4096, 64, head_types=["decay"] * 6, seed=seed)
        for tau in (1.0, 0.3):
            res = _run_and_check(mala, oracle, w, tau)
            assert res["skipped"] > 0
            flips += res["flips"]
            near += res["near"]
            band += res["band"]
    with capsys.disabled():
        print(f"\n[near-threshold forward] tiles with |C| < 1e-2: {near}, inside the 1e-3 band: {band}, "
              f"decisions that differ from the oracle (all inside the band): {flips}")
    assert near >= 10 and band >= 1, "the workload must put tiles next to the threshold"
