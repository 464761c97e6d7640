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


def _run_and_check(mala, oracle, w, tau, causal=True, units=None):
    dev = "cuda"
    q, k, v = (w[x].to(dev) for x in ("q", "k", "v"))
    B, N, Hq, d = q.shape
    o, lse, st = mala.fwd(q, k, v, w["scale"], tau, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    Bq, Bk = mala.tile_shape(mala.OP_FWD, d)
    ref = oracle.fwd(w["q"], w["k"], w["v"], w["scale"], tau, Bq, Bk, causal=causal, units=units)
    T = -(-N // Bq)
    gm = st.mask(T).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy(), lse.cpu().numpy()
    if units is None:
        units = [(b, h, i) for b in range(B) for h in range(Hq) for i in range(T)]
    flips = 0
    retained = skipped = 0
    for (b, h, i) in units:
        order = list(range(i, -1, -1)) if causal else list(range(T - 1, -1, -1))
        rows = slice(i * Bq, min(N, (i + 1) * Bq))
        flips += parity.check_mask(gm[b, h, i], ref["mask"][b, h, i], ref["crit"][b, h, i], order, tau,
                                   i * Bq + 1 if causal else N, Bk)
        parity.check_output(o_c[b, rows, h], ref["o"][b, rows, h])
        assert np.abs(lse_c[b, h, rows] - ref["lse"][b, h, rows]).max() <= parity.LSE_ABS
        retained += int((ref["mask"][b, h, i] == 2).sum())
        skipped += int((ref["mask"][b, h, i] == 1).sum())
        assert int(st.retained[b, h, i]) == int(gm[b, h, i].sum())
    return dict(flips=flips, retained=retained, skipped=skipped, totals=st.totals.cpu().numpy())


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
