"""GPU parity of mala_fwd_chunk / mala_bwd_chunk (fewer queries than keys) against the fp64 oracle."""
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


def _chunk(w, Nq):
    """The last Nq queries (and their upstream gradients) of a prefill workload; keys and values in full."""
    N = w["q"].shape[1]
    return dict(q=w["q"][:, N - Nq:].contiguous(), k=w["k"], v=w["v"], do=w["do"][:, N - Nq:].contiguous(),
                scale=w["scale"])


def _run(mala, oracle, c, tau, causal=True):
    q, k, v, do = (c[x].cuda() for x in ("q", "k", "v", "do"))
    B, Nq, Hq, d = q.shape
    Nk = k.shape[1]
    Bq, Bk = mala.tile_shape(mala.OP_FWD, d)
    Tq, Tk = -(-Nq // Bq), -(-Nk // Bk)
    off = Nk - Nq if causal else 0
    o, lse, fst = mala.fwd_chunk(q, k, v, c["scale"], tau, causal=causal, stats=True)
    dq, dk, dv, bst = mala.bwd_chunk(q, k, v, o, do, lse, c["scale"], tau, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ref = oracle.fwd(c["q"], c["k"], c["v"], c["scale"], tau, Bq, Bk, causal=causal)
    fm = fst.mask(Tk).cpu().numpy()                      # [B,Hq,Tq,Tk]
    o_c, lse_c = o.float().cpu().numpy(), lse.cpu().numpy()
    skipped = 0
    for b in range(B):
        for h in range(Hq):
            for i in range(Tq):
                order = list(range(i + off // Bk, -1, -1)) if causal else list(range(Tk - 1, -1, -1))
                rows = slice(i * Bq, min(Nq, (i + 1) * Bq))
                parity.check_mask(fm[b, h, i], ref["mask"][b, h, i], ref["crit"][b, h, i], order, tau,
                                  i * Bq + 1 + off if causal else Nk, Bk)
                parity.check_output(o_c[b, rows, h], ref["o"][b, rows, h])
                assert np.abs(lse_c[b, h, rows] - ref["lse"][b, h, rows]).max() <= parity.LSE_ABS
                assert int(fst.retained[b, h, i]) == int(fm[b, h, i].sum())
    skipped += int((ref["mask"] == 1).sum())
    # backward on the GPU's own forward output, as the kernel receives it
    rb = oracle.bwd(c["q"], c["k"], c["v"], o.float().cpu(), c["do"], lse.cpu().numpy(), c["scale"], tau, Bq, Bk,
                    causal=causal)
    bm = bst.mask(Tq).cpu().numpy()                      # [B,Hq,Tk,Tq]
    for b in range(B):
        for h in range(Hq):
            for j in range(Tk):
                om, oc = rb["mask"][b, h, j], rb["crit"][b, h, j]
                for i in range(Tq):
                    if om[i] == 0:
                        assert not bm[b, h, j, i]
                    elif bool(bm[b, h, j, i]) != (om[i] == 2):
                        assert abs(oc[i]) <= parity.MASK_BAND, (b, h, j, i, oc[i])
                assert int(bst.retained[b, h, j]) == int(bm[b, h, j].sum())
    parity.check_grad(dq.float().cpu().numpy(), rb["dq"], "dq")
    parity.check_grad(dk.float().cpu().numpy(), rb["dk"], "dk")
    parity.check_grad(dv.float().cpu().numpy(), rb["dv"], "dv")
    assert (bm.transpose(0, 1, 3, 2) <= fm).all()        # nesting
    skipped += int((rb["mask"] == 1).sum())
    legal_f, legal_b = int((ref["mask"] > 0).sum()), int((rb["mask"] > 0).sum())
    assert fst.totals.cpu().numpy()[1] == legal_f and bst.totals.cpu().numpy()[1] == legal_b
    return skipped


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,Nq,d,Hq,Hkv", [(512, 128, 128, 2, 1), (640, 256, 128, 4, 2), (1000, 232, 128, 2, 2),
                                            (768, 384, 64, 2, 1), (456, 200, 64, 2, 2), (384, 384, 128, 2, 1)])
def test_chunk_literal(mala, oracle, Nk, Nq, d, Hq, Hkv, tau):
    w = W.custom_prefill(2, Hq, Hkv, Nk, d, seed=Nk + Nq)
    _run(mala, oracle, _chunk(w, Nq), tau)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("Nk,Nq,d", [(2048, 512, 128), (1768, 744, 128), (2048, 1024, 64)])
def test_chunk_skipping_regime(mala, oracle, Nk, Nq, d, tau):
    w = W.custom_prefill(1, 4, 2, Nk, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=7, preset="R")
    assert _run(mala, oracle, _chunk(w, Nq), tau) > 0, "workload must exercise skipping"


@pytest.mark.parametrize("tau", [0.0, 1e-2])
def test_chunk_non_causal_any_lengths(mala, oracle, tau):
    # cross attention: 200 queries against 555 keys, every key legal, L = 555
    w = W.custom_prefill(1, 2, 1, 555, 128, head_types=["peaked", "diffuse"], seed=5, preset="R")
    _run(mala, oracle, _chunk(w, 200), tau, causal=False)


@pytest.mark.parametrize("tau", [0.0, 1e-2])
def test_chunk_non_causal_more_queries_than_keys(mala, oracle, tau):
    # cross attention the other way round: 370 queries against 184 keys
    w = W.custom_prefill(1, 2, 1, 370, 64, head_types=["peaked", "diffuse"], seed=15, preset="R")
    c = dict(q=w["q"], k=w["k"][:, :184].contiguous(), v=w["v"][:, :184].contiguous(), do=w["do"], scale=w["scale"])
    _run(mala, oracle, c, tau, causal=False)


def test_chunk_equals_rows_of_the_equal_length_call(mala):
    # both entry points on the GPU: the chunk call must give the last rows of the full call (the forward bit for bit)
    w = W.custom_prefill(1, 4, 2, 1536, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=3, preset="R")
    q, k, v, do = (w[x].cuda() for x in ("q", "k", "v", "do"))
    off = 1024
    for tau in (0.0, 1e-4):
        o, lse, _ = mala.fwd(q, k, v, w["scale"], tau)
        oc, lc, _ = mala.fwd_chunk(q[:, off:], k, v, w["scale"], tau)
        assert torch.equal(o[:, off:], oc) and torch.equal(lse[:, :, off:], lc)
        do0 = do.clone()
        do0[:, :off] = 0
        dq, dk, dv, _ = mala.bwd(q, k, v, o, do0, lse, w["scale"], tau)
        dqc, dkc, dvc, _ = mala.bwd_chunk(q[:, off:], k, v, oc, do[:, off:], lc, w["scale"], tau)
        # dQ is summed over the key blocks by fp32 reductions whose order varies from run to run
        assert (dq[:, off:].float() - dqc.float()).abs().max() <= 1e-2 * dqc.float().abs().max()
        assert (dq[:, :off] == 0).all()
        # dK, dV: the full call also runs the retained tiles of the earlier rows, whose dS and P^T dO are exact zeros
        assert (dk.float() - dkc.float()).abs().max() <= 1e-2 * dk.float().abs().max()
        assert (dv.float() - dvc.float()).abs().max() <= 1e-2 * dv.float().abs().max()


def _run_bwd_any_offset(mala, oracle, c, tau):
    """Backward of a chunk that may start inside a tile, on the GPU's own forward output."""
    q, k, v, do = (c[x].cuda() for x in ("q", "k", "v", "do"))
    B, Nq, Hq, d = q.shape
    Nk = k.shape[1]
    shift = (Nk - Nq) % 128
    Tq, Tk = -(-(Nq + shift) // 128), -(-Nk // 128)
    o, lse, fst = mala.fwd_chunk(q, k, v, c["scale"], tau, stats=True)
    dq, dk, dv, bst = mala.bwd_chunk(q, k, v, o, do, lse, c["scale"], tau, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    rb = oracle.bwd(c["q"], c["k"], c["v"], o.float().cpu(), c["do"], lse.cpu().numpy(), c["scale"], tau, 128, 128,
                    q_shift=shift)
    bm = bst.mask(Tq).cpu().numpy()                      # [B,Hq,Tk,Tq]
    assert rb["mask"].shape == bm.shape
    for b in range(B):
        for h in range(Hq):
            for j in range(Tk):
                om, oc = rb["mask"][b, h, j], rb["crit"][b, h, j]
                for i in range(Tq):
                    if om[i] == 0:
                        assert not bm[b, h, j, i]
                    elif bool(bm[b, h, j, i]) != (om[i] == 2):
                        assert abs(oc[i]) <= parity.MASK_BAND, (b, h, j, i, oc[i])
                assert int(bst.retained[b, h, j]) == int(bm[b, h, j].sum())
    parity.check_grad(dq.float().cpu().numpy(), rb["dq"], "dq")
    parity.check_grad(dk.float().cpu().numpy(), rb["dk"], "dk")
    parity.check_grad(dv.float().cpu().numpy(), rb["dv"], "dv")
    assert (bm.transpose(0, 1, 3, 2) <= fst.mask(Tk).cpu().numpy()).all()        # nesting
    assert bst.totals.cpu().numpy()[1] == int((rb["mask"] > 0).sum())
    return int((rb["mask"] == 1).sum())


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,Nq,d,Hq,Hkv", [(500, 100, 128, 2, 1), (1000, 333, 128, 4, 2), (777, 129, 64, 2, 2),
                                            (1300, 5, 128, 2, 1), (640, 639, 128, 2, 1)])
def test_chunk_backward_from_any_position_literal(mala, oracle, Nk, Nq, d, Hq, Hkv, tau):
    w = W.custom_prefill(2, Hq, Hkv, Nk, d, seed=Nk + Nq)
    _run_bwd_any_offset(mala, oracle, _chunk(w, Nq), tau)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("Nk,Nq,d", [(2000, 555, 128), (2500, 1300, 64)])
def test_chunk_backward_from_any_position_skipping_regime(mala, oracle, Nk, Nq, d, tau):
    w = W.custom_prefill(1, 4, 2, Nk, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=9, preset="R")
    assert _run_bwd_any_offset(mala, oracle, _chunk(w, Nq), tau) > 0, "workload must exercise skipping"


def test_chunk_backward_from_any_position_gives_the_rows_of_the_equal_length_call(mala):
    w = W.custom_prefill(1, 4, 2, 1536, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=3, preset="R")
    q, k, v, do = (w[x].cuda() for x in ("q", "k", "v", "do"))
    off = 1000
    for tau in (0.0, 1e-4):
        o, lse, _ = mala.fwd(q, k, v, w["scale"], tau)
        do0 = do.clone()
        do0[:, :off] = 0
        dq, dk, dv, _ = mala.bwd(q, k, v, o, do0, lse, w["scale"], tau)
        dqc, dkc, dvc, _ = mala.bwd_chunk(q[:, off:], k, v, o[:, off:], do[:, off:], lse[:, :, off:].contiguous(),
                                          w["scale"], tau)
        # the chunk's first block lacks the rows before `off`; with dout zero there they contribute nothing, but they
        # vote in the whole call: compare from the first whole block on for dQ, and dK / dV within the tolerance that
        # a tile retained by one call and skipped by the other leaves (entries below tau / L_q)
        first = 1024 - off
        assert (dq[:, 1024:].float() - dqc[:, first:].float()).abs().max() <= 1e-2 * dqc.float().abs().max()
        assert (dk.float() - dkc.float()).abs().max() <= 1e-2 * dk.float().abs().max()
        assert (dv.float() - dvc.float()).abs().max() <= 1e-2 * dv.float().abs().max()


def _run_fwd_any_offset(mala, oracle, c, tau, S=1):
    """Forward of a chunk that may start inside a tile: the query blocks follow the key positions."""
    q, k, v = (c[x].cuda() for x in ("q", "k", "v"))
    B, Nq, Hq, d = q.shape
    Nk = k.shape[1]
    off = Nk - Nq
    shift = off % 128
    Tq, Tk = -(-(Nq + shift) // 128), -(-Nk // 128)
    if S == 1:
        o, lse, st = mala.fwd_chunk(q, k, v, c["scale"], tau, stats=True)
    else:
        o, lse, st = mala.fwd_chunk_split(q, k, v, c["scale"], tau, S, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ref = oracle.fwd(c["q"], c["k"], c["v"], c["scale"], tau, 128, 128, num_splits=S, q_shift=shift)
    fm = st.mask(Tk).cpu().numpy()
    tps = -(-Tk // S)
    for b in range(B):
        for h in range(Hq):
            for i in range(Tq):
                newest = i + off // 128
                first_row = max(i * 128 - shift, 0)
                for s in range(S):
                    js = [j for j in range(min(newest, (s + 1) * tps - 1), s * tps - 1, -1)]
                    sel = np.zeros(Tk, dtype=bool)
                    sel[js] = True
                    parity.check_mask(np.where(sel, fm[b, h, i], False), np.where(sel, ref["mask"][b, h, i], 0),
                                      ref["crit"][b, h, i], js, tau, first_row + 1 + off)
                assert int(st.retained[b, h, i]) == int(fm[b, h, i].sum())
    parity.check_output(o.float().cpu().numpy(), ref["o"])
    assert np.abs(lse.cpu().numpy() - ref["lse"]).max() <= parity.LSE_ABS
    assert st.totals.cpu().numpy()[1] == int((ref["mask"] > 0).sum())
    return int((ref["mask"] == 1).sum())


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,Nq,d,Hq,Hkv,S", [(500, 100, 128, 2, 1, 1), (1000, 333, 128, 4, 2, 1), (777, 129, 64, 2, 2, 1),
                                              (1300, 5, 128, 2, 1, 1), (1000, 333, 128, 2, 1, 4), (901, 450, 64, 2, 1, 3)])
def test_chunk_from_any_position_literal(mala, oracle, Nk, Nq, d, Hq, Hkv, S, tau):
    w = W.custom_prefill(2, Hq, Hkv, Nk, d, seed=Nk + Nq)
    _run_fwd_any_offset(mala, oracle, _chunk(w, Nq), tau, S)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("Nk,Nq,S", [(2000, 555, 1), (2500, 300, 5)])
def test_chunk_from_any_position_skipping_regime(mala, oracle, Nk, Nq, S, tau):
    w = W.custom_prefill(1, 4, 2, Nk, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=7, preset="R")
    assert _run_fwd_any_offset(mala, oracle, _chunk(w, Nq), tau, S) > 0, "workload must exercise skipping"


def test_chunk_from_any_position_gives_the_rows_of_the_equal_length_call(mala):
    # where the chunk holds whole blocks of the full call the results are the same bits
    w = W.custom_prefill(1, 4, 2, 1536, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=3, preset="R")
    q, k, v = (w[x].cuda() for x in ("q", "k", "v"))
    off = 1000                                              # 1000 = 7 * 128 + 104: the first whole block starts at 1024
    for tau in (0.0, 1e-4):
        o, lse, _ = mala.fwd(q, k, v, w["scale"], tau)
        oc, lc, _ = mala.fwd_chunk(q[:, off:], k, v, w["scale"], tau)
        assert torch.equal(o[:, 1024:], oc[:, 24:]) and torch.equal(lse[:, :, 1024:], lc[:, :, 24:])


def _run_split(mala, oracle, c, tau, S, causal=True):
    q, k, v = (c[x].cuda() for x in ("q", "k", "v"))
    B, Nq, Hq, d = q.shape
    Nk = k.shape[1]
    Tq, Tk = -(-Nq // 128), -(-Nk // 128)
    off = Nk - Nq if causal else 0
    o, lse, st = mala.fwd_chunk_split(q, k, v, c["scale"], tau, S, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    ref = oracle.fwd(c["q"], c["k"], c["v"], c["scale"], tau, 128, 128, causal=causal, num_splits=S)
    fm = st.mask(Tk).cpu().numpy()
    tps = -(-Tk // S)
    o_c, lse_c = o.float().cpu().numpy(), lse.cpu().numpy()
    for b in range(B):
        for h in range(Hq):
            for i in range(Tq):
                newest = i + off // 128 if causal else Tk - 1
                for s in range(S):   # every range is its own run of the rule: its own visiting order and band
                    js = [j for j in range(min(newest, (s + 1) * tps - 1), s * tps - 1, -1)]
                    sel = np.zeros(Tk, dtype=bool)
                    sel[js] = True
                    parity.check_mask(np.where(sel, fm[b, h, i], False), np.where(sel, ref["mask"][b, h, i], 0),
                                      ref["crit"][b, h, i], js, tau, i * 128 + 1 + off if causal else Nk)
                assert int(st.retained[b, h, i]) == int(fm[b, h, i].sum())
    parity.check_output(o_c, ref["o"])
    assert np.abs(lse_c - ref["lse"]).max() <= parity.LSE_ABS
    assert st.totals.cpu().numpy()[1] == int((ref["mask"] > 0).sum())
    return int((ref["mask"] == 1).sum())


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("Nk,Nq,d,Hq,Hkv,S", [(1024, 128, 128, 2, 1, 4), (1152, 256, 128, 4, 2, 3), (1000, 232, 128, 2, 2, 8),
                                              (768, 384, 64, 2, 1, 2), (640, 640, 128, 2, 1, 5), (512, 128, 128, 2, 1, 9)])
def test_chunk_split_literal(mala, oracle, Nk, Nq, d, Hq, Hkv, S, tau):
    """Key ranges on different CTAs; (640, 5): equal lengths, ranges of one key block, so that a range can hold only
    the diagonal block of the second query block of a pair; (512, 9): more ranges than key blocks."""
    w = W.custom_prefill(2, Hq, Hkv, Nk, d, seed=Nk + Nq + S)
    _run_split(mala, oracle, _chunk(w, Nq), tau, S)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("Nk,Nq,S", [(4096, 256, 8), (2560, 512, 5)])
def test_chunk_split_skipping_regime(mala, oracle, Nk, Nq, S, tau):
    w = W.custom_prefill(1, 4, 2, Nk, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=7, preset="R")
    assert _run_split(mala, oracle, _chunk(w, Nq), tau, S) > 0, "workload must exercise skipping"


def test_chunk_split_non_causal(mala, oracle):
    w = W.custom_prefill(1, 2, 1, 1100, 128, head_types=["peaked", "diffuse"], seed=5, preset="R")
    _run_split(mala, oracle, _chunk(w, 200), 1e-2, 3, causal=False)


def test_chunk_split_of_one_range_equals_the_unsplit_call(mala):
    w = W.custom_prefill(1, 4, 2, 1536, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=3, preset="R")
    q, k, v = (w[x].cuda() for x in ("q", "k", "v"))
    o1, l1, _ = mala.fwd_chunk(q[:, 1024:], k, v, w["scale"], 1e-4)
    o2, l2, _ = mala.fwd_chunk_split(q[:, 1024:], k, v, w["scale"], 1e-4, 1)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
