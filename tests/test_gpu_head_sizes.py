"""Head sizes other than 64 and 128 (any multiple of 8 up to 128; up to 256 in the forward and the decode step): every
entry point against the oracle.  The kernels run them on the next of their column counts with the missing columns read as zeros, so what
these cases guard is that nothing beyond column d is stored and that the zero columns change no result; above 128 the
forward runs one query block per CTA and the decode step 64 KB tiles with two output accumulators, which the cases
at 136 to 256 columns cover on every forward and decode entry point."""
import numpy as np
import pytest
import torch

from paper_2609_32712_b200 import workloads as W
from tests import parity
from tests.test_gpu_chunk import _chunk, _run, _run_bwd_any_offset, _run_fwd_any_offset, _run_split
from tests.test_gpu_decode import _run_and_check, _run_multi, _run_paged
from tests.test_gpu_fwd import _run_and_check as _run_fwd

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mala():
    from paper_2609_32712_b200 import mala as m
    m.lib()
    return m


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("d,N,Hq,Hkv", [(96, 640, 4, 2), (80, 500, 2, 1), (32, 700, 2, 2), (8, 300, 2, 1), (120, 257, 2, 1),
                                        (40, 384, 4, 1)])
def test_forward_and_backward_literal(mala, oracle, d, N, Hq, Hkv, tau):
    w = W.custom_prefill(2, Hq, Hkv, N, d, seed=d + N)
    _run(mala, oracle, _chunk(w, N), tau)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("d", [96, 48])
def test_forward_and_backward_skipping_regime(mala, oracle, d, tau):
    w = W.custom_prefill(1, 4, 2, 2048, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=d, preset="R")
    assert _run(mala, oracle, _chunk(w, 2048), tau) > 0, "workload must exercise skipping"


@pytest.mark.parametrize("d", [96, 24])
def test_chunks_and_key_ranges(mala, oracle, d):
    w = W.custom_prefill(1, 4, 2, 1500, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=d + 1, preset="R")
    _run(mala, oracle, _chunk(w, 348), 1e-4)                      # starts on a tile boundary
    _run_fwd_any_offset(mala, oracle, _chunk(w, 333), 1e-4)
    _run_fwd_any_offset(mala, oracle, _chunk(w, 333), 1e-4, S=3)
    _run_bwd_any_offset(mala, oracle, _chunk(w, 333), 1e-4)
    _run_split(mala, oracle, _chunk(w, 220), 1e-4, 4)
    _run(mala, oracle, _chunk(w, 200), 1e-2, causal=False)


def test_nothing_is_stored_beyond_the_head_size(mala):
    # outputs are views of wider buffers filled with a sentinel: the columns past d must keep it
    d, dw, N = 96, 128, 400
    w = W.custom_prefill(1, 2, 1, N, d, seed=5)
    q, k, v, do = (w[x].cuda() for x in ("q", "k", "v", "do"))

    def wide(like):
        buf = torch.full(like.shape[:-1] + (dw,), 7.0, dtype=torch.bfloat16, device="cuda")
        return buf, buf[..., :d]

    ob, o = wide(q)
    mala.fwd(q, k, v, w["scale"], 1e-4, out=o)
    lse = mala.fwd(q, k, v, w["scale"], 1e-4)[1]
    (dqb, dq), (dkb, dk), (dvb, dv) = wide(q), wide(k), wide(v)
    mala.bwd(q, k, v, o, do, lse, w["scale"], 1e-4, dq=dq, dk=dk, dv=dv)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    for buf in (ob, dqb, dkb, dvb):
        assert (buf[..., d:] == 7.0).all() and not (buf[..., :d] == 7.0).all()
    o2, _, _ = mala.fwd(q, k, v, w["scale"], 1e-4)
    assert torch.equal(o2, o)


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("d,Nk,S,Hq,Hkv", [(96, 1024, 4, 8, 2), (80, 1000, 3, 8, 4), (32, 4096, 8, 16, 1), (8, 300, 2, 6, 2),
                                           (120, 2048, 4, 3, 1)])
def test_decode_literal(mala, oracle, d, Nk, S, Hq, Hkv, tau):
    w = W.custom_decode(2, Hq, Hkv, Nk, d, S, seed=Nk + d)
    _run_and_check(mala, oracle, w, tau, S)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("d", [96, 40])
def test_decode_gated_paged_several_tokens(mala, oracle, d, tau):
    w = W.custom_decode(2, 8, 2, 8192, d, 8, group_types=["diffuse", "peaked"], seed=3 + d, preset="D")
    res = _run_and_check(mala, oracle, w, tau, 8)
    assert res["skipped"] > 0, "workload must exercise skipping"
    _run_paged(mala, oracle, w, tau, 8, 256, [8192, 4096 + 77], seed=9)
    _run_paged(mala, oracle, w, tau, 8, 16, [8192, 1000], seed=10)
    assert _run_multi(mala, oracle, w, 3, tau, 8) > 0


def test_head_sizes_that_are_refused(mala):
    for d in (4, 100, 260, 264, 512):
        q = torch.zeros(1, 256, 2, d, dtype=torch.bfloat16, device="cuda")
        with pytest.raises(mala.MalaError) as e:
            mala.fwd(q, q, q, 0.1, 0.0)
        assert e.value.code in (-2, -3)
    for d in (136, 256):          # the backward stops at 128 columns
        q = torch.zeros(1, 256, 2, d, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(1, 2, 256, dtype=torch.float32, device="cuda")
        with pytest.raises(mala.MalaError) as e:
            mala.bwd(q, q, q, q, q, lse, 0.1, 0.0)
        assert e.value.code == -2


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("d,N,Hq,Hkv", [(256, 640, 4, 2), (256, 128, 1, 1), (192, 500, 2, 1), (136, 700, 2, 2), (160, 257, 2, 1),
                                        (256, 1100, 2, 1)])
def test_forward_above_128_columns_literal(mala, oracle, d, N, Hq, Hkv, tau):
    w = W.custom_prefill(2, Hq, Hkv, N, d, seed=d + N)
    _run_fwd(mala, oracle, w, tau)
    _run_fwd(mala, oracle, w, tau, causal=False)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("d", [256, 192])
def test_forward_above_128_columns_skipping_regime(mala, oracle, d, tau):
    w = W.custom_prefill(1, 4, 2, 2048, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=d, preset="R")
    res = _run_fwd(mala, oracle, w, tau, rounding_bound=True)
    assert res["skipped"] > 0, "workload must exercise skipping"


@pytest.mark.parametrize("d", [256, 144])
def test_forward_above_128_columns_chunks_and_key_ranges(mala, oracle, d):
    w = W.custom_prefill(1, 4, 2, 1500, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=d + 1, preset="R")
    _run_fwd_any_offset(mala, oracle, _chunk(w, 333), 1e-4)
    _run_fwd_any_offset(mala, oracle, _chunk(w, 333), 1e-4, S=3)
    _run_fwd_any_offset(mala, oracle, _chunk(w, 348), 0.0)
    _run_split(mala, oracle, _chunk(w, 220), 1e-4, 4)
    _run_split(mala, oracle, _chunk(w, 220), 0.0, 5)


def test_forward_above_128_columns_stores_nothing_beyond_the_head_size(mala):
    d, dw, N = 192, 256, 400
    w = W.custom_prefill(1, 2, 1, N, d, seed=5)
    q, k, v = (w[x].cuda() for x in ("q", "k", "v"))
    ob = torch.full(q.shape[:-1] + (dw,), 7.0, dtype=torch.bfloat16, device="cuda")
    o = ob[..., :d]
    for tau in (0.0, 1e-4):
        mala.fwd(q, k, v, w["scale"], tau, out=o)
        torch.cuda.synchronize()
        assert mala.device_status() == 0
        assert (ob[..., d:] == 7.0).all() and not (ob[..., :d] == 7.0).all()
        assert torch.equal(mala.fwd(q, k, v, w["scale"], tau)[0], o)
    # the result on the inputs padded with zero columns to the kernel's width is the same
    pad = lambda t: torch.cat([t, torch.zeros(t.shape[:-1] + (dw - d,), dtype=t.dtype, device=t.device)], dim=-1)
    op, lsep, _ = mala.fwd(pad(q), pad(k), pad(v), w["scale"], 1e-4)
    o1, lse1, _ = mala.fwd(q, k, v, w["scale"], 1e-4)
    assert torch.equal(op[..., :d], o1) and torch.equal(lsep, lse1) and (op[..., d:] == 0).all()


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("d,Nk,S,Hq,Hkv", [(256, 1024, 4, 8, 2), (256, 1000, 3, 8, 1), (192, 4096, 8, 16, 1), (136, 300, 2, 6, 2),
                                           (256, 2048, 4, 3, 1), (256, 128, 1, 1, 1)])
def test_decode_above_128_columns_literal(mala, oracle, d, Nk, S, Hq, Hkv, tau):
    w = W.custom_decode(2, Hq, Hkv, Nk, d, S, seed=Nk + d)
    _run_and_check(mala, oracle, w, tau, S)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
@pytest.mark.parametrize("d", [256, 160])
def test_decode_above_128_columns_gated_paged_several_tokens(mala, oracle, d, tau):
    w = W.custom_decode(2, 8, 2, 8192, d, 8, group_types=["diffuse", "peaked"], seed=3 + d, preset="D")
    res = _run_and_check(mala, oracle, w, tau, 8)
    assert res["skipped"] > 0, "workload must exercise skipping"
    _run_paged(mala, oracle, w, tau, 8, 256, [8192, 4096 + 77], seed=9)
    _run_paged(mala, oracle, w, tau, 8, 16, [8192, 1000], seed=10)
    _run_paged(mala, oracle, w, tau, 8, 8, [700, 8192], seed=11)
    assert _run_multi(mala, oracle, w, 3, tau, 8) > 0


def test_decode_above_128_columns_stores_nothing_beyond_the_head_size(mala):
    d, dw = 192, 256
    w = W.custom_decode(2, 8, 2, 3000, d, 4, seed=8, device="cuda")
    ob = torch.full(w["q"].shape[:-1] + (dw,), 7.0, dtype=torch.bfloat16, device="cuda")
    o = ob[..., :d]
    mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], 1e-4, 4, out=o)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert (ob[..., d:] == 7.0).all() and not (ob[..., :d] == 7.0).all()
    assert torch.equal(mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], 1e-4, 4)[0], o)


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("d,causal", [(256, True), (168, True), (256, False)])
def test_forward_above_128_columns_packed_sequences_behind_prefixes(mala, oracle, d, causal, tau):
    """mala_fwd_varlen and mala_fwd_varlen_prefix (forward only) with one query block per CTA: sequences of different
    lengths, chunks that start inside a tile, a chunk of one query."""
    Hq, Hkv = 4, 2
    nk = [900, 128, 517, 300, 64]
    nq = [260, 128, 100, 1, 64]
    ws = [W.custom_prefill(1, Hq, Hkv, n, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=60 + x, preset="R")
          for x, n in enumerate(nk)]
    q = torch.cat([w["q"][:, n - m:] for w, n, m in zip(ws, nk, nq)], dim=1).contiguous()
    k = torch.cat([w["k"] for w in ws], dim=1).contiguous()
    v = torch.cat([w["v"] for w in ws], dim=1).contiguous()
    cq = torch.tensor(np.concatenate([[0], np.cumsum(nq)]), dtype=torch.int32)
    ck = torch.tensor(np.concatenate([[0], np.cumsum(nk)]), dtype=torch.int32)
    o, lse, st = mala.fwd_varlen_prefix(q.cuda(), k.cuda(), v.cuda(), cq.cuda(), ck.cuda(), max(nq), max(nk),
                                        ws[0]["scale"], tau, causal=causal, stats=True)
    o2, lse2, st2 = mala.fwd_varlen(torch.cat([w["q"] for w in ws], dim=1).contiguous().cuda(), k.cuda(), v.cuda(), ck.cuda(),
                                    max(nk), ws[0]["scale"], tau, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    fm = st.mask(-(-max(nk) // 128)).cpu().numpy()
    fm2 = st2.mask(-(-max(nk) // 128)).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy()[0], lse.cpu().numpy()
    o2_c, lse2_c = o2.float().cpu().numpy()[0], lse2.cpu().numpy()
    for b, (w, n, m) in enumerate(zip(ws, nk, nq)):
        off = n - m
        shift = off % 128 if causal else 0
        ref = oracle.fwd(w["q"][:, n - m:], w["k"], w["v"], w["scale"], tau, 128, 128, causal=causal, q_shift=shift)
        ref_abs = oracle.fwd(w["q"][:, n - m:], w["k"], w["v"].abs(), w["scale"], tau, 128, 128, causal=causal, q_shift=shift)
        Tq, Tk = ref["mask"].shape[2], ref["mask"].shape[3]
        r0 = int(cq[b])
        for h in range(Hq):
            for i in range(Tq):
                order = list(range(i + off // 128, -1, -1)) if causal else list(range(Tk - 1, -1, -1))
                parity.check_mask(fm[b, h, i, :Tk], ref["mask"][0, h, i], ref["crit"][0, h, i], order, tau,
                                  (max(i * 128 - shift, 0) + 1 + off) if causal else n)
        parity.check_output(o_c[r0:r0 + m], ref["o"][0], a_ref=ref_abs["o"][0])
        assert np.abs(lse_c[:, r0:r0 + m] - ref["lse"][0]).max() <= parity.LSE_ABS
        # the whole sequence as its own packed sequence
        full = oracle.fwd(w["q"], w["k"], w["v"], w["scale"], tau, 128, 128, causal=causal)
        full_abs = oracle.fwd(w["q"], w["k"], w["v"].abs(), w["scale"], tau, 128, 128, causal=causal)
        k0, T = int(ck[b]), -(-n // 128)
        for h in range(Hq):
            for i in range(T):
                order = list(range(i, -1, -1)) if causal else list(range(T - 1, -1, -1))
                parity.check_mask(fm2[b, h, i, :T], full["mask"][0, h, i], full["crit"][0, h, i], order, tau,
                                  i * 128 + 1 if causal else n)
        parity.check_output(o2_c[k0:k0 + n], full["o"][0], a_ref=full_abs["o"][0])
        assert np.abs(lse2_c[:, k0:k0 + n] - full["lse"][0]).max() <= parity.LSE_ABS
