"""GPU parity of mala_fwd_varlen / mala_bwd_varlen (packed sequences of different lengths) against the fp64 oracle,
which runs every sequence on its own."""
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


def _run(mala, oracle, lens, Hq, Hkv, d, tau, preset="literal", causal=True, head_types=None):
    ws = [W.custom_prefill(1, Hq, Hkv, n, d, head_types=head_types, seed=100 + 7 * x + n, preset=preset)
          for x, n in enumerate(lens)]
    pk = W.pack_sequences(ws)
    q, k, v, do, cu = (pk[x].cuda() for x in ("q", "k", "v", "do", "cu_seqlens"))
    mx = max(lens)
    o, lse, fst = mala.fwd_varlen(q, k, v, cu, mx, pk["scale"], tau, causal=causal, stats=True)
    dq, dk, dv, bst = mala.bwd_varlen(q, k, v, o, do, lse, cu, mx, pk["scale"], tau, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    Tm = -(-mx // 128)
    fm, bm = fst.mask(Tm).cpu().numpy(), bst.mask(Tm).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy()[0], lse.cpu().numpy()
    dq_c, dk_c, dv_c = (t.float().cpu().numpy()[0] for t in (dq, dk, dv))
    skipped = legal_f = legal_b = 0
    for b, (w, n) in enumerate(zip(ws, lens)):
        r0 = int(pk["cu_seqlens"][b])
        T = -(-n // 128)
        ref = oracle.fwd(w["q"], w["k"], w["v"], w["scale"], tau, 128, 128, causal=causal)
        for h in range(Hq):
            for i in range(T):
                order = list(range(i, -1, -1)) if causal else list(range(T - 1, -1, -1))
                parity.check_mask(fm[b, h, i, :T], ref["mask"][0, h, i], ref["crit"][0, h, i], order, tau,
                                  i * 128 + 1 if causal else n)
                assert int(fst.retained[b, h, i]) == int(fm[b, h, i].sum())
            assert not fm[b, h, T:].any() and not fm[b, h, :, T:].any()
        parity.check_output(o_c[r0:r0 + n], ref["o"][0])
        assert np.abs(lse_c[:, r0:r0 + n] - ref["lse"][0]).max() <= parity.LSE_ABS
        # backward on the GPU's own forward output of this sequence
        g = oracle.bwd(w["q"], w["k"], w["v"], o[:, r0:r0 + n].float().cpu(), w["do"],
                       lse[:, r0:r0 + n].cpu().numpy()[None], w["scale"], tau, 128, 128, causal=causal)
        flipped = False
        for h in range(Hq):
            for j in range(T):
                om, oc = g["mask"][0, h, j], g["crit"][0, h, j]
                for i in range(T):
                    if om[i] == 0:
                        assert not bm[b, h, j, i]
                    elif bool(bm[b, h, j, i]) != (om[i] == 2):
                        assert abs(oc[i]) <= parity.MASK_BAND, (b, h, j, i, oc[i])
                        flipped = True
            assert not bm[b, h, T:].any()
        # (a tile decided the other way inside the exemption band -- e.g. one key at tau = 1, where p = tau / L exactly --
        # changes the gradients by that tile's whole contribution: nothing to compare element by element then)
        for got, want, what in (() if flipped else ((dq_c, g["dq"], "dq"), (dk_c, g["dk"], "dk"), (dv_c, g["dv"], "dv"))):
            if n == 1 and what != "dv":
                # one key: p = 1 and dS = p (dP - D) = 0 exactly; the kernel's D comes from the bf16 output
                assert np.abs(got[r0:r0 + n]).max() <= 1e-2 * np.abs(want).max() + 1e-5
            else:
                parity.check_grad(got[r0:r0 + n], want[0], f"{what} seq {b}")
        skipped += int((ref["mask"] == 1).sum()) + int((g["mask"] == 1).sum())
        legal_f += int((ref["mask"] > 0).sum())
        legal_b += int((g["mask"] > 0).sum())
    assert fst.totals.cpu().numpy()[1] == legal_f and bst.totals.cpu().numpy()[1] == legal_b
    return skipped


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("lens,Hq,Hkv,d", [([128, 384, 256], 2, 1, 128), ([333, 100, 1, 517], 4, 2, 128),
                                           ([200, 640, 129], 2, 2, 64), ([700], 2, 1, 128)])
def test_varlen_literal(mala, oracle, lens, Hq, Hkv, d, tau):
    _run(mala, oracle, lens, Hq, Hkv, d, tau)


@pytest.mark.parametrize("tau", [1e-4, 1.0])
def test_varlen_skipping_regime(mala, oracle, tau):
    sk = _run(mala, oracle, [1024, 300, 1500, 777], 4, 2, 128, tau, preset="R",
              head_types=["diffuse", "peaked", "peaked", "sink"])
    assert sk > 0, "workload must exercise skipping"


@pytest.mark.parametrize("tau", [0.0, 1e-2])
def test_varlen_non_causal(mala, oracle, tau):
    # every key of the sequence legal: the rows of the next sequence inside a sequence's last tile must be masked
    _run(mala, oracle, [300, 130, 450], 2, 1, 128, tau, preset="R", causal=False, head_types=["peaked", "diffuse"])


def test_varlen_of_equal_lengths_equals_the_batched_call(mala):
    w = W.custom_prefill(3, 4, 2, 512, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=3, preset="R")
    q, k, v = (w[x].cuda() for x in ("q", "k", "v"))
    cu = torch.tensor([0, 512, 1024, 1536], dtype=torch.int32, device="cuda")
    for tau in (0.0, 1e-4):
        o, lse, _ = mala.fwd(q, k, v, w["scale"], tau)
        ov, lv, _ = mala.fwd_varlen(q.reshape(1, 1536, 4, 128), k.reshape(1, 1536, 2, 128), v.reshape(1, 1536, 2, 128),
                                    cu, 512, w["scale"], tau)
        assert torch.equal(o.reshape(1, 1536, 4, 128), ov)
        assert torch.equal(lse.permute(1, 0, 2).reshape(4, 1536), lv)


def test_varlen_with_an_empty_sequence(mala, oracle):
    # cu_seqlens = [0, 200, 200, 456]: the second sequence has no rows; the others must come out as if it were not there
    ws = [W.custom_prefill(1, 2, 1, n, 128, seed=50 + n) for n in (200, 256)]
    pk = W.pack_sequences(ws)
    q, k, v, do = (pk[x].cuda() for x in ("q", "k", "v", "do"))
    cu3 = torch.tensor([0, 200, 200, 456], dtype=torch.int32, device="cuda")
    cu2 = torch.tensor([0, 200, 456], dtype=torch.int32, device="cuda")
    for tau in (0.0, 1e-4):
        o3, l3, _ = mala.fwd_varlen(q, k, v, cu3, 256, pk["scale"], tau)
        o2, l2, _ = mala.fwd_varlen(q, k, v, cu2, 256, pk["scale"], tau)
        assert torch.equal(o3, o2) and torch.equal(l3, l2)
        g3 = mala.bwd_varlen(q, k, v, o3, do, l3, cu3, 256, pk["scale"], tau)
        g2 = mala.bwd_varlen(q, k, v, o2, do, l2, cu2, 256, pk["scale"], tau)
        torch.cuda.synchronize()
        assert mala.device_status() == 0
        for a, b_ in zip(g3[:3], g2[:3]):
            assert (a.float() - b_.float()).abs().max() <= 1e-2 * b_.float().abs().max()
    ref = oracle.fwd(ws[1]["q"], ws[1]["k"], ws[1]["v"], pk["scale"], 1e-4, 128, 128)
    parity.check_output(o3.float().cpu().numpy()[0, 200:], ref["o"][0])


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("causal", [True, False])
def test_varlen_with_cached_prefixes(mala, oracle, tau, causal):
    """Packed prefill chunks behind prefixes of different lengths (chunks that start inside a tile included): every
    sequence against the oracle's chunk rule with its query blocks laid out by position."""
    Hq, Hkv, d = 4, 2, 128
    nk = [900, 128, 517, 300, 64]
    nq = [260, 128, 100, 1, 64]                       # prefix lengths 640, 0, 417, 299, 0
    ws = [W.custom_prefill(1, Hq, Hkv, n, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=60 + x, preset="R")
          for x, n in enumerate(nk)]
    q = torch.cat([w["q"][:, n - m:] for w, n, m in zip(ws, nk, nq)], dim=1).contiguous()
    k = torch.cat([w["k"] for w in ws], dim=1).contiguous()
    v = torch.cat([w["v"] for w in ws], dim=1).contiguous()
    cq = torch.tensor(np.concatenate([[0], np.cumsum(nq)]), dtype=torch.int32)
    ck = torch.tensor(np.concatenate([[0], np.cumsum(nk)]), dtype=torch.int32)
    o, lse, st = mala.fwd_varlen_prefix(q.cuda(), k.cuda(), v.cuda(), cq.cuda(), ck.cuda(), max(nq), max(nk),
                                        ws[0]["scale"], tau, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    Tkm = -(-max(nk) // 128)
    fm = st.mask(Tkm).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy()[0], lse.cpu().numpy()
    legal = skipped = 0
    for b, (w, n, m) in enumerate(zip(ws, nk, nq)):
        off = n - m
        shift = off % 128 if causal else 0
        ref = oracle.fwd(w["q"][:, n - m:], w["k"], w["v"], w["scale"], tau, 128, 128, causal=causal, q_shift=shift)
        Tq, Tk = ref["mask"].shape[2], ref["mask"].shape[3]
        r0 = int(cq[b])
        for h in range(Hq):
            for i in range(Tq):
                order = list(range(i + off // 128, -1, -1)) if causal else list(range(Tk - 1, -1, -1))
                parity.check_mask(fm[b, h, i, :Tk], ref["mask"][0, h, i], ref["crit"][0, h, i], order, tau,
                                  max(i * 128 - shift, 0) + 1 + off if causal else n)
            assert not fm[b, h, Tq:].any() and not fm[b, h, :, Tk:].any()
        parity.check_output(o_c[r0:r0 + m], ref["o"][0])
        assert np.abs(lse_c[:, r0:r0 + m] - ref["lse"][0]).max() <= parity.LSE_ABS
        legal += int((ref["mask"] > 0).sum())
        skipped += int((ref["mask"] == 1).sum())
    assert st.totals.cpu().numpy()[1] == legal
    if tau > 0 and causal:
        assert skipped > 0
    # backward on the GPU's own forward output: every sequence against the oracle's chunk backward
    do = torch.cat([w["do"][:, n - m:] for w, n, m in zip(ws, nk, nq)], dim=1).contiguous()
    dq, dk, dv, bst = mala.bwd_varlen_prefix(q.cuda(), k.cuda(), v.cuda(), o, do.cuda(), lse, cq.cuda(), ck.cuda(),
                                             max(nq), max(nk), ws[0]["scale"], tau, causal=causal, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    Tqm = -(-(max(nq) + 127) // 128)
    bm = bst.mask(Tqm).cpu().numpy()                     # [B,Hq,Tkm,Tqm]
    legal_b = 0
    for b, (w, n, m) in enumerate(zip(ws, nk, nq)):
        shift = (n - m) % 128 if causal else 0
        r0, k0 = int(cq[b]), int(ck[b])
        rb = oracle.bwd(w["q"][:, n - m:], w["k"], w["v"], o[:, r0:r0 + m].float().cpu(), w["do"][:, n - m:],
                        lse_c[None, :, r0:r0 + m], w["scale"], tau, 128, 128, causal=causal, q_shift=shift)
        Tk, Tq = rb["mask"].shape[2], rb["mask"].shape[3]
        for h in range(Hq):
            for j in range(Tk):
                om, oc = rb["mask"][0, h, j], rb["crit"][0, h, j]
                for i in range(Tq):
                    if om[i] == 0:
                        assert not bm[b, h, j, i]
                    elif bool(bm[b, h, j, i]) != (om[i] == 2):
                        assert abs(oc[i]) <= parity.MASK_BAND, (b, h, j, i, oc[i])
            assert not bm[b, h, Tk:].any() and not bm[b, h, :, Tq:].any()
        if m > 1:
            parity.check_grad(dq[0, r0:r0 + m].float().cpu().numpy(), rb["dq"][0], "dq")
        else:     # (a single query: its gradient may be exactly zero, see the packed test above)
            assert np.abs(dq[0, r0:r0 + m].float().cpu().numpy() - rb["dq"][0]).max() <= 1e-2 * max(np.abs(rb["dq"]).max(), 1e-3)
        parity.check_grad(dk[0, k0:k0 + n].float().cpu().numpy(), rb["dk"][0], "dk")
        parity.check_grad(dv[0, k0:k0 + n].float().cpu().numpy(), rb["dv"][0], "dv")
        legal_b += int((rb["mask"] > 0).sum())
    assert bst.totals.cpu().numpy()[1] == legal_b


def test_varlen_prefix_backward_sequences_without_queries_get_zero_gradients(mala):
    Hq, Hkv, d = 2, 1, 64
    nk, nq = [300, 200, 140], [100, 0, 140]
    w = W.custom_prefill(1, Hq, Hkv, sum(nk), d, seed=88)
    q = w["q"][:, :sum(nq)].contiguous().cuda()
    do = w["do"][:, :sum(nq)].contiguous().cuda()
    k, v = w["k"].cuda(), w["v"].cuda()
    cq = torch.tensor(np.concatenate([[0], np.cumsum(nq)]), dtype=torch.int32).cuda()
    ck = torch.tensor(np.concatenate([[0], np.cumsum(nk)]), dtype=torch.int32).cuda()
    o, lse, _ = mala.fwd_varlen_prefix(q, k, v, cq, ck, max(nq), max(nk), w["scale"], 1e-4)
    dq, dk, dv, _ = mala.bwd_varlen_prefix(q, k, v, o, do, lse, cq, ck, max(nq), max(nk), w["scale"], 1e-4)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert (dk[0, 300:500] == 0).all() and (dv[0, 300:500] == 0).all()
    assert dk[0, :300].float().abs().max() > 0 and dk[0, 500:].float().abs().max() > 0
    # the neighbours are what separate calls give
    for b, (r0, k0) in enumerate([(0, 0), (100, 300), (100, 500)]):
        if nq[b] == 0:
            continue
        qs, ks, vs = q[:, r0:r0 + nq[b]], k[:, k0:k0 + nk[b]], v[:, k0:k0 + nk[b]]
        o1, l1, _ = mala.fwd_chunk(qs.contiguous(), ks.contiguous(), vs.contiguous(), w["scale"], 1e-4)
        g = mala.bwd_chunk(qs.contiguous(), ks.contiguous(), vs.contiguous(), o1, do[:, r0:r0 + nq[b]].contiguous(), l1,
                           w["scale"], 1e-4)
        assert torch.equal(o1, o[:, r0:r0 + nq[b]])
        assert torch.equal(g[1], dk[:, k0:k0 + nk[b]]) and torch.equal(g[2], dv[:, k0:k0 + nk[b]])
        assert (g[0].float() - dq[:, r0:r0 + nq[b]].float()).abs().max() <= 1e-2 * g[0].float().abs().max()


@pytest.mark.parametrize("tau", [0.0, 1e-4])
@pytest.mark.parametrize("page,d", [(128, 128), (256, 128), (16, 128), (64, 128), (8, 64), (32, 96), (128, 40),
                                    (256, 256), (16, 256), (128, 200), (8, 256), (8, 136)])
def test_prefill_chunks_against_a_paged_cache(mala, oracle, tau, page, d):
    """Packed prefill chunks whose keys and values (prefix and chunk) lie in pages scattered over a shuffled pool."""
    Hq, Hkv = 4, 2
    nk = [900, 128, 517, 300]
    nq = [260, 128, 100, 1]
    ws = [W.custom_prefill(1, Hq, Hkv, n, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=70 + x, preset="R")
          for x, n in enumerate(nk)]
    Nmax = -(-max(nk) // page) * page
    kc = torch.zeros((len(nk), Nmax, Hkv, d), dtype=torch.bfloat16)
    vc = torch.zeros_like(kc)
    for b, (w, n) in enumerate(zip(ws, nk)):
        kc[b, :n], vc[b, :n] = w["k"][0], w["v"][0]
    kp, vp, bt, sl = W.paginate(kc, vc, page, seqlens=nk, seed=page)
    q = torch.cat([w["q"][:, n - m:] for w, n, m in zip(ws, nk, nq)], dim=1).contiguous()
    cq = torch.tensor(np.concatenate([[0], np.cumsum(nq)]), dtype=torch.int32)
    o, lse, st = mala.fwd_paged(q.cuda(), kp.cuda(), vp.cuda(), cq.cuda(), bt.cuda(), sl.cuda(), max(nq), ws[0]["scale"],
                                tau, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    fm = st.mask(-(-Nmax // 128)).cpu().numpy()
    o_c, lse_c = o.float().cpu().numpy()[0], lse.cpu().numpy()
    legal = 0
    for b, (w, n, m) in enumerate(zip(ws, nk, nq)):
        off = n - m
        ref = oracle.fwd(w["q"][:, n - m:], w["k"], w["v"], w["scale"], tau, 128, 128, q_shift=off % 128)
        Tq, Tk = ref["mask"].shape[2], ref["mask"].shape[3]
        r0 = int(cq[b])
        for h in range(Hq):
            for i in range(Tq):
                parity.check_mask(fm[b, h, i, :Tk], ref["mask"][0, h, i], ref["crit"][0, h, i],
                                  list(range(i + off // 128, -1, -1)), tau, max(i * 128 - off % 128, 0) + 1 + off)
        parity.check_output(o_c[r0:r0 + m], ref["o"][0])
        assert np.abs(lse_c[:, r0:r0 + m] - ref["lse"][0]).max() <= parity.LSE_ABS
        legal += int((ref["mask"] > 0).sum())
    assert st.totals.cpu().numpy()[1] == legal


@pytest.mark.parametrize("page", [128, 16])
def test_paged_prefill_clamps_a_length_beyond_the_block_table(mala, page):
    """A sequence that reports more keys than its block-table row can map is treated as holding exactly what the row
    maps: no table lookup leaves the row, and the result equals the call with the clamped length."""
    Hq, Hkv, d, nk, nq = 4, 2, 128, 1024, 100
    w = W.custom_prefill(1, Hq, Hkv, nk, d, seed=91, preset="R")
    kp, vp, bt, _ = W.paginate(w["k"], w["v"], page, seqlens=[nk], seed=3)
    assert bt.shape[1] * page == nk
    q = w["q"][:, nk - nq:].contiguous().cuda()
    cq = torch.tensor([0, nq], dtype=torch.int32).cuda()
    outs = []
    for reported in (nk, 5 * nk):
        sl = torch.tensor([reported], dtype=torch.int32).cuda()
        o, lse, _ = mala.fwd_paged(q, kp.cuda(), vp.cuda(), cq, bt.cuda(), sl, nq, w["scale"], 1e-4)
        torch.cuda.synchronize()
        assert mala.device_status() == 0
        outs.append((o, lse))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
