"""GPU checks beyond plain parity: strided tensor views, run-to-run determinism, tau-monotonic support,
ragged mid-size shapes in the skipping regime, and error reporting through the binding."""
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


def _bhnd_view(t):
    """Same values, stored [B,H,N,d] and viewed as [B,N,H,d] (strides sn = d, sh = N*d)."""
    return t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)


def test_strided_views_give_identical_results(mala):
    w = W.custom_prefill(2, 4, 2, 640, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=31, preset="R")
    q, k, v, do = (w[x].cuda() for x in ("q", "k", "v", "do"))
    tau = 1e-4
    o, lse, st = mala.fwd(q, k, v, w["scale"], tau, stats=True)
    dq, dk, dv, _ = mala.bwd(q, k, v, o, do, lse, w["scale"], tau)
    qs, ks, vs, dos = (_bhnd_view(t) for t in (q, k, v, do))
    assert qs.stride() != q.stride()
    o2 = _bhnd_view(torch.empty_like(q))
    o2, lse2, st2 = mala.fwd(qs, ks, vs, w["scale"], tau, stats=True, out=o2)
    dq2, dk2, dv2 = (_bhnd_view(torch.empty_like(t)) for t in (q, k, v))
    mala.bwd(qs, ks, vs, o2, dos, lse2, w["scale"], tau, dq=dq2, dk=dk2, dv=dv2)
    torch.cuda.synchronize()
    assert torch.equal(o, o2) and torch.equal(lse, lse2) and torch.equal(st.bitmask, st2.bitmask)
    assert torch.equal(dk, dk2) and torch.equal(dv, dv2)
    assert (dq.float() - dq2.float()).abs().max() <= 1e-2 * dq.float().abs().max()   # fp32 adds in another order


def test_forward_and_mask_are_deterministic(mala):
    w = W.custom_prefill(1, 4, 2, 2048, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=33, preset="R")
    q, k, v, do = (w[x].cuda() for x in ("q", "k", "v", "do"))
    runs = []
    for _ in range(3):
        o, lse, st = mala.fwd(q, k, v, w["scale"], 1e-4, stats=True)
        dq, dk, dv, bst = mala.bwd(q, k, v, o, do, lse, w["scale"], 1e-4, stats=True)
        torch.cuda.synchronize()
        runs.append((o.clone(), lse.clone(), st.bitmask.clone(), dk.clone(), dv.clone(), bst.bitmask.clone(), dq.clone()))
    for r in runs[1:]:
        for a, b in zip(runs[0][:6], r[:6]):
            assert torch.equal(a, b)
        assert (runs[0][6].float() - r[6].float()).abs().max() <= 1e-2 * runs[0][6].float().abs().max()


def test_support_shrinks_as_tau_grows(mala):
    # tau1 (1 + tau2) <= tau2 for consecutive values: the support under tau1 contains the support under tau2
    w = W.custom_prefill(1, 4, 2, 4096, 128, head_types=["peaked", "peaked", "sink", "diffuse"], seed=35, preset="R")
    q, k, v = (w[x].cuda() for x in ("q", "k", "v"))
    masks = []
    for tau in (0.0, 1e-5, 1e-4, 1e-3, 1e-1, 1.0):
        _, _, st = mala.fwd(q, k, v, w["scale"], tau, stats=True)
        masks.append(st.mask(32))
    for a, b in zip(masks[:-1], masks[1:]):
        assert (b <= a).all()
    assert masks[-1].sum() < masks[1].sum()


@pytest.mark.parametrize("N,d,tau", [(3000, 128, 1e-4), (2900, 64, 1e-3), (5000, 128, 1.0)])
def test_ragged_mid_size_sampled(mala, oracle, N, d, tau):
    w = W.custom_prefill(1, 4, 2, N, d, head_types=["diffuse", "peaked", "peaked", "sink"], seed=N, preset="R")
    q, k, v, do = (w[x].cuda() for x in ("q", "k", "v", "do"))
    T = -(-N // 128)
    o, lse, fst = mala.fwd(q, k, v, w["scale"], tau, stats=True)
    dq, dk, dv, bst = mala.bwd(q, k, v, o, do, lse, w["scale"], tau, stats=True)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    fwd_units = [(0, 1, T - 1), (0, 2, T // 2), (0, 3, 1)]
    ref = oracle.fwd(w["q"], w["k"], w["v"], w["scale"], tau, 128, 128, units=fwd_units)
    fm = fst.mask(T).cpu().numpy()
    for (b, h, i) in fwd_units:
        rows = slice(i * 128, min(N, (i + 1) * 128))
        parity.check_mask(fm[b, h, i], ref["mask"][b, h, i], ref["crit"][b, h, i], list(range(i, -1, -1)), tau, i * 128 + 1)
        parity.check_output(o[b, rows, h].float().cpu().numpy(), ref["o"][b, rows, h])
    g = oracle.bwd(w["q"], w["k"], w["v"], o.float().cpu(), w["do"], lse.cpu().numpy(), w["scale"], tau, 128, 128,
                   key_units=[(0, 0, T - 1), (0, 1, T // 3)], dq_units=[(0, 2, T - 1)])
    for (b, hk, j) in [(0, 0, T - 1), (0, 1, T // 3)]:
        rows = slice(j * 128, min(N, (j + 1) * 128))
        parity.check_grad(dk[b, rows, hk].float().cpu().numpy(), g["dk"][b, rows, hk], "dk")
        parity.check_grad(dv[b, rows, hk].float().cpu().numpy(), g["dv"][b, rows, hk], "dv")
    rows = slice((T - 1) * 128, N)
    parity.check_grad(dq[0, rows, 2].float().cpu().numpy(), g["dq"][0, rows, 2], "dq")
    assert (bst.mask(T).transpose(2, 3) <= fst.mask(T)).all()


def test_binding_reports_errors(mala):
    q = torch.zeros(1, 256, 2, 128, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(1, 2, 256, device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(mala.MalaError) as e:
        mala.bwd(q, q, q, q, q, lse, 0.1, 1e-4, ws=small)
    assert e.value.code == -4
    with pytest.raises(mala.MalaError) as e:
        mala.fwd(q, q, q, 0.1, -1.0)
    assert e.value.code == -1
    q264 = torch.zeros(1, 256, 2, 264, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mala.MalaError) as e:
        mala.fwd(q264, q264, q264, 0.1, 0.0)
    assert e.value.code == -2
    q256 = torch.zeros(1, 256, 2, 256, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mala.MalaError) as e:        # the backward stops at 128 columns
        mala.bwd(q256, q256, q256, q256, q256, lse, 0.1, 0.0)
    assert e.value.code == -2
    q17 = torch.zeros(1, 1, 34, 128, dtype=torch.bfloat16, device="cuda")
    kv1 = torch.zeros(1, 256, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mala.MalaError) as e:        # decode packs at most 16 query heads per KV head
        mala.decode(q17, kv1, kv1, 0.1, 0.0, 2)
    assert e.value.code == -2
    assert mala.device_status() == 0


def test_calls_can_be_captured_in_a_cuda_graph(mala):
    """The library allocates nothing and never synchronises, so a decode step and a forward pass can be captured
    once and replayed on new inputs written into the same buffers."""
    wd = W.custom_decode(2, 8, 2, 4096, 128, 8, group_types=["diffuse", "peaked"], seed=31, preset="D")
    q, kc, vc = (wd[x].cuda() for x in ("q", "kcache", "vcache"))
    wp = W.custom_prefill(1, 4, 2, 1024, 128, seed=32, preset="R")
    pq, pk, pv = (wp[x].cuda() for x in ("q", "k", "v"))
    ws = torch.empty(mala.workspace_bytes(mala.OP_DECODE, 2, 8, 2, 4096, 128, 8), dtype=torch.uint8, device="cuda")
    o, lse = torch.empty_like(q), torch.empty((2, 8), dtype=torch.float32, device="cuda")
    po, plse = torch.empty_like(pq), torch.empty((1, 4, 1024), dtype=torch.float32, device="cuda")

    def step():
        mala.decode(q, kc, vc, wd["scale"], 1e-4, 8, ws=ws, out=o)
        mala.fwd(pq, pk, pv, wp["scale"], 1e-4, out=po, lse=plse)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                    # first calls outside the capture (one-time set-up per device)
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    # new inputs in the captured buffers, then replay and compare with direct calls
    q.copy_(torch.roll(q, 1, dims=2))
    pq.copy_(torch.roll(pq, 3, dims=1))
    graph.replay()
    torch.cuda.synchronize()
    o_g, po_g, plse_g = o.clone(), po.clone(), plse.clone()
    o_d, _, _ = mala.decode(q, kc, vc, wd["scale"], 1e-4, 8)
    po_d, plse_d, _ = mala.fwd(pq, pk, pv, wp["scale"], 1e-4)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    assert torch.equal(o_g, o_d) and torch.equal(po_g, po_d) and torch.equal(plse_g, plse_d)


def test_autograd_function_runs_both_algorithms(mala, oracle):
    from paper_2609_32712_b200.autograd import mala_attention
    w = W.custom_prefill(1, 4, 2, 640, 128, head_types=["diffuse", "peaked", "peaked", "sink"], seed=41, preset="R")
    for tau in (0.0, 1e-4):
        q, k, v = (w[x].cuda().requires_grad_(True) for x in ("q", "k", "v"))
        o = mala_attention(q, k, v, tau, scale=w["scale"])
        (o.float() * w["do"].cuda().float()).sum().backward()
        o_d, lse_d, _ = mala.fwd(q.detach(), k.detach(), v.detach(), w["scale"], tau)
        dq, dk, dv, _ = mala.bwd(q.detach(), k.detach(), v.detach(), o_d, w["do"].cuda(), lse_d, w["scale"], tau)
        assert torch.equal(o.detach(), o_d)
        for got, want in ((q.grad, dq), (k.grad, dk), (v.grad, dv)):
            assert (got.float() - want.float()).abs().max() <= 1e-2 * want.float().abs().max()
    # against the oracle at tau = 0: the exact gradient of dense attention
    q, k, v = (w[x].cuda().requires_grad_(True) for x in ("q", "k", "v"))
    mala_attention(q, k, v, 0.0, scale=w["scale"]).backward(w["do"].cuda())
    gq, gk, gv = oracle.dense_bwd(w["q"], w["k"], w["v"], w["do"], w["scale"])
    parity.check_grad(q.grad.float().cpu().numpy(), gq, "dq")
    parity.check_grad(k.grad.float().cpu().numpy(), gk, "dk")
    parity.check_grad(v.grad.float().cpu().numpy(), gv, "dv")


def test_autograd_functions_for_chunks_and_packed_sequences(mala):
    from paper_2609_32712_b200.autograd import mala_attention, mala_attention_packed
    w = W.custom_prefill(1, 4, 2, 900, 96, head_types=["diffuse", "peaked", "peaked", "sink"], seed=43, preset="R")
    tau, Nq = 1e-4, 333
    # a chunk of queries from a position inside a tile
    q = w["q"][:, 900 - Nq:].cuda().requires_grad_(True)
    k, v = (w[x].cuda().requires_grad_(True) for x in ("k", "v"))
    do = w["do"][:, 900 - Nq:].cuda()
    o = mala_attention(q, k, v, tau, scale=w["scale"])
    o.backward(do)
    o_d, lse_d, _ = mala.fwd_chunk(q.detach(), k.detach(), v.detach(), w["scale"], tau)
    dq, dk, dv, _ = mala.bwd_chunk(q.detach(), k.detach(), v.detach(), o_d, do, lse_d, w["scale"], tau)
    assert torch.equal(o.detach(), o_d) and torch.equal(k.grad, dk) and torch.equal(v.grad, dv)
    assert (q.grad.float() - dq.float()).abs().max() <= 1e-2 * dq.float().abs().max()
    # two packed sequences, the second behind a prefix
    nq, nk = [200, 100], [200, 700]
    qp = torch.cat([w["q"][:, :200], w["q"][:, 800:900]], dim=1).contiguous().cuda().requires_grad_(True)
    kp = torch.cat([w["k"][:, :200], w["k"][:, 200:900]], dim=1).contiguous().cuda().requires_grad_(True)
    vp = torch.cat([w["v"][:, :200], w["v"][:, 200:900]], dim=1).contiguous().cuda().requires_grad_(True)
    dop = torch.cat([w["do"][:, :200], w["do"][:, 800:900]], dim=1).contiguous().cuda()
    cq = torch.tensor([0, 200, 300], dtype=torch.int32, device="cuda")
    ck = torch.tensor([0, 200, 900], dtype=torch.int32, device="cuda")
    op = mala_attention_packed(qp, kp, vp, cq, ck, max(nq), max(nk), tau, scale=w["scale"])
    op.backward(dop)
    for b in range(2):
        qs = qp.detach()[:, int(cq[b]):int(cq[b + 1])].contiguous()
        ks, vs = (t.detach()[:, int(ck[b]):int(ck[b + 1])].contiguous() for t in (kp, vp))
        o1, l1, _ = mala.fwd_chunk(qs, ks, vs, w["scale"], tau)
        g = mala.bwd_chunk(qs, ks, vs, o1, dop[:, int(cq[b]):int(cq[b + 1])].contiguous(), l1, w["scale"], tau)
        assert torch.equal(o1, op.detach()[:, int(cq[b]):int(cq[b + 1])])
        assert torch.equal(g[1], kp.grad[:, int(ck[b]):int(ck[b + 1])]) and torch.equal(g[2], vp.grad[:, int(ck[b]):int(ck[b + 1])])
        assert (g[0].float() - qp.grad[:, int(cq[b]):int(cq[b + 1])].float()).abs().max() <= 1e-2 * g[0].float().abs().max()
    assert mala.device_status() == 0


def test_an_expired_device_wait_is_reported_and_later_launches_do_nothing_until_cleared(mala, oracle):
    """The time-out path of the kernels' bounded waits, made to run out in the one harmless way: a single small block
    waits (with a short limit) on a barrier nobody arrives on and gives up.  Nothing faults, traps or hangs."""
    w = W.custom_prefill(1, 2, 1, 256, 128, seed=4, preset="R")
    q, k, v = (w[x].cuda() for x in ("q", "k", "v"))
    assert mala.device_status() == 0
    try:
        mala.test_expire_wait(100000)
        torch.cuda.synchronize()
        assert mala.device_status(clear=False) == -8                    # MALA_ERR_DEVICE_TIMEOUT, sticky
        assert mala.lib().mala_strerror(-8).decode() == "bounded device-side wait expired"
        # a launch while the word is set returns at once and leaves its outputs alone
        o = torch.full_like(q, 7.0)
        lse = torch.full((1, 2, 256), 7.0, dtype=torch.float32, device="cuda")
        mala.fwd(q, k, v, w["scale"], 1e-4, out=o, lse=lse)
        torch.cuda.synchronize()
        assert (o == 7.0).all() and (lse == 7.0).all()
        assert mala.device_status(clear=False) == -8
    finally:
        mala.device_status(clear=True)                                   # read and clear
    assert mala.device_status() == 0
    # ... and afterwards the same call computes the right result
    o, lse, _ = mala.fwd(q, k, v, w["scale"], 1e-4)
    torch.cuda.synchronize()
    ref = oracle.fwd(w["q"], w["k"], w["v"], w["scale"], 1e-4, 128, 128)
    parity.check_output(o.float().cpu().numpy(), ref["o"])
    assert np.abs(lse.cpu().numpy() - ref["lse"]).max() <= parity.LSE_ABS
    with pytest.raises(mala.MalaError):
        mala.test_expire_wait(0)


def test_debug_mode_reports_errors_from_the_call_itself():
    """MALA_DEBUG=1 (with MALA_NVTX=1 alongside): a call waits for its stream and returns a recorded device time-out
    itself.  Run in a child process, since the variables are read once per process.  The time-out is the bounded wait
    that nothing satisfies (mala_test_expire_wait), not a fault."""
    import os, subprocess, sys, textwrap
    code = textwrap.dedent("""
        import torch
        from paper_2609_32712_b200 import mala, workloads as W
        w = W.custom_decode(1, 4, 1, 1024, 128, 2, seed=1, device="cuda")
        o, lse, _ = mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], 1e-4, 2)      # fine: returns 0
        p = W.custom_prefill(1, 2, 1, 256, 64, seed=2, device="cuda")
        mala.fwd(p["q"], p["k"], p["v"], p["scale"], 1e-4)
        assert mala.lib().mala_test_expire_wait(20000, None) == 0                              # sets the status word
        try:
            mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], 1e-4, 2)
            print("NO ERROR")
        except mala.MalaError as e:
            print("CODE", e.code)
        assert mala.device_status(clear=True) == -8
        o2, lse2, _ = mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], 1e-4, 2)    # recovered
        assert torch.equal(o, o2) and torch.equal(lse, lse2)
        print("DONE")
    """)
    env = dict(os.environ, MALA_DEBUG="1", MALA_NVTX="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", code], env=env, cwd=root, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    assert "CODE -8" in r.stdout and "DONE" in r.stdout, r.stdout + r.stderr[-1000:]
    assert "[mala debug] mala_decode: device status" in r.stderr
