"""Pins of the fp64 oracle against things other than itself (CPU only).

Each test states what fixes the expected value: the paper's equations re-stated independently
(explicit key sets and direct sums, ratio form of Eq. 2), textbook softmax, finite differences,
closed forms, Proposition 1, the nesting property, special cases that reduce to dense attention.
"""
import math

import numpy as np
import pytest

from oracle import mala_oracle as orc


def _rng(seed):
    return np.random.default_rng(seed)


def peaky_inputs(N, d, seed, Hq=1, Hkv=1, B=1, boost=4.0, retrieval=True):
    """Random heads with a strong self key (and a few far retrieval keys) so that tiles do get skipped."""
    r = _rng(seed)
    q = r.standard_normal((B, N, Hq, d))
    k = r.standard_normal((B, N, Hkv, d))
    v = r.standard_normal((B, N, Hkv, d))
    k *= math.sqrt(d) / np.linalg.norm(k, axis=-1, keepdims=True)
    G = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            q[b, :, h] += boost * k[b, :, h // G]
            if retrieval:
                for i in range(8, N, 23):
                    j = int(r.integers(0, i))
                    q[b, i, h] += boost * k[b, j, h // G]
    return q, k, v


# ------------------------------------------------------------------------------------------------
# independent restatements used as pins
# ------------------------------------------------------------------------------------------------
def textbook_attention(Q, K, V, scale):
    N = Q.shape[0]
    O = np.zeros_like(V[:N])
    lse = np.zeros(N)
    for q in range(N):
        e = np.array([math.exp(scale * float(Q[q] @ K[k])) for k in range(q + 1)])
        p = e / e.sum()
        O[q] = sum(p[k] * V[k] for k in range(q + 1))
        lse[q] = math.log(e.sum())
    return O, lse


def brute_mala_fwd(Q, K, V, scale, tau, Bq, Bk):
    """Eqs. 1-2 with explicit retained key sets and direct summation; ratio form of the test."""
    N = Q.shape[0]
    S = scale * (Q @ K.T)
    Tr, Tc = -(-N // Bq), -(-N // Bk)
    mask = np.zeros((Tr, Tc), dtype=np.uint8)
    O = np.zeros((N, V.shape[1]))
    lse = np.zeros(N)
    for i in range(Tr):
        rows = list(range(i * Bq, min(N, (i + 1) * Bq)))
        R = {q: [] for q in rows}
        for j in reversed(range(Tc)):
            keys = list(range(j * Bk, min(N, (j + 1) * Bk)))
            if keys[0] > rows[-1]:
                continue
            skip = True
            for q in rows:
                legal = [k for k in keys if k <= q]
                if not legal:
                    continue                      # row does not constrain the tile
                Zt = sum(math.exp(S[q, k]) for k in R[q])
                if Zt == 0.0:
                    skip = False                  # first legal tile of a row is always kept
                    continue
                ratio = math.exp(max(S[q, k] for k in legal)) / Zt
                if not (ratio < tau / (q + 1)):
                    skip = False
            mask[i, j] = 1 if skip else 2
            if not skip:
                for q in rows:
                    R[q] += [k for k in keys if k <= q]
        for q in rows:
            Z = sum(math.exp(S[q, k]) for k in R[q])
            O[q] = sum(math.exp(S[q, k]) / Z * V[k] for k in R[q])
            lse[q] = math.log(Z)
    return O, lse, mask


def brute_mala_bwd(Q, K, V, dO, O, lse, scale, tau, Bq, Bk, shift=0):
    """Eq. 4 per tile with the saved lse, then the attention-backward equations restricted to the
    retained tiles, written with whole-matrix products.  The queries are the last rows of the keys' positions;
    query block i holds the rows q with i*Bq <= q + shift < (i+1)*Bq."""
    N, Nk = Q.shape[0], K.shape[0]
    off = Nk - N
    S = scale * (Q @ K.T)                                       # [q, k]
    Tr, Tc = -(-(N + shift) // Bq), -(-Nk // Bk)
    mask = np.zeros((Tc, Tr), dtype=np.uint8)
    keep = np.zeros((N, Nk), dtype=bool)
    for j in range(Tc):
        for i in range(Tr):
            qs = range(max(0, i * Bq - shift), min(N, (i + 1) * Bq - shift))
            ks = range(j * Bk, min(Nk, (j + 1) * Bk))
            ent = [(q, k) for q in qs for k in ks if k <= q + off]
            if not ent:
                continue
            skip = all(math.exp(S[q, k] - lse[q]) < tau / (q + 1 + off) for (q, k) in ent)
            mask[j, i] = 1 if skip else 2
            if not skip:
                for (q, k) in ent:
                    keep[q, k] = True
    P = np.where(keep, np.exp(S - lse[:, None]), 0.0)
    D = (O * dO).sum(axis=1)
    dP = dO @ V.T
    dS = P * (dP - D[:, None])
    return scale * dS @ K, scale * dS.T @ Q, P.T @ dO, mask


# ------------------------------------------------------------------------------------------------
# FullAttn (tau = 0)
# ------------------------------------------------------------------------------------------------
def test_dense_fwd_is_textbook_softmax():
    q, k, v = peaky_inputs(37, 8, 1, boost=0.5)
    o, lse = orc.dense_fwd(q, k, v, 0.3)
    O, L = textbook_attention(q[0, :, 0], k[0, :, 0], v[0, :, 0], 0.3)
    assert np.allclose(o[0, :, 0], O, rtol=0, atol=1e-12)
    assert np.allclose(lse[0, 0], L, rtol=0, atol=1e-12)


def test_dense_bwd_matches_finite_differences():
    N, d, scale = 12, 4, 0.7
    q, k, v = peaky_inputs(N, d, 2, boost=0.3)
    do = _rng(3).standard_normal((1, N, 1, d))
    dq, dk, dv = orc.dense_bwd(q, k, v, do, scale)

    def loss(qq, kk, vv):
        o, _ = orc.dense_fwd(qq, kk, vv, scale)
        return float((o * do).sum())

    eps = 1e-6
    for (x, g, name) in ((q, dq, "dq"), (k, dk, "dk"), (v, dv, "dv")):
        num = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps
            xm[idx] -= eps
            args_p = [q, k, v]
            args_m = [q, k, v]
            pos = {"dq": 0, "dk": 1, "dv": 2}[name]
            args_p[pos], args_m[pos] = xp, xm
            num[idx] = (loss(*args_p) - loss(*args_m)) / (2 * eps)
        assert np.linalg.norm(num - g) <= 1e-6 * max(1.0, np.linalg.norm(g)), name


def test_dense_bwd_gqa_sums_group_heads():
    q, k, v = peaky_inputs(16, 4, 4, Hq=4, Hkv=2, boost=0.3)
    do = _rng(5).standard_normal(q.shape)
    dq, dk, dv = orc.dense_bwd(q, k, v, do, 0.5)
    for g in range(2):
        acc_k = np.zeros((16, 4))
        acc_v = np.zeros((16, 4))
        for h in (2 * g, 2 * g + 1):
            a, c, e = orc.dense_bwd(q[:, :, h:h + 1], k[:, :, g:g + 1], v[:, :, g:g + 1], do[:, :, h:h + 1], 0.5)
            assert np.allclose(dq[0, :, h], a[0, :, 0], atol=1e-13)
            acc_k += c[0, :, 0]
            acc_v += e[0, :, 0]
        assert np.allclose(dk[0, :, g], acc_k, atol=1e-12)
        assert np.allclose(dv[0, :, g], acc_v, atol=1e-12)


@pytest.mark.parametrize("N,Bq,Bk", [(64, 8, 8), (50, 8, 8), (50, 16, 4), (33, 4, 16), (20, 32, 32)])
def test_tau_zero_recovers_fullattn(N, Bq, Bk):
    d, scale = 8, 0.35
    q, k, v = peaky_inputs(N, d, 6, Hq=2, Hkv=1)
    do = _rng(7).standard_normal(q.shape)
    o_d, lse_d = orc.dense_fwd(q, k, v, scale)
    f = orc.fwd(q, k, v, scale, 0.0, Bq, Bk)
    assert np.allclose(f["o"], o_d, atol=1e-12) and np.allclose(f["lse"], lse_d, atol=1e-12)
    assert not (f["mask"] == orc.SKIPPED).any()
    dq_d, dk_d, dv_d = orc.dense_bwd(q, k, v, do, scale)
    g = orc.bwd(q, k, v, f["o"], do, f["lse"], scale, 0.0, Bq, Bk)
    for a, b_ in ((g["dq"], dq_d), (g["dk"], dk_d), (g["dv"], dv_d)):
        assert np.allclose(a, b_, atol=1e-10)
    assert not (g["mask"] == orc.SKIPPED).any()


# ------------------------------------------------------------------------------------------------
# the online rule (Eqs. 1-3, Algorithm 1)
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,Bq,Bk,tau", [(64, 8, 8, 1e-2), (61, 8, 8, 1e-1), (48, 16, 4, 1e-2), (40, 4, 8, 1.0),
                                         (24, 1, 1, 1e-1)])
def test_fwd_matches_bruteforce_key_sets(N, Bq, Bk, tau):
    d, scale = 32, 1.0 / math.sqrt(32)
    q, k, v = peaky_inputs(N, d, 11 + N, boost=5.0)
    f = orc.fwd(q, k, v, scale, tau, Bq, Bk)
    O, L, M = brute_mala_fwd(q[0, :, 0], k[0, :, 0], v[0, :, 0], scale, tau, Bq, Bk)
    assert (np.abs(f["crit"][np.isfinite(f["crit"])]) > 1e-9).all()
    assert (f["mask"][0, 0] == M).all()
    assert (M == 1).sum() > 0, "workload must exercise skipping"
    assert np.allclose(f["o"][0, :, 0], O, atol=1e-11) and np.allclose(f["lse"][0, 0], L, atol=1e-11)


def test_fwd_bq_larger_than_bk_rows_without_legal_keys_do_not_constrain():
    # with B_q = 16, B_k = 4 the first tiles visited have no legal key for the early rows of a block
    N, d, scale, tau = 32, 4, 0.5, 1e-1
    q, k, v = peaky_inputs(N, d, 21, boost=6.0)
    f = orc.fwd(q, k, v, scale, tau, 16, 4)
    O, L, M = brute_mala_fwd(q[0, :, 0], k[0, :, 0], v[0, :, 0], scale, tau, 16, 4)
    assert (f["mask"][0, 0] == M).all() and np.isfinite(f["lse"]).all()
    assert np.allclose(f["o"][0, :, 0], O, atol=1e-11)


def test_fwd_first_tile_retained_rows_nonempty_and_illegal_tiles_uncounted():
    q, k, v = peaky_inputs(96, 8, 31, Hq=2, Hkv=2, boost=6.0)
    f = orc.fwd(q, k, v, 0.35, 1.0, 8, 8)
    m = f["mask"]
    for i in range(12):
        assert (m[:, :, i, i] == orc.RETAINED).all()
        assert (m[:, :, i, i + 1:] == orc.ILLEGAL).all()
        assert (m[:, :, i, :i + 1] != orc.ILLEGAL).all()
    assert np.isfinite(f["lse"]).all() and np.isfinite(f["o"]).all()
    assert np.isnan(f["crit"][m == orc.ILLEGAL]).all()


@pytest.mark.parametrize("tau", [1e-3, 1e-1, 1.0, 4.0])
def test_proposition1_omitted_mass_and_output_bounds(tau):
    N, d, scale = 128, 32, 1.0 / math.sqrt(32)
    q, k, v = peaky_inputs(N, d, 41, Hq=2, Hkv=1, boost=4.0)
    o_d, lse_d = orc.dense_fwd(q, k, v, scale)
    f = orc.fwd(q, k, v, scale, tau, 8, 8)
    eps = 1.0 - np.exp(f["lse"] - lse_d)                       # omitted mass from the two normalizers
    assert (eps >= -1e-12).all() and (eps <= tau / (1 + tau) + 1e-12).all()
    vmax = np.linalg.norm(v, axis=-1).max()
    err = np.linalg.norm(f["o"] - o_d, axis=-1)
    assert (err <= 2 * tau / (1 + tau) * vmax + 1e-12).all()
    if tau >= 1e-1:
        assert (f["mask"] == orc.SKIPPED).sum() > 0


def test_closed_form_zero_queries_uniform_rows():
    N, d = 40, 4
    r = _rng(51)
    q = np.zeros((1, N, 1, d))
    k, v = r.standard_normal((1, N, 1, d)), r.standard_normal((1, N, 1, d))
    for tau in (1e-3, 1.0):
        f = orc.fwd(q, k, v, 0.5, tau, 8, 8)
        assert not (f["mask"] == orc.SKIPPED).any()            # ratio 1/Z_t >= 1/L_q >= tau/L_q
        mean = np.cumsum(v[0, :, 0], axis=0) / np.arange(1, N + 1)[:, None]
        assert np.allclose(f["o"][0, :, 0], mean, atol=1e-13)
        assert np.allclose(f["lse"][0, 0], np.log(np.arange(1, N + 1)), atol=1e-13)


def _one_hot_case(N, C):
    q = np.zeros((1, N, 1, N))
    k = np.zeros((1, N, 1, N))
    for t in range(N):
        q[0, t, 0, t] = C
        k[0, t, 0, t] = 1.0
    v = _rng(61).standard_normal((1, N, 1, 3))
    return q, k, np.concatenate([v, np.zeros((1, N, 1, N - 3))], axis=-1)


def _one_hot_expected_mask(N, B, C, tau):
    T = N // B
    m = np.zeros((T, T), dtype=np.uint8)
    for i in range(T):
        Z = [math.exp(C) + r for r in range(B)]                # after the diagonal tile: self key + r zeros
        m[i, i] = 2
        for j in range(i - 1, -1, -1):
            skip = all(1.0 / Z[r] < tau / (i * B + r + 1) for r in range(B))
            m[i, j] = 1 if skip else 2
            if not skip:
                Z = [z + B for z in Z]
    return m


@pytest.mark.parametrize("C", [3.0, 7.0, 8.0, 10.0])
def test_closed_form_one_boosted_key_per_row(C):
    N, B, tau = 64, 8, 1e-2
    q, k, v = _one_hot_case(N, C)
    f = orc.fwd(q, k, v, 1.0, tau, B, B)
    assert (f["mask"][0, 0] == _one_hot_expected_mask(N, B, C, tau)).all()


def test_closed_form_threshold_crossing_at_predicted_boost():
    # block 1 (rows 8..15), tile (1,0): the binding row is the last one, r = 7, L = 16:
    # skipped iff 1/(e^C + 7) < tau/16  <=>  C > log(16/tau - 7)
    N, B, tau = 64, 8, 1e-2
    Cstar = math.log(16 / tau - 7)
    for C, expect in ((Cstar - 1e-6, orc.RETAINED), (Cstar + 1e-6, orc.SKIPPED)):
        q, k, v = _one_hot_case(N, C)
        f = orc.fwd(q, k, v, 1.0, tau, B, B, units=[(0, 0, 1)])
        assert f["mask"][0, 0, 1, 0] == expect
        assert abs(f["crit"][0, 0, 1, 0]) < 1e-5


def test_single_tile_is_dense_for_any_tau():
    q, k, v = peaky_inputs(30, 8, 71, boost=6.0)
    o_d, lse_d = orc.dense_fwd(q, k, v, 0.4)
    f = orc.fwd(q, k, v, 0.4, 10.0, 32, 32)
    assert np.allclose(f["o"], o_d, atol=1e-12) and np.allclose(f["lse"], lse_d, atol=1e-12)


def test_per_element_rule_when_tiles_are_single_entries():
    N, d, scale, tau = 20, 4, 0.5, 0.3
    q, k, v = peaky_inputs(N, d, 81, boost=4.0)
    f = orc.fwd(q, k, v, scale, tau, 1, 1)
    S = scale * q[0, :, 0] @ k[0, :, 0].T
    for i in range(N):
        Z = 0.0
        for j in range(i, -1, -1):
            keep = (Z == 0.0) or not (math.exp(S[i, j]) / Z < tau / (i + 1))
            assert f["mask"][0, 0, i, j] == (2 if keep else 1)
            if keep:
                Z += math.exp(S[i, j])
        assert abs(f["lse"][0, 0, i] - math.log(Z)) < 1e-12


def test_tau_monotonicity_of_forward_support():
    # if tau1 (1 + tau2) <= tau2 the support under tau1 contains the support under tau2
    q, k, v = peaky_inputs(128, 32, 91, boost=6.0)
    taus = [0.0, 1e-5, 1e-4, 1e-3, 1e-1]
    masks = [orc.fwd(q, k, v, 1.0 / math.sqrt(32), t, 8, 8)["mask"] for t in taus]
    for a, b_ in zip(masks[:-1], masks[1:]):
        assert ((b_ == orc.RETAINED) <= (a == orc.RETAINED)).all()
    assert (masks[-1] == orc.SKIPPED).sum() > (masks[1] == orc.SKIPPED).sum()


def test_fwd_units_select_blocks_and_match_full_run():
    q, k, v = peaky_inputs(70, 8, 101, Hq=2, Hkv=1, boost=5.0)
    full = orc.fwd(q, k, v, 0.35, 1e-1, 8, 8)
    part = orc.fwd(q, k, v, 0.35, 1e-1, 8, 8, units=[(0, 1, 3), (0, 1, 8)])
    for i in (3, 8):
        rows = slice(i * 8, min(70, i * 8 + 8))
        assert np.array_equal(part["o"][0, rows, 1], full["o"][0, rows, 1])
        assert np.array_equal(part["mask"][0, 1, i], full["mask"][0, 1, i])
    assert np.isnan(part["o"][0, :, 0]).all() and np.isnan(part["o"][0, 0:24, 1]).all()


# ------------------------------------------------------------------------------------------------
# the offline rule (Eq. 4, Algorithm 2)
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,Bq,Bk,tau", [(64, 8, 8, 1e-2), (61, 8, 8, 1e-1), (48, 4, 8, 1.0), (48, 16, 4, 1e-1)])
def test_bwd_matches_bruteforce_and_is_nested(N, Bq, Bk, tau):
    d, scale = 32, 1.0 / math.sqrt(32)
    q, k, v = peaky_inputs(N, d, 111 + N, boost=5.0)
    do = _rng(112).standard_normal(q.shape)
    f = orc.fwd(q, k, v, scale, tau, Bq, Bk)
    g = orc.bwd(q, k, v, f["o"], do, f["lse"], scale, tau, Bq, Bk)
    dQ, dK, dV, M = brute_mala_bwd(q[0, :, 0], k[0, :, 0], v[0, :, 0], do[0, :, 0], f["o"][0, :, 0], f["lse"][0, 0],
                                   scale, tau, Bq, Bk)
    assert (g["mask"][0, 0] == M).all()
    assert np.allclose(g["dq"][0, :, 0], dQ, atol=1e-11)
    assert np.allclose(g["dk"][0, :, 0], dK, atol=1e-11)
    assert np.allclose(g["dv"][0, :, 0], dV, atol=1e-11)
    # nesting: every tile kept by backward was kept by forward (same partition), none stored
    fm = f["mask"][0, 0]
    bm = g["mask"][0, 0].T
    assert ((bm == orc.RETAINED) <= (fm == orc.RETAINED)).all()
    assert ((bm == orc.ILLEGAL) == (fm == orc.ILLEGAL)).all()
    assert (bm == orc.SKIPPED).sum() >= (fm == orc.SKIPPED).sum() > 0


def test_bwd_may_skip_the_diagonal_tile():
    # rows whose mass sits on one far key: the diagonal tile falls below tau/L under the final normalizer
    N, B, d = 32, 8, 32
    r = _rng(121)
    k = np.zeros((1, N, 1, d))
    for t in range(N):
        k[0, t, 0, t] = 1.0
    q = np.zeros((1, N, 1, d))
    q[0, :, 0, 0] = 30.0                                        # every query points at key 0
    v = r.standard_normal((1, N, 1, d))
    do = r.standard_normal((1, N, 1, d))
    f = orc.fwd(q, k, v, 1.0, 1e-2, B, B)
    g = orc.bwd(q, k, v, f["o"], do, f["lse"], 1.0, 1e-2, B, B)
    assert (f["mask"][0, 0].diagonal() == orc.RETAINED).all()
    assert (g["mask"][0, 0].diagonal()[1:] == orc.SKIPPED).all()
    assert (g["mask"][0, 0, 0, :] == orc.RETAINED).all()


def test_bwd_key_units_and_dq_units_match_full_run():
    N, Bq, Bk, d, scale, tau = 72, 8, 8, 8, 0.35, 1e-1
    q, k, v = peaky_inputs(N, d, 131, Hq=4, Hkv=2, boost=5.0)
    do = _rng(132).standard_normal(q.shape)
    f = orc.fwd(q, k, v, scale, tau, Bq, Bk)
    full = orc.bwd(q, k, v, f["o"], do, f["lse"], scale, tau, Bq, Bk)
    part = orc.bwd(q, k, v, f["o"], do, f["lse"], scale, tau, Bq, Bk, key_units=[(0, 1, 2), (0, 0, 8)],
                   dq_units=[(0, 3, 5)])
    assert np.allclose(part["dk"][0, 16:24, 1], full["dk"][0, 16:24, 1], atol=1e-12)
    assert np.allclose(part["dv"][0, 64:72, 0], full["dv"][0, 64:72, 0], atol=1e-12)
    assert np.allclose(part["dq"][0, 40:48, 3], full["dq"][0, 40:48, 3], atol=1e-12)
    assert np.array_equal(part["mask"][0, 2:4, 2], full["mask"][0, 2:4, 2])
    assert np.isnan(part["dk"][0, 0:8, 1]).all()


# ------------------------------------------------------------------------------------------------
# split-KV decode
# ------------------------------------------------------------------------------------------------
def _decode_inputs(Nk, d, G, seed, gate=True):
    r = _rng(seed)
    q = r.standard_normal((1, G, d))
    kc = r.standard_normal((1, Nk, 1, d))
    vc = r.standard_normal((1, Nk, 1, d))
    if gate:                                                    # most keys far below a few live ones
        live = r.random(Nk) < 0.1
        live[-4:] = True
        kc[0, :, 0, d - 1] = np.where(live, 0.0, -6.0)
        q[0, :, d - 1] = 6.0
    return q, kc, vc


@pytest.mark.parametrize("S", [1, 3, 8])
def test_decode_tau_zero_any_split_count_is_dense(S):
    q, kc, vc = _decode_inputs(100, 8, 4, 141)
    dec = orc.decode(q, kc, vc, 0.4, 0.0, S, 8)
    for h in range(4):
        e = np.exp(0.4 * kc[0, :, 0] @ q[0, h])
        assert np.allclose(dec["o"][0, h], (e / e.sum()) @ vc[0, :, 0], atol=1e-12)
        assert abs(dec["lse"][0, h] - math.log(e.sum())) < 1e-12
    assert not (dec["mask"] == orc.SKIPPED).any()


@pytest.mark.parametrize("packed", [True, False])
def test_decode_rule_bruteforce_per_split_and_mass_bound(packed):
    Nk, d, G, S, Bk, scale, tau = 96, 8, 4, 3, 8, 0.5, 0.5
    q, kc, vc = _decode_inputs(Nk, d, G, 151)
    dec = orc.decode(q, kc, vc, scale, tau, S, Bk, packed_rows=packed)
    sc = scale * kc[0, :, 0] @ q[0].T                            # [Nk, G]
    chunk = 32
    row_sets = [list(range(G))] if packed else [[h] for h in range(G)]
    assert (dec["mask"] == orc.SKIPPED).sum() > 0
    for ri, hs in enumerate(row_sets):
        for s in range(S):
            kept = []
            for t in reversed(range(chunk // Bk)):
                keys = list(range(s * chunk + t * Bk, s * chunk + (t + 1) * Bk))
                skip = True
                for h in hs:
                    Z = sum(math.exp(sc[k_, h]) for k_ in kept)
                    if Z == 0.0 or not (math.exp(max(sc[k_, h] for k_ in keys)) / Z < tau / Nk):
                        skip = False
                assert dec["mask"][0, ri, s, t] == (1 if skip else 2)
                if not skip:
                    kept += keys
            for h in hs:
                Z = sum(math.exp(sc[k_, h]) for k_ in kept)
                assert abs(dec["lse_part"][0, h, s] - math.log(Z)) < 1e-12
    # Proposition 1 carries over to the merged result (each omitted key is below tau/L of a partial Z)
    for h in range(G):
        lse_d = math.log(np.exp(sc[:, h]).sum())
        eps = 1.0 - math.exp(dec["lse"][0, h] - lse_d)
        assert -1e-12 <= eps <= tau / (1 + tau) + 1e-12


def test_decode_merge_is_logsumexp_weighted_mean():
    r = _rng(161)
    op = r.standard_normal((1, 2, 5, 3))
    lp = r.standard_normal((1, 2, 5))
    L = orc.lib()
    import ctypes
    for h in range(2):
        o = np.zeros((1, 3))
        l = np.zeros((1,))
        a = np.ascontiguousarray(op[0, h][:, None, :])
        b_ = np.ascontiguousarray(lp[0, h][:, None])
        L.mala_oracle_decode_merge(a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                   b_.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), 5, 1, 3,
                                   o.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                   l.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
        w = np.exp(lp[0, h])
        assert np.allclose(o[0], (w / w.sum()) @ op[0, h], atol=1e-13)
        assert abs(l[0] - math.log(w.sum())) < 1e-13


def test_decode_ragged_cache_and_empty_trailing_split():
    q, kc, vc = _decode_inputs(70, 8, 2, 171, gate=False)
    dec = orc.decode(q, kc, vc, 0.4, 0.0, 5, 16)                 # chunk = 16, 5 splits cover 80 > 70 keys
    assert np.isneginf(dec["lse_part"]).sum() == 0                # 70 keys -> split 4 holds keys 64..69
    dec2 = orc.decode(q, kc, vc, 0.4, 0.0, 8, 16)                # chunk = 16, splits 5..7 are empty
    assert np.isneginf(dec2["lse_part"][0, :, 5:]).all()
    assert np.allclose(dec["o"], dec2["o"], atol=1e-13)


# ------------------------------------------------------------------ paged cache, one length per sequence
def _paged_inputs(B, Nmax, d, G, page, lens, seed):
    """Contiguous caches of B sequences cut into pages that are scattered over a shuffled pool; slots that no
    sequence uses hold large finite junk."""
    r = _rng(seed)
    q = r.standard_normal((B, G, d))
    kc = r.standard_normal((B, Nmax, 1, d))
    vc = r.standard_normal((B, Nmax, 1, d))
    live = r.random((B, Nmax)) < 0.1
    kc[:, :, 0, d - 1] = np.where(live, 0.0, -6.0)
    q[:, :, d - 1] = 6.0
    mp = Nmax // page
    pool = B * mp + 3
    perm = r.permutation(pool)
    kp = 50.0 * r.standard_normal((pool, page, 1, d))
    vp = 50.0 * r.standard_normal((pool, page, 1, d))
    bt = np.full((B, mp), pool + 5, dtype=np.int64)             # unused entries point outside the pool
    for b in range(B):
        for x in range(-(-lens[b] // page)):
            n = min(page, lens[b] - x * page)
            bt[b, x] = perm[b * mp + x]
            kp[bt[b, x], :n] = kc[b, x * page:x * page + n]
            vp[bt[b, x], :n] = vc[b, x * page:x * page + n]
    return q, kc, vc, kp, vp, bt


def test_decode_paged_tau_zero_is_softmax_over_each_sequences_own_keys():
    lens = [64, 37, 5, 0]
    q, kc, vc, kp, vp, bt = _paged_inputs(4, 64, 8, 2, 16, lens, 181)
    dec = orc.decode_paged(q, kp, vp, bt, lens, 0.4, 0.0, 4, 8)
    for b, n in enumerate(lens):
        for h in range(2):
            if n == 0:
                assert (dec["o"][b, h] == 0).all() and np.isneginf(dec["lse"][b, h])
                continue
            e = np.exp(0.4 * kc[b, :n, 0] @ q[b, h])
            assert np.allclose(dec["o"][b, h], (e / e.sum()) @ vc[b, :n, 0], atol=1e-12)
            assert abs(dec["lse"][b, h] - math.log(e.sum())) < 1e-12
    assert np.isneginf(dec["lse_part"][2, :, 1:]).all()            # 5 keys: only the first 16-key split is used


@pytest.mark.parametrize("tau", [0.5, 1e-2])
def test_decode_paged_equals_contiguous_rule_per_sequence(tau):
    # 128 positions, 4 splits of 32 keys; a sequence of n keys must behave like a contiguous cache of n keys cut
    # into the same 32-key chunks (L = n), wherever its pages lie in the pool
    lens = [128, 96, 64, 51]
    q, kc, vc, kp, vp, bt = _paged_inputs(4, 128, 8, 4, 16, lens, 191)
    dec = orc.decode_paged(q, kp, vp, bt, lens, 0.5, tau, 4, 8)
    assert (dec["mask"] == orc.SKIPPED).sum() > 0
    for b, n in enumerate(lens):
        S = -(-n // 32)
        ref = orc.decode(q[b:b + 1], kc[b:b + 1, :n], vc[b:b + 1, :n], 0.5, tau, S, 8)
        assert orc.lib().mala_oracle_decode_tiles_per_split(n, S, 8) == 4
        assert np.array_equal(dec["mask"][b, :, :S], ref["mask"][0])
        assert np.allclose(dec["lse_part"][b, :, :S], ref["lse_part"][0], atol=1e-13)
        assert np.allclose(dec["o"][b], ref["o"][0], atol=1e-13)
        assert np.allclose(dec["lse"][b], ref["lse"][0], atol=1e-13)
        assert (dec["mask"][b, :, S:] == 0).all()


def test_decode_paged_does_not_depend_on_where_pages_lie():
    lens = [80, 33]
    q, kc, vc, kp, vp, bt = _paged_inputs(2, 96, 8, 2, 16, lens, 201)
    a = orc.decode_paged(q, kp, vp, bt, lens, 0.5, 0.3, 3, 8)
    # the same sequences in an orderly pool: sequence b, page x -> pool page b * 6 + x
    kp2 = np.zeros((12, 16, 1, 8))
    vp2 = np.zeros((12, 16, 1, 8))
    bt2 = np.arange(12).reshape(2, 6)
    for b in range(2):
        kp2[b * 6:(b + 1) * 6] = kc[b].reshape(6, 16, 1, 8)
        vp2[b * 6:(b + 1) * 6] = vc[b].reshape(6, 16, 1, 8)
    c = orc.decode_paged(q, kp2, vp2, bt2, lens, 0.5, 0.3, 3, 8)
    for key in ("o", "lse", "mask", "lse_part"):
        assert np.array_equal(a[key], c[key])


# ------------------------------------------------------------------ fewer queries than keys (chunked prefill)
@pytest.mark.parametrize("Nq,Nk,Bq,Bk", [(24, 64, 8, 8), (13, 50, 8, 8), (16, 48, 16, 4)])
def test_chunk_tau_zero_is_softmax_over_the_visible_keys(Nq, Nk, Bq, Bk):
    # the queries are the last Nq positions: row q attends to the keys 0 .. q + Nk - Nq, nothing else
    d, scale = 8, 0.4
    q, k, v = peaky_inputs(Nk, d, 211)
    qc = q[:, Nk - Nq:]
    f = orc.fwd(qc, k, v, scale, 0.0, Bq, Bk)
    for r in range(Nq):
        vis = r + 1 + Nk - Nq
        e = np.exp(scale * k[0, :vis, 0] @ qc[0, r, 0])
        assert np.allclose(f["o"][0, r, 0], (e / e.sum()) @ v[0, :vis, 0], atol=1e-12)
        assert abs(f["lse"][0, 0, r] - math.log(e.sum())) < 1e-12
    od, ld = orc.dense_fwd(qc, k, v, scale)
    assert np.allclose(od, f["o"], atol=1e-12) and np.allclose(ld, f["lse"], atol=1e-12)


@pytest.mark.parametrize("tau", [1e-2, 0.5])
@pytest.mark.parametrize("Nq,Nk,Bq,Bk", [(32, 96, 8, 8), (21, 69, 8, 8), (32, 64, 16, 4)])
def test_chunk_equals_the_same_rows_of_the_full_run(Nq, Nk, Bq, Bk, tau):
    # a query block's result depends on its own rows and the keys only, so when the chunk starts on a block
    # boundary the chunked run must reproduce the last rows of the equal-length run: masks, O, lse and gradients
    d, scale = 32, 1.0 / math.sqrt(32)
    off = Nk - Nq
    assert off % Bq == 0
    q, k, v = peaky_inputs(Nk, d, 221, Hq=2, Hkv=1, boost=5.0)
    do = _rng(223).standard_normal(q.shape)
    full = orc.fwd(q, k, v, scale, tau, Bq, Bk)
    ch = orc.fwd(q[:, off:], k, v, scale, tau, Bq, Bk)
    assert (ch["mask"] == orc.SKIPPED).sum() > 0
    assert np.array_equal(ch["mask"], full["mask"][:, :, off // Bq:])
    assert np.array_equal(ch["o"], full["o"][:, off:]) and np.array_equal(ch["lse"], full["lse"][:, :, off:])
    # backward: with dO = 0 on the rows before the chunk those rows contribute nothing (dS = P o (0 - 0))
    do0 = do.copy()
    do0[:, :off] = 0.0
    gf = orc.bwd(q, k, v, full["o"], do0, full["lse"], scale, tau, Bq, Bk)
    gc = orc.bwd(q[:, off:], k, v, ch["o"], do[:, off:], ch["lse"], scale, tau, Bq, Bk)
    assert np.array_equal(gc["mask"], gf["mask"][:, :, :, off // Bq:])
    assert np.allclose(gc["dq"], gf["dq"][:, off:], atol=1e-13)
    assert np.allclose(gc["dk"], gf["dk"], atol=1e-13) and np.allclose(gc["dv"], gf["dv"], atol=1e-13)
    assert np.abs(gf["dq"][:, :off]).max() == 0.0
    # sampled dQ blocks follow the same tiles
    gd = orc.bwd(q[:, off:], k, v, ch["o"], do[:, off:], ch["lse"], scale, tau, Bq, Bk, dq_units=[(0, 1, 0), (0, 0, 1)])
    for (h, i) in ((1, 0), (0, 1)):
        rows = slice(i * Bq, min(Nq, (i + 1) * Bq))
        assert np.allclose(gd["dq"][0, rows, h], gc["dq"][0, rows, h], atol=1e-13)


def test_chunk_of_one_query_is_the_unsplit_decode_rule():
    # Nq = 1: the single query sees all Nk keys, L = Nk, tiles visited newest first -- the decode rule with one
    # split and one row
    Nk, d, scale, tau, Bk = 96, 8, 0.5, 0.5, 8
    q, kc, vc = _decode_inputs(Nk, d, 1, 231)
    dec = orc.decode(q, kc, vc, scale, tau, 1, Bk, packed_rows=False)
    f = orc.fwd(q[:, None, :, :].reshape(1, 1, 1, d), kc, vc, scale, tau, 4, Bk)
    assert (dec["mask"] == orc.SKIPPED).sum() > 0
    assert np.array_equal(f["mask"][0, 0, 0], dec["mask"][0, 0, 0])
    assert np.allclose(f["o"][0, 0, 0], dec["o"][0, 0], atol=1e-13)
    assert abs(f["lse"][0, 0, 0] - dec["lse"][0, 0]) < 1e-13


def test_chunk_offset_inside_a_tile_rows_without_legal_keys_do_not_constrain():
    # Nk - Nq not a multiple of the tile: the diagonal crosses two key tiles of a query block; brute force
    Nq, Nk, B_, d, scale, tau = 16, 37, 8, 32, 1.0 / math.sqrt(32), 0.1
    off = Nk - Nq
    q, k, v = peaky_inputs(Nk, d, 241, boost=5.0)
    qc = q[:, off:]
    f = orc.fwd(qc, k, v, scale, tau, B_, B_)
    S = scale * (qc[0, :, 0] @ k[0, :, 0].T)
    for i in range(2):
        rows = list(range(i * B_, (i + 1) * B_))
        R = {r: [] for r in rows}
        for j in reversed(range(-(-Nk // B_))):
            keys = list(range(j * B_, min(Nk, (j + 1) * B_)))
            if keys[0] > rows[-1] + off:
                assert f["mask"][0, 0, i, j] == 0
                continue
            skip = True
            for r in rows:
                legal = [x for x in keys if x <= r + off]
                if not legal:
                    continue
                Z = sum(math.exp(S[r, x]) for x in R[r])
                if Z == 0.0 or not (math.exp(max(S[r, x] for x in legal)) / Z < tau / (r + 1 + off)):
                    skip = False
            assert f["mask"][0, 0, i, j] == (1 if skip else 2)
            if not skip:
                for r in rows:
                    R[r] += [x for x in keys if x <= r + off]
        for r in rows:
            Z = sum(math.exp(S[r, x]) for x in R[r])
            assert abs(f["lse"][0, 0, r] - math.log(Z)) < 1e-12
    assert (f["mask"] == orc.SKIPPED).sum() > 0


# ------------------------------------------------------------------ several new tokens per decode step
def _multi_inputs(Nk, Sq, d, G, seed):
    r = _rng(seed)
    q = r.standard_normal((1, Sq, G, d))
    kc = r.standard_normal((1, Nk, 1, d))
    vc = r.standard_normal((1, Nk, 1, d))
    live = r.random(Nk) < 0.1
    live[-Sq - 2:] = True
    kc[0, :, 0, d - 1] = np.where(live, 0.0, -6.0)
    q[0, :, :, d - 1] = 6.0
    return q, kc, vc


@pytest.mark.parametrize("Nk,Sq", [(100, 4), (97, 3), (64, 1)])
def test_decode_multi_tau_zero_is_softmax_over_each_tokens_visible_keys(Nk, Sq):
    q, kc, vc = _multi_inputs(Nk, Sq, 8, 2, 251)
    dec = orc.decode_multi(q, kc, vc, 0.4, 0.0, 3, 8)
    for s in range(Sq):
        vis = Nk - Sq + s + 1
        for h in range(2):
            e = np.exp(0.4 * kc[0, :vis, 0] @ q[0, s, h])
            assert np.allclose(dec["o"][0, s, h], (e / e.sum()) @ vc[0, :vis, 0], atol=1e-12)
            assert abs(dec["lse"][0, s, h] - math.log(e.sum())) < 1e-12
    if Sq == 1:
        one = orc.decode(q[:, 0], kc, vc, 0.4, 0.0, 3, 8)
        assert np.array_equal(one["o"], dec["o"][:, 0]) and np.array_equal(one["lse"], dec["lse"][:, 0])


@pytest.mark.parametrize("Nk,Sq,G", [(96, 4, 2), (91, 5, 1), (98, 3, 2)])
def test_decode_multi_rule_bruteforce_with_per_row_visible_keys(Nk, Sq, G):
    d, S, Bk, scale, tau = 8, 3, 8, 0.5, 0.5
    q, kc, vc = _multi_inputs(Nk, Sq, d, G, 261 + Nk)
    dec = orc.decode_multi(q, kc, vc, scale, tau, S, Bk)
    tps = dec["mask"].shape[-1]
    chunk = tps * Bk
    rows = [(s, g) for s in range(Sq) for g in range(G)]
    sc = {(s, g): scale * kc[0, :, 0] @ q[0, s, g] for (s, g) in rows}
    assert (dec["mask"] == orc.SKIPPED).sum() > 0
    for sp in range(S):
        kept = {r: [] for r in rows}
        for t in reversed(range(tps)):
            keys = [x for x in range(sp * chunk + t * Bk, sp * chunk + (t + 1) * Bk) if x < Nk]
            if not keys:
                assert dec["mask"][0, 0, sp, t] == 0
                continue
            skip = True
            for (s, g) in rows:
                vis = Nk - Sq + s + 1
                legal = [x for x in keys if x < vis]
                if not legal:
                    continue                          # the row sees no key of the tile: it does not constrain it
                Z = sum(math.exp(sc[(s, g)][x]) for x in kept[(s, g)])
                if Z == 0.0 or not (math.exp(max(sc[(s, g)][x] for x in legal)) / Z < tau / vis):
                    skip = False
            assert dec["mask"][0, 0, sp, t] == (1 if skip else 2)
            if not skip:
                for (s, g) in rows:
                    kept[(s, g)] += [x for x in keys if x < Nk - Sq + s + 1]
        for (s, g) in rows:
            Z = sum(math.exp(sc[(s, g)][x]) for x in kept[(s, g)])
            want = math.log(Z) if Z > 0 else -math.inf
            got = dec["lse_part"][0, s, g, sp]
            assert (got == want) if Z == 0 else abs(got - want) < 1e-12


def test_decode_multi_one_split_is_the_forward_rule_on_a_chunk_of_the_new_tokens():
    # the Sq new tokens as one query block of a chunked prefill (one head, one split): same rows, same tiles
    Nk, Sq, d, Bk, scale, tau = 93, 5, 8, 8, 0.5, 0.5
    q, kc, vc = _multi_inputs(Nk, Sq, d, 1, 271)
    dec = orc.decode_multi(q, kc, vc, scale, tau, 1, Bk)
    f = orc.fwd(q, kc, vc, scale, tau, 8, Bk)           # q [1,Sq,1,d]: the last Sq positions
    assert (dec["mask"] == orc.SKIPPED).sum() > 0
    assert np.array_equal(f["mask"][0, 0, 0], dec["mask"][0, 0, 0])
    assert np.allclose(f["o"][0, :, 0], dec["o"][0, :, 0], atol=1e-13)
    assert np.allclose(f["lse"][0, 0], dec["lse"][0, :, 0], atol=1e-13)


# ------------------------------------------------------------------ forward with the key range cut into splits
@pytest.mark.parametrize("S", [2, 3, 5])
@pytest.mark.parametrize("Nq,Nk", [(64, 64), (24, 72), (13, 50)])
def test_fwd_splits_tau_zero_is_dense_for_any_split_count(Nq, Nk, S):
    d, scale = 8, 0.4
    q, k, v = peaky_inputs(Nk, d, 281)
    qc = q[:, Nk - Nq:]
    f = orc.fwd(qc, k, v, scale, 0.0, 8, 8, num_splits=S)
    od, ld = orc.dense_fwd(qc, k, v, scale)
    assert np.allclose(f["o"], od, atol=1e-12) and np.allclose(f["lse"], ld, atol=1e-12)
    assert not (f["mask"] == orc.SKIPPED).any()


def test_fwd_splits_of_one_query_are_the_decode_rule():
    # one query against 96 keys, 3 ranges of 4 key blocks: exactly split-KV decode of one row
    Nk, d, scale, tau, Bk, S = 96, 8, 0.5, 0.5, 8, 3
    q, kc, vc = _decode_inputs(Nk, d, 1, 291)
    dec = orc.decode(q, kc, vc, scale, tau, S, Bk, packed_rows=False)
    f = orc.fwd(q.reshape(1, 1, 1, d), kc, vc, scale, tau, 4, Bk, num_splits=S)
    assert (dec["mask"] == orc.SKIPPED).sum() > 0
    assert np.array_equal(f["mask"][0, 0, 0], dec["mask"][0, 0].reshape(-1))
    assert np.allclose(f["o"][0, 0, 0], dec["o"][0, 0], atol=1e-13)
    assert abs(f["lse"][0, 0, 0] - dec["lse"][0, 0]) < 1e-13


@pytest.mark.parametrize("Nq,Nk,S,tau", [(32, 96, 3, 0.1), (21, 69, 2, 0.5), (64, 64, 4, 1e-2)])
def test_fwd_splits_match_bruteforce_key_sets_per_range(Nq, Nk, S, tau):
    d, scale, B_ = 32, 1.0 / math.sqrt(32), 8
    off = Nk - Nq
    q, k, v = peaky_inputs(Nk, d, 301 + Nk, boost=5.0)
    qc = q[:, off:]
    f = orc.fwd(qc, k, v, scale, tau, B_, B_, num_splits=S)
    Sm = scale * (qc[0, :, 0] @ k[0, :, 0].T)
    Tc = -(-Nk // B_)
    tps = -(-Tc // S)
    assert (f["mask"] == orc.SKIPPED).sum() > 0
    for i in range(-(-Nq // B_)):
        rows = list(range(i * B_, min(Nq, (i + 1) * B_)))
        Z = {r: [] for r in rows}                     # per row: the ranges' normalizers
        num = {r: np.zeros(d) for r in rows}
        for s in range(S):
            R = {r: [] for r in rows}
            for j in reversed(range(s * tps, min(Tc, (s + 1) * tps))):
                keys = list(range(j * B_, min(Nk, (j + 1) * B_)))
                if keys[0] > rows[-1] + off:
                    assert f["mask"][0, 0, i, j] == 0
                    continue
                skip = True
                for r in rows:
                    legal = [x for x in keys if x <= r + off]
                    if not legal:
                        continue
                    Zt = sum(math.exp(Sm[r, x]) for x in R[r])
                    if Zt == 0.0 or not (math.exp(max(Sm[r, x] for x in legal)) / Zt < tau / (r + 1 + off)):
                        skip = False
                assert f["mask"][0, 0, i, j] == (1 if skip else 2)
                if not skip:
                    for r in rows:
                        R[r] += [x for x in keys if x <= r + off]
            for r in rows:                            # merging by the log-normalizers = pooling the retained keys
                Z[r].append(sum(math.exp(Sm[r, x]) for x in R[r]))
                num[r] += sum((math.exp(Sm[r, x]) * v[0, x, 0] for x in R[r]), np.zeros(d))
        for r in rows:
            assert abs(f["lse"][0, 0, r] - math.log(sum(Z[r]))) < 1e-12
            assert np.allclose(f["o"][0, r, 0], num[r] / sum(Z[r]), atol=1e-12)


def test_decode_paged_with_several_new_tokens_per_sequence():
    # per sequence: the contiguous multi-token rule on its own n keys (same 32-key chunks); a sequence with fewer keys
    # than new tokens leaves its oldest tokens without any key: (0, -inf)
    lens = [128, 96, 64, 2]
    Sq, G, d = 3, 2, 8
    q1, kc, vc, kp, vp, bt = _paged_inputs(4, 128, d, G, 16, lens, 311)
    r = _rng(313)
    q = np.repeat(q1[:, None], Sq, axis=1) + 0.3 * r.standard_normal((4, Sq, G, d))
    q[..., d - 1] = 6.0
    dec = orc.decode_paged(q, kp, vp, bt, lens, 0.5, 0.5, 4, 8)
    assert (dec["mask"] == orc.SKIPPED).sum() > 0
    for b, n in enumerate(lens[:3]):
        S = -(-n // 32)
        ref = orc.decode_multi(q[b:b + 1], kc[b:b + 1, :n], vc[b:b + 1, :n], 0.5, 0.5, S, 8)
        assert np.array_equal(dec["mask"][b, :, :S], ref["mask"][0])
        assert np.allclose(dec["o"][b], ref["o"][0], atol=1e-13) and np.allclose(dec["lse"][b], ref["lse"][0], atol=1e-13)
    # two keys, three new tokens: token 0 sees none, token 1 the first key, token 2 both
    assert (dec["o"][3, 0] == 0).all() and np.isneginf(dec["lse"][3, 0]).all()
    for h in range(G):
        assert np.allclose(dec["o"][3, 1, h], vc[3, 0, 0], atol=1e-12)
        e = np.exp(0.5 * kc[3, :2, 0] @ q[3, 2, h])
        assert np.allclose(dec["o"][3, 2, h], (e / e.sum()) @ vc[3, :2, 0], atol=1e-12)


def test_non_causal_with_more_queries_than_keys_is_plain_softmax():
    # cross attention: 40 queries, 17 keys, every key legal, L = 17
    r = _rng(321)
    q, k, v = r.standard_normal((1, 40, 1, 8)), r.standard_normal((1, 17, 1, 8)), r.standard_normal((1, 17, 1, 8))
    f = orc.fwd(q, k, v, 0.4, 0.0, 8, 8, causal=False)
    for i in range(40):
        e = np.exp(0.4 * k[0, :, 0] @ q[0, i, 0])
        assert np.allclose(f["o"][0, i, 0], (e / e.sum()) @ v[0, :, 0], atol=1e-12)
    do = r.standard_normal(q.shape)
    g = orc.bwd(q, k, v, f["o"], do, f["lse"], 0.4, 0.0, 8, 8, causal=False)
    P = np.exp(0.4 * q[0, :, 0] @ k[0, :, 0].T - f["lse"][0, 0][:, None])
    dP = do[0, :, 0] @ v[0, :, 0].T
    dS = P * (dP - (f["o"][0, :, 0] * do[0, :, 0]).sum(-1)[:, None])
    assert np.allclose(g["dv"][0, :, 0], P.T @ do[0, :, 0], atol=1e-12)
    assert np.allclose(g["dq"][0, :, 0], 0.4 * dS @ k[0, :, 0], atol=1e-12)
    assert np.allclose(g["dk"][0, :, 0], 0.4 * dS.T @ q[0, :, 0], atol=1e-12)


# ------------------------------------------------------------------ a chunk that starts inside a tile
@pytest.mark.parametrize("tau", [1e-2, 0.5])
@pytest.mark.parametrize("Nq,Nk,Bq,Bk,S", [(27, 64, 8, 8, 1), (30, 75, 8, 8, 1), (19, 50, 16, 4, 1), (27, 64, 8, 8, 3)])
def test_chunk_from_any_position_equals_the_rows_of_the_full_run_when_its_blocks_follow_the_positions(Nq, Nk, Bq, Bk,
                                                                                                     S, tau):
    # Nk - Nq is not a multiple of the block: with the query blocks laid out by position (q_shift) the chunked run is
    # the full run restricted to the chunk's rows -- masks of the blocks they share, O and lse; the first block is the
    # last rows of a block of the full run, and a row's result does not depend on the other rows of its block EXCEPT
    # through the block's votes, so equality holds only if the absent rows would not have changed a vote: compare
    # against the full run with those rows' queries removed from the votes, i.e. against a brute force
    d, scale = 32, 1.0 / math.sqrt(32)
    off = Nk - Nq
    shift = off % Bq
    assert shift != 0
    q, k, v = peaky_inputs(Nk, d, 331 + Nk, boost=5.0)
    qc = q[:, off:]
    f = orc.fwd(qc, k, v, scale, tau, Bq, Bk, num_splits=S, q_shift=shift)
    Sm = scale * (qc[0, :, 0] @ k[0, :, 0].T)
    Tc = -(-Nk // Bk)
    tps = -(-Tc // S)
    Tr = -(-(Nq + shift) // Bq)
    assert f["mask"].shape[2] == Tr
    skipped = 0
    for i in range(Tr):
        rows = [r for r in range(i * Bq - shift, (i + 1) * Bq - shift) if 0 <= r < Nq]
        Z = {r: [] for r in rows}
        num = {r: np.zeros(d) for r in rows}
        for s in range(S):
            R = {r: [] for r in rows}
            for j in reversed(range(s * tps, min(Tc, (s + 1) * tps))):
                keys = list(range(j * Bk, min(Nk, (j + 1) * Bk)))
                if keys[0] > rows[-1] + off:
                    assert f["mask"][0, 0, i, j] == 0
                    continue
                skip = True
                for r in rows:
                    legal = [x for x in keys if x <= r + off]
                    if not legal:
                        continue
                    Zt = sum(math.exp(Sm[r, x]) for x in R[r])
                    if Zt == 0.0 or not (math.exp(max(Sm[r, x] for x in legal)) / Zt < tau / (r + 1 + off)):
                        skip = False
                assert f["mask"][0, 0, i, j] == (1 if skip else 2)
                skipped += skip
                if not skip:
                    for r in rows:
                        R[r] += [x for x in keys if x <= r + off]
            for r in rows:
                Z[r].append(sum(math.exp(Sm[r, x]) for x in R[r]))
                num[r] += sum((math.exp(Sm[r, x]) * v[0, x, 0] for x in R[r]), np.zeros(d))
        for r in rows:
            assert abs(f["lse"][0, 0, r] - math.log(sum(Z[r]))) < 1e-12
            assert np.allclose(f["o"][0, r, 0], num[r] / sum(Z[r]), atol=1e-12)
    assert skipped > 0
    if S == 1:   # the blocks that lie wholly inside the chunk are blocks of the full run
        full = orc.fwd(q, k, v, scale, tau, Bq, Bk)
        i_full0 = off // Bq
        for i in range(1, Tr):
            assert np.array_equal(f["mask"][0, 0, i], full["mask"][0, 0, i_full0 + i])
            rows = slice(i * Bq - shift, min(Nq, (i + 1) * Bq - shift))
            assert np.array_equal(f["o"][0, rows], full["o"][0, off:][rows])


@pytest.mark.parametrize("tau", [1e-2, 0.5])
@pytest.mark.parametrize("Nq,Nk,Bq,Bk", [(27, 64, 8, 8), (30, 75, 8, 8), (19, 50, 16, 4), (24, 64, 8, 8)])
def test_bwd_of_a_chunk_from_any_position_matches_bruteforce(Nq, Nk, Bq, Bk, tau):
    # the offline rule on a chunk whose query blocks follow the positions (q_shift = (Nk - Nq) mod Bq): every tile
    # decision and the three gradients against a brute force over entries, and the tile decisions of every query
    # block the chunk holds completely against the backward pass of the whole sequence with the same lse
    d, scale = 32, 1.0 / math.sqrt(32)
    off = Nk - Nq
    shift = off % Bq
    q, k, v = peaky_inputs(Nk, d, 431 + Nk, boost=5.0)
    do = _rng(432).standard_normal(q.shape)
    qc, doc = q[:, off:], do[:, off:]
    f = orc.fwd(qc, k, v, scale, tau, Bq, Bk, q_shift=shift)
    g = orc.bwd(qc, k, v, f["o"], doc, f["lse"], scale, tau, Bq, Bk, q_shift=shift)
    dQ, dK, dV, M = brute_mala_bwd(qc[0, :, 0], k[0, :, 0], v[0, :, 0], doc[0, :, 0], f["o"][0, :, 0], f["lse"][0, 0],
                                   scale, tau, Bq, Bk, shift=shift)
    assert (g["mask"][0, 0] == M).all() and (M == 1).any()
    assert np.allclose(g["dq"][0, :, 0], dQ, atol=1e-11)
    assert np.allclose(g["dk"][0, :, 0], dK, atol=1e-11)
    assert np.allclose(g["dv"][0, :, 0], dV, atol=1e-11)
    # whole sequence, its lse rows replaced by the chunk's: the blocks they share decide alike
    ff = orc.fwd(q, k, v, scale, tau, Bq, Bk)
    lse = ff["lse"].copy()
    lse[:, :, off:] = f["lse"]
    gg = orc.bwd(q, k, v, ff["o"], do, lse, scale, tau, Bq, Bk)
    i_first = off // Bq + (1 if shift else 0)                   # first block of the whole run made of chunk rows only
    assert np.array_equal(g["mask"][0, 0][:, i_first - off // Bq:], gg["mask"][0, 0][:, i_first:])
    # dq_units / key_units take the same blocks
    part = orc.bwd(qc, k, v, f["o"], doc, f["lse"], scale, tau, Bq, Bk, key_units=[(0, 0, 1)], dq_units=[(0, 0, 0), (0, 0, 2)],
                   q_shift=shift)
    r0 = slice(0, Bq - shift)
    r2 = slice(2 * Bq - shift, min(Nq, 3 * Bq - shift))
    assert np.allclose(part["dq"][0, r0, 0], dQ[r0], atol=1e-11) and np.allclose(part["dq"][0, r2, 0], dQ[r2], atol=1e-11)
    assert np.allclose(part["dk"][0, Bk:2 * Bk, 0], dK[Bk:2 * Bk], atol=1e-11)


# ------------------------------------------------------------------ matched-work diagnostics (analysis on the oracle)
def test_matched_work_controls():
    from oracle import matched_work as mw
    B, N, Hq, Hkv, d, Bq, Bk, tau = 3, 96, 4, 2, 16, 8, 8, 0.3
    q, k, v = peaky_inputs(N, d, 501, Hq=Hq, Hkv=Hkv, B=B, boost=3.0)
    q[:, :, 0] *= 0.3                                            # one diffuse head: the heads' counts differ
    scale = 1.0 / math.sqrt(d)
    res = mw.matched_work(q, k, v, scale, tau, Bq, Bk)
    f = orc.fwd(q, k, v, scale, tau, Bq, Bk)
    assert res["tiles"] == int((f["mask"] == orc.RETAINED).sum()) and (f["mask"] == orc.SKIPPED).sum() > 0
    # MALA's omitted mass from the tile masses of the dense softmax = 1 - exp(lse_screened - lse_reference)
    _, lse_ref = orc.dense_fwd(q, k, v, scale)
    om = 1.0 - np.exp(f["lse"] - lse_ref)                        # [B,Hq,N]
    assert np.allclose(res["mala_per_block"], om.reshape(B, Hq, N // Bq, Bq).mean(axis=3), atol=1e-12)
    assert 0 < res["mala"] <= tau / (1 + tau)
    # every policy spends exactly MALA's number of tiles
    for p_ in ("per_instance", "static", "position_only"):
        assert int(res["budgets"][p_].sum()) == res["tiles"]
    # with MALA's own count per decision, keeping the heaviest tiles cannot omit more (block sums) than MALA does
    assert (res["per_instance_per_block"] <= res["mala_per_block"] + 1e-12).all()
    assert res["per_instance"] <= res["mala"] and res["per_instance"] <= res["static"] + 1e-12
    # brute force of the per-instance control on one decision
    b, h, i = 1, 2, 7
    S = scale * (q[b, :, h] @ k[b, :, h // 2].T)
    S[np.triu_indices(N, 1)] = -np.inf
    P = np.exp(S - S.max(axis=1, keepdims=True))
    P /= P.sum(axis=1, keepdims=True)
    rows = P[i * Bq:(i + 1) * Bq]
    mass = [rows[:, j * Bk:(j + 1) * Bk].sum() for j in range(i + 1)]
    n = int((f["mask"][b, h, i] == orc.RETAINED).sum())
    best = sorted(mass, reverse=True)[:n]
    assert abs(res["per_instance_per_block"][b, h, i] - (1.0 - sum(best) / Bq)) < 1e-12
    # tau = 0: nothing omitted by anyone; one batch entry: the static control is the per-instance one
    z = mw.matched_work(q, k, v, scale, 0.0, Bq, Bk)
    assert max(abs(z[p_]) for p_ in ("mala", "per_instance", "static", "position_only")) < 1e-12
    one = mw.matched_work(q[:1], k[:1], v[:1], scale, tau, Bq, Bk)
    assert np.array_equal(one["budgets"]["static"], one["budgets"]["per_instance"])
