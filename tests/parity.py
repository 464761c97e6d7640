"""Shared comparison helpers for the GPU parity tests (no method arithmetic lives here)."""
import numpy as np

# limits fixed by the benchmark definition for bf16 inputs
O_MAX_ABS, O_MEAN_ABS = 2e-2, 2e-3
GRAD_REL_L2 = 1e-2
LSE_ABS = 1e-3          # fp32 log-sum-exp of scores of magnitude <= ~100
MASK_BAND = 1e-3        # tiles whose criterion lies within 1e-3 (relative, i.e. in log) of tau are exempt


def check_mask(gpu_retained, oracle_mask, oracle_crit, order, tau, L_min, Bk=128):
    """Bit-exact comparison of one row of retention decisions, except near-threshold tiles.

    gpu_retained: bool [T]; oracle_mask: uint8 [T] (0 illegal, 1 skipped, 2 retained); oracle_crit [T];
    order: tile indices in visiting order.  A tile may differ only if |C| <= MASK_BAND; after such a flip the
    running normalizer of that row block differs by at most Bk*tau/L, which widens the band for later tiles.
    Returns the number of exempted flips."""
    band = MASK_BAND
    flips = 0
    for x in order:
        if oracle_mask[x] == 0:
            assert not gpu_retained[x], f"tile {x} is not legal but was reported retained"
            continue
        want = oracle_mask[x] == 2
        if bool(gpu_retained[x]) != bool(want):
            assert abs(oracle_crit[x]) <= band, (
                f"tile {x}: gpu={bool(gpu_retained[x])} oracle={bool(want)} criterion={oracle_crit[x]:.3e} band={band:.1e}")
            flips += 1
            band = MASK_BAND + Bk * tau / max(L_min, 1)
    return flips


BF16_U = 2.0 ** -8      # unit roundoff of bf16 (8 significand bits)


def check_output(o_gpu, o_ref, what="o", a_ref=None):
    """Output limits.  Default: the benchmark definition's absolute limits (max-abs, mean-abs).

    With ``a_ref`` (the oracle's result for the same call with |V| in place of V, i.e. a = sum_k p_k |v_k| over the
    retained keys) the comparison is the rounding model of the kernels instead: P is cast to bf16 before P V
    (relative error <= u per probability, the normalizer is summed in fp32 before the cast) and the output is cast to
    bf16 (relative error <= u), so |o_gpu - o| <= u (|o| + a) up to second-order and fp32 terms.  That bound is asserted
    element by element; the absolute max-abs limit stays asserted on every element with |o| <= 3, and the mean error
    must stay below half the mean bound (rounding errors are spread over +-bound, not all at the bound)."""
    diff = np.abs(np.asarray(o_gpu, dtype=np.float64) - o_ref)
    assert np.isfinite(diff).all(), f"{what}: non-finite values"
    if a_ref is None:
        assert diff.max() <= O_MAX_ABS, f"{what}: max abs err {diff.max():.3e}"
        assert diff.mean() <= O_MEAN_ABS, f"{what}: mean abs err {diff.mean():.3e}"
        return diff.max(), diff.mean()
    bound = BF16_U * (np.abs(o_ref) + np.abs(a_ref)) * 1.02 + 1e-5
    worst = (diff - bound).max()
    assert worst <= 0, f"{what}: error exceeds the bf16 rounding bound by {worst:.3e}"
    small = np.abs(o_ref) <= 3.0
    if small.any():
        assert diff[small].max() <= O_MAX_ABS, f"{what}: max abs err {diff[small].max():.3e} where |o| <= 3"
    assert diff.mean() <= 0.5 * bound.mean(), f"{what}: mean abs err {diff.mean():.3e} vs mean bound {bound.mean():.3e}"
    return diff.max(), diff.mean()


def rel_l2(a, ref):
    a = np.asarray(a, dtype=np.float64)
    return float(np.linalg.norm(a - ref) / max(np.linalg.norm(ref), 1e-30))


def check_grad(g_gpu, g_ref, what):
    assert np.isfinite(np.asarray(g_gpu, dtype=np.float64)).all(), f"{what}: non-finite values"
    e = rel_l2(g_gpu, g_ref)
    assert e <= GRAD_REL_L2, f"{what}: relative L2 error {e:.3e}"
    return e
