"""A structural fact about the search of Eq. 8, checked on the oracle: for a fixed E4M3
dequantization code the block error over the multiplier grid of App. B.3 falls until the
quantization divisor alpha * dq passes alpha * value(code) and rises afterwards, so the
oracle's argmin over the whole grid always sits at one of the grid points that bracket
that crossing.  The CUDA search relies on this to visit two or three multipliers instead
of 101; here the claim is tested against the oracle's own single-step functions
(every candidate re-rounded and its error summed term by term), independently of any kernel.
"""
import numpy as np
import pytest

from oracle import soar_ref as R
from paper_2605_12245_b200 import workloads as WL

F32 = np.float32


def grid_errors(w16, alpha, center, code, n_beta, step):
    """Error of every multiplier of the grid for one block and one E4M3 code, and the codes."""
    errs, codes, divisors = [], [], []
    for k in range(n_beta):
        dq = F32(F32(center) * F32(R.beta(k, n_beta, step)))
        m, _, _ = R.round_block(w16, alpha, dq)
        errs.append(R.block_error(w16, m, alpha, code))
        codes.append(m)
        divisors.append(float(F32(F32(alpha) * dq)))
    return np.array(errs), np.array(codes), np.array(divisors, dtype=np.float64)


def bracket(divisors, sd):
    """Grid points that can win: the last with divisor <= sd (1 - 2^-23), the first with
    divisor >= sd (1 + 2^-22), and any in between."""
    lo, hi = sd * (1 - 2.0 ** -23), sd * (1 + 2.0 ** -22)
    k_lo = int(np.searchsorted(divisors, lo, side="right")) - 1
    k_hi = int(np.searchsorted(divisors, hi, side="left"))
    return list(range(max(k_lo, 0), min(k_hi, len(divisors) - 1) + 1))


@pytest.mark.parametrize("n_beta,step", [(101, 1), (21, 3), (8, 1)])
def test_grid_argmin_lies_in_the_bracket_around_the_dequantization_scale(n_beta, step):
    rng = np.random.default_rng(7 + n_beta)
    checked = 0
    widths = []
    for trial in range(160):
        w16 = WL.small_case(1, 16, 9000 + trial, dist=("laplace" if trial % 3 == 0 else "student_t4"),
                            outlier_entry_frac=0.05 * (trial % 2), outlier_scale=50.0)[0]
        mag = np.abs(WL.bf16_bits_to_f32(w16))
        if mag.max() == 0:
            continue
        # alpha with a full significand, so that no element sits exactly on a rounding midpoint
        alpha = float(F32(rng.uniform(0.5, 2.0) * 1e-4 * (1 + 2.0 ** -20)))
        center = float(F32(mag.max() / (6 * alpha) * rng.uniform(0.55, 1.45)))
        for code in R.dq_candidates(center, 2):
            errs, codes, divisors = grid_errors(w16, alpha, center, code, n_beta, step)
            sd = float(np.float64(F32(alpha)) * np.float64(R.e4m3_decode(code)))
            cand = bracket(divisors, sd)
            widths.append(len(cand))
            k_all = int(np.argmin(errs))
            k_br = cand[int(np.argmin(errs[cand]))]
            assert np.array_equal(codes[k_br], codes[k_all]), (trial, code, k_all, k_br, errs[k_all], errs[k_br])
            # the error never rises before the bracket and never falls after it
            assert np.all(np.diff(errs[: cand[0] + 1]) <= 0) and np.all(np.diff(errs[cand[-1]:]) >= 0)
            checked += 1
    assert checked > 250 and max(widths) <= 3


def test_bracket_holds_for_a_weighted_error_with_positive_weights():
    rng = np.random.default_rng(3)
    for trial in range(60):
        w16 = WL.small_case(1, 16, 9500 + trial, outlier_entry_frac=0.05, outlier_scale=30.0)[0]
        mag = np.abs(WL.bf16_bits_to_f32(w16))
        if mag.max() == 0:
            continue
        h = np.exp(rng.normal(0, 1.0, 16)).astype(np.float32)
        alpha = float(F32(rng.uniform(0.5, 2.0) * 1e-4 * (1 + 2.0 ** -20)))
        center = float(F32(mag.max() / (6 * alpha) * rng.uniform(0.6, 1.4)))
        for code in R.dq_candidates(center, 2):
            errs, codes, divisors = [], [], []
            for k in range(101):
                dq = F32(F32(center) * F32(R.beta(k, 101, 1)))
                m, _, _ = R.round_block(w16, alpha, dq, h=h)
                errs.append(R.block_error(w16, m, alpha, code, h=h))
                codes.append(m)
                divisors.append(float(F32(F32(alpha) * dq)))
            errs, codes = np.array(errs), np.array(codes)
            sd = float(np.float64(F32(alpha)) * np.float64(R.e4m3_decode(code)))
            cand = bracket(np.array(divisors), sd)
            assert np.array_equal(codes[cand[int(np.argmin(errs[cand]))]], codes[int(np.argmin(errs))])
