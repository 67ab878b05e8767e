"""Pins of the oracle's MXFP4 mode (Sec. 4.3, "DSS on MXFP4").  The paper gives no procedure for
it, so the oracle follows a stated reading; these tests hold that reading to the format's
definition (E8M0 powers of two, the plain rule's shared exponent), to a separate NumPy
restatement built on library casts, to a brute-force argmin, and to the properties the
reading must have: the plain exponent is always a candidate, the search is bounded below
by nearest rounding under each candidate scale, and on heavy-tailed synthetic weights it
ends below plain MXFP4's error.
"""
import ml_dtypes
import numpy as np
import pytest

from oracle import soar_ref as R
from paper_2605_12245_b200 import workloads as WL

F32 = np.float32
GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def mags_of(bits):
    return np.abs(WL.bf16_bits_to_f32(bits)).astype(F32)


def np_round(mag, r):
    """E2M1 rounding of fl32(mag * r) through the library cast (saturating at 6)."""
    x = np.minimum((mag.astype(F32) * F32(r)).astype(F32), F32(6.0))
    return x.astype(ml_dtypes.float4_e2m1fn).astype(np.float64)


def test_e8m0_codes_are_the_powers_of_two():
    lib = np.arange(255, dtype=np.uint8).view(ml_dtypes.float8_e8m0fnu).astype(np.float64)
    for c in range(255):
        assert R.e8m0_decode(c) == 2.0 ** (c - 127) == lib[c]


def test_plain_rule_is_floor_log2_of_the_maximum_minus_two():
    for bmax, want in ((1.0, 125), (1.99, 125), (2.0, 126), (6.0, 127), (7.9, 127), (8.0, 128), (2.0 ** -100, 25),
                       (3.0 * 2.0 ** 90, 127 + 91 - 2)):
        assert R.mx_plain_code(bmax) == want
    # with that scale the largest element lands in [4, 8): one binade below saturation or clipped at 6
    for e in range(-20, 20):
        for m in (1.0, 1.25, 1.5, 1.9921875):
            bmax = m * 2.0 ** e
            x = bmax / R.e8m0_decode(R.mx_plain_code(bmax))
            assert 4.0 <= x < 8.0


def test_candidates_bracket_the_scale_and_hold_the_plain_exponent():
    assert R.mx_candidates(1.0, 2) == [127, 128] and R.mx_candidates(1.99, 2) == [127, 128]
    assert R.mx_candidates(0.3, 2) == [125, 126] and R.mx_candidates(3.0, 4) == [127, 128, 129, 130]
    assert R.mx_candidates(1.4, 1) == [127] and R.mx_candidates(1.6, 1) == [128] and R.mx_candidates(1.5, 1) == [127]
    assert R.mx_candidates(2.0 ** -127, 2) == [0, 1] and R.mx_candidates(2.0 ** -127 * 0.5, 2) == [0]
    rng = np.random.default_rng(0)
    for _ in range(2000):                       # every block maximum: the plain exponent is one of the two
        bmax = float(F32(np.exp(rng.uniform(-30, 30))))
        assert R.mx_plain_code(bmax) in R.mx_candidates(float(F32(bmax) / F32(6.0)), 2)


def test_plain_mxfp4_equals_a_numpy_restatement():
    w = WL.small_case(24, 256, 401, outlier_entry_frac=0.01, outlier_scale=40.0)
    w[3, 32:64] = 0
    got = R.mx_quantize(w, n_beta=0)
    mag = mags_of(w).reshape(-1, 32)
    bmax = mag.max(axis=1)
    live = bmax > 0
    exp = np.where(live, np.floor(np.log2(np.where(live, bmax, 1.0))).astype(np.int64) - 2, -127)
    scale = np.ldexp(1.0, exp)
    m = np.stack([np_round(mag[i], 1.0 / scale[i]) if live[i] else np.zeros(32) for i in range(len(mag))])
    code = (np.searchsorted(GRID, m).astype(np.uint8) | ((w.reshape(-1, 32) >> 15).astype(np.uint8) << 3))
    packed = (code[:, 0::2] | (code[:, 1::2] << 4)).reshape(24, 128)
    assert np.array_equal(got.packed, packed)
    assert np.array_equal(got.scales.reshape(-1), np.where(live, exp + 127, 0).astype(np.uint8))
    sse = float(((mag.astype(np.float64) - m * scale[:, None]) ** 2).sum())
    assert got.sse == pytest.approx(sse, rel=1e-12)
    assert got.sumsq == pytest.approx(float((mag.astype(np.float64) ** 2).sum()), rel=1e-12)


@pytest.mark.parametrize("n_dq,n_beta,step", [(2, 101, 1), (4, 21, 4), (1, 11, 2)])
def test_search_winner_is_the_brute_force_first_minimum(n_dq, n_beta, step):
    w = WL.small_case(6, 128, 402 + n_dq, dist="laplace", outlier_entry_frac=0.02, outlier_scale=30.0)
    got = R.mx_quantize(w, n_dq=n_dq, n_beta=n_beta, beta_step_pct=step)
    mag = mags_of(w).reshape(-1, 32)
    total = 0.0
    for i, a in enumerate(mag):
        center = F32(a.max() / F32(6.0))
        cands = R.mx_candidates(float(center), n_dq)
        best, best_m, best_c = None, None, None
        for k in range(n_beta):
            dq = F32(center * F32((100.0 + (k - n_beta // 2) * step) / 100.0))
            m = np_round(a, F32(1.0) / dq)
            for c in cands:
                e = a.astype(np.float64) - m * 2.0 ** (c - 127)
                L = 0.0
                for t in e * e:
                    L += t
                if best is None or L < best:
                    best, best_m, best_c = L, m, c
        total += best
        code = np.searchsorted(GRID, best_m).astype(np.uint8) | ((w.reshape(-1, 32)[i] >> 15).astype(np.uint8) << 3)
        assert got.scales.reshape(-1)[i] == best_c, i
        assert np.array_equal(got.packed.reshape(-1, 16)[i], code[0::2] | (code[1::2] << 4)), i
    assert got.sse == pytest.approx(total, rel=1e-12)


def test_search_is_bounded_by_nearest_rounding_and_beats_the_plain_rule_on_heavy_tails():
    """For a fixed stored scale the error-minimising codes are the nearest ones under that very scale, so
    no multiplier can do better than that: a lower bound for every block.  Against the plain rule the
    search gains where it counts, on blocks whose maximum the plain exponent clips."""
    w = WL.small_case(64, 1024, 410, outlier_entry_frac=0.003, outlier_scale=30.0)
    plain, dss = R.mx_quantize(w, n_beta=0), R.mx_quantize(w)
    assert dss.sse < 0.97 * plain.sse
    mag = mags_of(w).reshape(-1, 32)
    blocks = w.reshape(-1, 32)
    sum_got = sum_floor = 0.0
    for i in range(0, len(mag), 7):
        a = mag[i]
        if a.max() == 0:
            continue
        cands = R.mx_candidates(float(F32(a.max()) / F32(6.0)), 2)
        floor = min(R.mx_block_error(blocks[i], R.mx_round_block(blocks[i], 2.0 ** (c - 127)), c) for c in cands)
        m = GRID[(dss.packed.reshape(-1, 16)[i][:, None] >> np.array([0, 4])) & 7].reshape(-1)
        got = R.mx_block_error(blocks[i], m, int(dss.scales.reshape(-1)[i]))
        assert got >= floor * (1 - 1e-12)
        sum_got += got
        sum_floor += floor
    # the grid of a hundredth comes close to that bound (the upper candidate's own value can lie beyond
    # the largest multiplier, 1.5, so single blocks may stay above it)
    assert sum_got <= 1.1 * sum_floor


def test_zero_and_tiny_blocks_and_bad_input():
    w = WL.small_case(2, 96, 420)
    w[0, :32] = 0
    w[0, 5] = 0x8000
    w[1, 32:64] = WL.f32_to_bf16_bits(np.full(32, 1e-38, np.float32))
    for nb in (0, 101):
        r = R.mx_quantize(w, n_beta=nb)
        assert r.scales[0, 0] == 0 and r.packed[0, 2] == 0x80 and not r.packed[0, :2].any()
        assert r.scales[1, 1] == 0 and not (r.packed[1, 16:32] & 0x77).any()
        assert r.status == 0
    bad = w.copy()
    bad[1, 3] = 0x7FC0
    assert R.mx_quantize(bad).status & R.STATUS_NONFINITE
    assert R.mx_quantize(np.zeros((2, 64), np.uint16)).status & R.STATUS_ZERO_TENSOR
