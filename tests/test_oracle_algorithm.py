"""Pins for the oracle's whole loop (Algorithm 1 of the paper): the C oracle against the
separately written NumPy restatement, special cases with a closed-form answer, and the
invariants the method guarantees."""
import ml_dtypes
import numpy as np
import pytest

from oracle import soar_np as N
from oracle import soar_ref as R
from paper_2605_12245_b200 import workloads as WL

GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def unpack(packed):
    lo, hi = packed & 0xF, packed >> 4
    return np.stack([lo, hi], axis=-1).reshape(packed.shape[0], -1)


def dequant(packed, scales, alpha):
    codes = unpack(packed)
    q = GRID[codes & 7] * np.where(codes & 8, -1.0, 1.0)
    s = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)[scales]
    return q * np.repeat(s, 16, axis=1) * alpha


@pytest.mark.parametrize("rows,cols,seed,kw", [
    (8, 64, 0, {}),
    (16, 256, 1, dict(outlier_entry_frac=0.01, outlier_scale=50.0)),
    (12, 320, 2, dict(dist="laplace", outlier_cols_frac=0.01, outlier_scale=20.0)),
    (6, 512, 3, dict(dist="gauss_t2mix")),
])
@pytest.mark.parametrize("cfg", [
    dict(),                                                   # the paper's setting
    dict(max_iters=3, early_stop_rel=0.0, n_dq=1, n_beta=1),  # coupled nearest scale, no search
    dict(max_iters=2, early_stop_rel=0.0, n_dq=4, n_beta=5, beta_step_pct=3),
    dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1),
])
def test_c_oracle_equals_numpy_restatement(rows, cols, seed, kw, cfg):
    w = WL.small_case(rows, cols, seed, **kw)
    a = R.quantize(w, R.RefCfg(**cfg))
    b = N.quantize(w, **cfg)
    assert a.status == 0
    assert a.iters_run == b["iters_run"]
    assert a.alpha == b["alpha"]
    assert np.array_equal(a.trace_alpha, b["trace_alpha"])
    assert np.array_equal(a.packed, b["packed"])
    assert np.array_equal(a.scales, b["scales"])
    assert np.allclose(a.trace_sse, b["trace_sse"], rtol=1e-12, atol=0)


def test_zero_iterations_is_the_max_based_rule():
    """T = 0 must be Eq. 1-3 written out: checked against a direct evaluation here."""
    w = WL.small_case(16, 128, 7)
    r = R.quantize(w, R.RefCfg(max_iters=0))
    wf = WL.bf16_bits_to_f32(w).astype(np.float64)
    amax = np.abs(wf).max()
    assert r.alpha == pytest.approx(amax / (6 * 448), rel=1e-7)
    bmax = np.abs(wf).reshape(16, -1, 16).max(axis=2)
    want_scale = (bmax / (r.alpha * 6)).astype(np.float32).astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    # the binary32 quotient can differ from this binary64 one only next to an E4M3 midpoint
    assert np.mean(want_scale != r.scales) < 0.01
    x = np.abs(wf) / (r.alpha * np.repeat(np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)[r.scales], 16, axis=1))
    want_m = np.minimum(x, 6).astype(np.float32).astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    got_m = GRID[unpack(r.packed) & 7]
    assert np.mean(want_m != got_m) < 1e-3
    assert np.array_equal((unpack(r.packed) >> 3).astype(bool), (w >> 15).astype(bool))
    sse = float(np.sum((wf - dequant(r.packed, r.scales, r.alpha)) ** 2))
    assert r.trace_sse[0] == pytest.approx(sse, rel=1e-12)


def test_grid_aligned_tensor_reconstructs_exactly():
    """Entries c_i * g with g on the E2M1 grid, c_i = 2^k * (an E4M3 value), a 6*c_i in
    every block and one block at the top of the range: the max-based rule already
    represents the tensor, Eq. 5 leaves alpha unchanged and no iteration can change it."""
    rng = np.random.default_rng(0)
    rows, nb = 4, 8
    e4 = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    # block scales with <= 2 significant bits so that 6*c and every product fit bf16's 8 bits
    sc_codes = rng.choice([0x7E - 8 * i - 6 for i in range(1, 6)] + [0x7E - 8 * i - 2 for i in range(1, 6)], size=(rows, nb))
    unit = 2.0 ** -12
    qs = rng.choice(GRID, size=(rows, nb, 16)) * rng.choice([-1.0, 1.0], size=(rows, nb, 16))
    qs[:, :, 0] = 6.0
    scales = e4[sc_codes]
    scales[0, 0] = 448.0
    sc_codes[0, 0] = 0x7E
    w = (qs * scales[:, :, None] * unit).reshape(rows, -1)
    bits = WL.f32_to_bf16_bits(w.astype(np.float32))
    assert np.array_equal(WL.bf16_bits_to_f32(bits).astype(np.float64), w)   # representable
    for T in (0, 3):
        r = R.quantize(bits, R.RefCfg(max_iters=T, early_stop_rel=0.0))
        assert r.alpha == pytest.approx(unit, rel=2e-7)
        rec = dequant(r.packed, r.scales, r.alpha)
        assert np.allclose(rec, w, rtol=3e-7, atol=0)
        assert r.trace_sse[-1] <= 1e-12 * r.sumsq
        assert np.array_equal(r.scales, sc_codes)
        assert np.array_equal(GRID[unpack(r.packed) & 7], np.abs(qs).reshape(rows, -1))


def test_error_never_above_max_based_and_reported_error_is_true_error():
    for seed, kw in enumerate([{}, dict(outlier_entry_frac=0.005, outlier_scale=50.0), dict(dist="laplace")]):
        w = WL.small_case(32, 512, 10 + seed, **kw)
        base = R.quantize(w, R.RefCfg(max_iters=0))
        one = R.quantize(w, R.RefCfg(max_iters=1))
        full = R.quantize(w, R.RefCfg())
        assert full.trace_sse[0] == base.trace_sse[0]
        assert one.trace_sse[-1] < base.trace_sse[0]
        assert full.trace_sse[-1] <= one.trace_sse[-1]
        assert full.trace_sse[-1] < 0.99 * base.trace_sse[0]      # SOAR improves on amax scaling
        wf = WL.bf16_bits_to_f32(w).astype(np.float64)
        for r in (base, one, full):
            true = float(np.sum((wf - dequant(r.packed, r.scales, r.alpha)) ** 2))
            assert r.trace_sse[-1] == pytest.approx(true, rel=1e-11)
            sse, ss = R.dequant_error(w, r.packed, r.scales, r.alpha)
            assert sse == pytest.approx(true, rel=1e-12)
            assert ss == pytest.approx(float(np.sum(wf ** 2)), rel=1e-12)
            assert r.sumsq == pytest.approx(ss, rel=1e-12)


def test_search_never_worse_than_coupled_nearest_scale_in_the_same_iteration():
    """beta = 1.00 and the nearest E4M3 code are in the candidate set, so one SOAR
    iteration cannot end above one CJSO-only iteration from the same start (Eq. 8)."""
    w = WL.small_case(16, 512, 21)
    soar = R.quantize(w, R.RefCfg(max_iters=1, early_stop_rel=0.0))
    # per block: n_dq = 2 contains the nearest code; n_beta = 101 contains beta = 1
    cjso_q = R.quantize(w, R.RefCfg(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1))
    assert soar.trace_alpha[1] == cjso_q.trace_alpha[1]
    assert soar.trace_sse[1] <= cjso_q.trace_sse[1]
    cjso = R.quantize(w, R.RefCfg(max_iters=1, early_stop_rel=0.0, n_dq=1, n_beta=1))
    assert cjso_q.trace_sse[1] <= cjso.trace_sse[1]


def test_early_stop_rule():
    w = WL.small_case(16, 256, 30)
    free = R.quantize(w, R.RefCfg(max_iters=6, early_stop_rel=0.0))
    assert free.iters_run == 6
    for eps in (1e-3, 1e-2, 0.5):
        r = R.quantize(w, R.RefCfg(max_iters=6, early_stop_rel=eps))
        gains = (free.trace_sse[:-1] - free.trace_sse[1:]) / free.trace_sse[:-1]
        first = next((i for i, g in enumerate(gains) if g < eps), 5)
        assert r.iters_run == first + 1
        assert np.array_equal(r.trace_sse, free.trace_sse[: r.iters_run + 1])


def test_output_footprint_is_plain_nvfp4():
    w = WL.small_case(8, 128, 40)
    r = R.quantize(w, R.RefCfg(max_iters=2))
    assert r.packed.nbytes == w.size // 2 and r.scales.nbytes == w.size // 16
    assert r.packed.nbytes + r.scales.nbytes + 4 == w.size * 4.5 / 8 + 4


def test_degenerate_inputs():
    z = np.zeros((2, 32), np.uint16)
    z[0, 3] = 0x8000                                     # a negative zero keeps its sign bit
    r = R.quantize(z, R.RefCfg())
    assert r.status == R.STATUS_ZERO_TENSOR and r.alpha == 1.0
    assert not r.scales.any() and unpack(r.packed)[0, 3] == 8 and unpack(r.packed).sum() == 8
    w = WL.small_case(4, 64, 50)
    w[1, 16:32] = 0                                      # one all-zero block
    w[2, 32:48] = WL.f32_to_bf16_bits(np.full(16, 1e-12, np.float32))   # far below the range
    r = R.quantize(w, R.RefCfg())
    assert r.status == 0 and r.scales[1, 1] == 0 and not unpack(r.packed)[1, 16:32].any()
    assert r.scales[2, 2] == 1 and not (unpack(r.packed)[2, 32:48] & 7).any()
    b = N.quantize(w)
    assert np.array_equal(r.packed, b["packed"]) and np.array_equal(r.scales, b["scales"])
    bad = w.copy(); bad[0, 0] = 0x7F80
    assert R.quantize(bad, R.RefCfg()).status & R.STATUS_NONFINITE
    bad[0, 0] = 0x7FC0
    assert R.quantize(bad, R.RefCfg()).status & R.STATUS_NONFINITE
    tiny = WL.f32_to_bf16_bits(np.full((1, 16), 1e-35, np.float32))
    assert R.quantize(tiny, R.RefCfg()).status & R.STATUS_RANGE


def test_tie_flags_mark_structural_ties_only():
    w = WL.small_case(64, 512, 60)
    r = R.quantize(w, R.RefCfg(max_iters=2), tie_rel=1e-6)
    assert r.tie_flags.mean() < 1e-3
    loose = R.quantize(w, R.RefCfg(max_iters=2), tie_rel=1e-2)
    assert loose.tie_flags.sum() > r.tie_flags.sum()
    # a block whose codes are all zero for every candidate ties exactly between its two scales
    w[3, 0:16] = WL.f32_to_bf16_bits(np.full(16, 1e-9, np.float32))
    r = R.quantize(w, R.RefCfg(max_iters=1), tie_rel=1e-6)
    assert r.tie_flags[3, 0] == 1
