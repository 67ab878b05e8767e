"""Pins for the oracle's column-weighted objective (the diagonal form of the output-distortion
objective the paper's Sec. 5 proposes): sum_ij h_j (W_ij - What_ij)^2.

What fixes it, independently of the oracle's own formulas: the unweighted method (h = 1),
invariance under a constant weight, weighted least squares computed here by a library solver,
columns of zero weight, a separate NumPy restatement, and the true weighted error of the
returned codes."""
import numpy as np
import pytest

from oracle import soar_np as N
from oracle import soar_ref as R
from paper_2605_12245_b200 import workloads as WL

GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
FAST = dict(max_iters=2, early_stop_rel=0.0, n_dq=2, n_beta=11, beta_step_pct=5)


def e4m3_vals():
    return np.array([R.e4m3_decode(c) for c in range(0x7F)])


def dequant(res):
    lo, hi = res.packed & 0xF, res.packed >> 4
    codes = np.stack([lo, hi], axis=-1).reshape(res.packed.shape[0], -1)
    q = GRID[codes & 7] * np.where(codes & 8, -1.0, 1.0)
    return q * np.repeat(e4m3_vals()[res.scales], 16, axis=1) * np.float64(np.float32(res.alpha))


def same_outputs(a, b):
    return (np.array_equal(a.packed, b.packed) and np.array_equal(a.scales, b.scales)
            and a.alpha == b.alpha and a.iters_run == b.iters_run)


@pytest.mark.parametrize("cfg", [dict(), FAST, dict(max_iters=0), dict(max_iters=3, n_dq=1, n_beta=1, flags=R.FLAG_COUPLED_SCALE)])
def test_unit_weights_are_the_unweighted_method(cfg):
    w = WL.small_case(16, 256, 5, outlier_entry_frac=0.01, outlier_scale=30.0)
    a = R.quantize(w, R.RefCfg(**cfg))
    b = R.quantize(w, R.RefCfg(**cfg), h=np.ones(256, np.float32))
    assert same_outputs(a, b)
    assert np.array_equal(a.trace_sse, b.trace_sse) and a.sumsq == b.sumsq
    assert np.array_equal(a.tie_flags, b.tie_flags)


@pytest.mark.parametrize("c", [4.0, 0.125, 3.0, 0.3])
def test_constant_weight_changes_nothing_but_the_error_scale(c):
    """The minimiser of c * f is the minimiser of f.  A power of two scales every binary64
    term exactly; any other constant perturbs roundings, which only near-ties could feel."""
    w = WL.small_case(12, 320, 7)
    a = R.quantize(w, R.RefCfg(**FAST))
    b = R.quantize(w, R.RefCfg(**FAST), h=np.full(320, c, np.float32))
    cf = float(np.float32(c))
    if c in (4.0, 0.125):
        assert same_outputs(a, b)
        assert np.array_equal(b.trace_sse, a.trace_sse * cf) and b.sumsq == a.sumsq * cf
    else:
        clear = a.tie_flags == 0
        assert np.array_equal(a.scales[clear], b.scales[clear])
        assert np.allclose(b.trace_sse, a.trace_sse * cf, rtol=1e-6)
        assert b.alpha == pytest.approx(a.alpha, rel=1e-6)


def test_block_sums_and_error_carry_the_weights():
    rng = np.random.default_rng(0)
    for _ in range(50):
        w = WL.f32_to_bf16_bits((rng.standard_t(4, 16) * 0.02).astype(np.float32))
        h = rng.uniform(0.01, 30.0, 16).astype(np.float32)
        wm = np.abs(WL.bf16_bits_to_f32(w)).astype(np.float64)
        alpha = float(np.float32(wm.max() / 2688.0))
        dq = float(np.float32(rng.uniform(100, 448)))
        m0, _, _ = R.round_block(w, alpha, dq)
        m, A, B = R.round_block(w, alpha, dq, h=h)
        assert np.array_equal(m, m0)                       # the rounding itself ignores the weights
        hd = h.astype(np.float64)
        assert A == pytest.approx(float(np.sum(hd * wm * m)), rel=1e-15)
        assert B == pytest.approx(float(np.sum(hd * m * m)), rel=1e-15)
        d = 0x70
        s = np.float64(np.float32(alpha)) * R.e4m3_decode(d)
        assert R.block_error(w, m, alpha, d, h=h) == pytest.approx(float(np.sum(hd * (wm - m * s) ** 2)), rel=1e-13)


def test_eq5_and_eq6_are_weighted_least_squares():
    """For fixed codes the objective is linear least squares in alpha (all blocks) and in one
    block's scale; Eq. 5 / Eq. 6 with weighted sums must equal a library solver's answer on the
    rows scaled by sqrt(h)."""
    rng = np.random.default_rng(1)
    nb = 48
    h = WL.column_weights(16 * nb, 11)
    blocks = [WL.f32_to_bf16_bits((rng.standard_t(4, 16) * 0.02).astype(np.float32)) for _ in range(nb)]
    alpha0 = float(np.float32(max(np.abs(WL.bf16_bits_to_f32(b)).max() for b in blocks) / 2688.0))
    num = den = 0.0
    xs, ys = [], []
    for i, b in enumerate(blocks):
        hb = h[16 * i:16 * i + 16]
        wm = np.abs(WL.bf16_bits_to_f32(b)).astype(np.float64)
        d = max(1, R.e4m3_encode(float(np.float32(wm.max() / (6 * alpha0)))))
        v = R.e4m3_decode(d)
        m, A, B = R.round_block(b, alpha0, v, h=hb)
        num += A * v
        den += B * v * v
        rt = np.sqrt(hb.astype(np.float64))
        xs.append(rt * m * v)
        ys.append(rt * wm)
        # Eq. 6 for this block, alpha fixed: scalar weighted least squares
        if B > 0:
            sol = np.linalg.lstsq((rt * m * alpha0)[:, None], rt * wm, rcond=None)[0][0]
            assert R.block_scale(A, B, alpha0, d) == pytest.approx(sol, rel=2e-6)
    sol = np.linalg.lstsq(np.concatenate(xs)[:, None], np.concatenate(ys), rcond=None)[0][0]
    assert num / den == pytest.approx(sol, rel=1e-12)


@pytest.mark.parametrize("rows,cols,seed,cfg,npkw", [
    (8, 64, 0, dict(), {}),
    (16, 256, 1, FAST, {}),
    (12, 320, 2, dict(max_iters=2, early_stop_rel=0.0, n_dq=4, n_beta=5, beta_step_pct=3), {}),
    (6, 512, 3, dict(max_iters=3, n_dq=2, n_beta=1, flags=R.FLAG_COUPLED_SCALE), dict(coupled_scale=True)),
])
def test_c_oracle_equals_numpy_restatement_with_weights(rows, cols, seed, cfg, npkw):
    w = WL.small_case(rows, cols, seed, outlier_entry_frac=0.005, outlier_scale=40.0)
    h = WL.column_weights(cols, seed, zero_frac=0.05)
    a = R.quantize(w, R.RefCfg(**cfg), h=h)
    kw = {k: v for k, v in cfg.items() if k != "flags"}
    b = N.quantize(w, h=h, **kw, **npkw)
    assert a.status == 0
    assert a.iters_run == b["iters_run"] and a.alpha == b["alpha"]
    assert np.array_equal(a.packed, b["packed"]) and np.array_equal(a.scales, b["scales"])
    assert np.allclose(a.trace_sse, b["trace_sse"], rtol=1e-12, atol=0)


def test_reported_error_is_the_true_weighted_error_and_beats_the_unweighted_run():
    w = WL.small_case(32, 512, 9, outlier_cols_frac=0.01, outlier_scale=20.0)
    h = WL.column_weights(512, 9)
    wf = WL.bf16_bits_to_f32(w).astype(np.float64)
    hd = h.astype(np.float64)[None, :]
    res_w = R.quantize(w, R.RefCfg(), h=h)
    res_u = R.quantize(w, R.RefCfg())
    err_w = float(np.sum(hd * (wf - dequant(res_w)) ** 2))
    err_u = float(np.sum(hd * (wf - dequant(res_u)) ** 2))
    assert res_w.trace_sse[-1] == pytest.approx(err_w, rel=1e-10)
    assert res_w.sumsq == pytest.approx(float(np.sum(hd * wf ** 2)), rel=1e-12)
    sse, ss = R.dequant_error(w, res_w.packed, res_w.scales, res_w.alpha, h=h)
    assert sse == pytest.approx(err_w, rel=1e-12) and ss == pytest.approx(res_w.sumsq, rel=1e-12)
    # optimising the weighted error must do better on it than optimising the plain one, and
    # better than the max-based start
    assert err_w < err_u
    assert res_w.trace_sse[-1] < res_w.trace_sse[0]


def test_zero_weight_columns_do_not_steer_the_scales():
    """Changing W in columns of zero weight (without touching a block's or the tensor's maximum)
    leaves alpha and every block scale where they were; only those columns' codes move."""
    rng = np.random.default_rng(4)
    w = WL.small_case(8, 256, 21)
    h = WL.column_weights(256, 21)
    dead = np.arange(3, 256, 16)                           # one column per block
    h[dead] = 0.0
    wf = WL.bf16_bits_to_f32(w)
    w2 = w.copy()
    bmax = np.abs(wf).reshape(8, 16, 16).max(axis=2)        # per block
    repl = (rng.uniform(0.0, 0.9, (8, 16)) * bmax).astype(np.float32)
    # keep every block's maximum in a live column
    for r in range(8):
        for b in range(16):
            if np.abs(wf[r, 16 * b + 3]) == bmax[r, b]:
                repl[r, b] = wf[r, 16 * b + 3]
    w2[:, dead] = WL.f32_to_bf16_bits(repl)
    a = R.quantize(w, R.RefCfg(**FAST), h=h)
    b = R.quantize(w2, R.RefCfg(**FAST), h=h)
    assert a.alpha == b.alpha and np.array_equal(a.scales, b.scales)
    live = np.setdiff1d(np.arange(256), dead)
    ca = np.stack([a.packed & 0xF, a.packed >> 4], -1).reshape(8, -1)
    cb = np.stack([b.packed & 0xF, b.packed >> 4], -1).reshape(8, -1)
    assert np.array_equal(ca[:, live], cb[:, live])
    assert np.array_equal(a.trace_sse, b.trace_sse)


def test_search_winner_is_the_weighted_brute_force_argmin():
    """One iteration from the max-based start on a one-block tensor: the stored scale and codes
    must be the argmin, over the whole candidate grid enumerated here, of the weighted error."""
    rng = np.random.default_rng(6)
    vals = e4m3_vals()
    for trial in range(30):
        w = WL.f32_to_bf16_bits((rng.standard_t(4, (1, 16)) * 0.05).astype(np.float32))
        h = rng.uniform(0.05, 20.0, 16).astype(np.float32)
        cfg = R.RefCfg(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=21, beta_step_pct=2)
        res = R.quantize(w, cfg, h=h)
        wm = np.abs(WL.bf16_bits_to_f32(w[0])).astype(np.float64)
        hd = h.astype(np.float64)
        # replay the iteration's inputs from the definitions
        alpha0 = np.float32(np.float32(wm.max()) / np.float32(2688.0))
        d0 = max(1, R.e4m3_encode(float(np.float32(wm.max()) / np.float32(alpha0 * np.float32(6.0)))))
        m0, A0, B0 = R.round_block(w[0], float(alpha0), R.e4m3_decode(d0), h=h)
        alpha1 = np.float32((A0 * vals[d0]) / (B0 * vals[d0] ** 2))
        assert res.alpha == float(alpha1)
        center = np.float32(np.float32(A0) / np.float32(alpha1 * np.float32(B0)))
        cf = int(np.searchsorted(vals, float(center), side="right") - 1)
        best = (np.inf, None, None)
        for k in range(21):
            beta = np.float32((100.0 + (k - 10) * 2) / 100.0)
            s = np.float32(alpha1 * np.float32(center * beta))
            x = (wm.astype(np.float32) * np.float32(np.float32(1.0) / s)).astype(np.float32)
            m = np.array([R.e2m1_round(float(v)) for v in x])
            for d in (cf, cf + 1):
                d = min(max(d, 1), 0x7E)
                L = float(np.sum(hd * (wm - m * (np.float64(alpha1) * vals[d])) ** 2))
                if L < best[0] * (1 - 1e-12):
                    best = (L, d, m)
        if res.tie_flags[0, 0]:
            continue
        assert res.scales[0, 0] == best[1]
        lo, hi = res.packed[0] & 0xF, res.packed[0] >> 4
        codes = np.stack([lo, hi], -1).reshape(-1) & 7
        assert np.array_equal(GRID[codes], best[2])
        assert res.trace_sse[-1] == pytest.approx(best[0], rel=1e-10)


def test_bad_weights_are_reported():
    w = WL.small_case(4, 64, 0)
    for bad in (-1.0, np.inf, np.nan, 2.0 ** -30, 2.0 ** 30):
        h = np.ones(64, np.float32)
        h[17] = bad
        assert R.quantize(w, R.RefCfg(**FAST), h=h).status & R.STATUS_BAD_WEIGHT
    h = np.ones(64, np.float32)
    h[17] = 0.0
    assert R.quantize(w, R.RefCfg(**FAST), h=h).status == 0
