"""Pins for the oracle's stand-alone arms of the paper's ablation: Sec. 3.2 alone (closed-form
scale updates with one block scale for both quantization and dequantization) and Sec. 3.3
alone (the decoupled search around the max-based start, no closed-form updates)."""
import ml_dtypes
import numpy as np
import pytest

from oracle import soar_np as N
from oracle import soar_ref as R
from paper_2605_12245_b200 import workloads as WL

GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
E4M3 = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)

CJSO = dict(max_iters=4, early_stop_rel=0.0, n_dq=1, n_beta=1)
DSS = dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=101)


def magnitudes(packed):
    lo, hi = packed & 7, (packed >> 4) & 7
    return GRID[np.stack([lo, hi], axis=-1).reshape(packed.shape[0], -1)]


def block_errors(w, packed, scales, alpha):
    a = np.abs(WL.bf16_bits_to_f32(w).astype(np.float64))
    s = np.repeat(E4M3[scales], 16, axis=1) * alpha
    e = a - magnitudes(packed) * s
    return (e * e).reshape(w.shape[0], -1, 16).sum(axis=2)


@pytest.mark.parametrize("rows,cols,seed,kw", [
    (8, 64, 0, {}),
    (12, 320, 2, dict(dist="laplace", outlier_cols_frac=0.01, outlier_scale=20.0)),
    (16, 256, 1, dict(outlier_entry_frac=0.01, outlier_scale=50.0)),
])
@pytest.mark.parametrize("cfg,flags,npkw", [
    (CJSO, R.FLAG_COUPLED_SCALE, dict(coupled_scale=True)),
    (dict(CJSO, n_dq=2, n_beta=3, beta_step_pct=5), R.FLAG_COUPLED_SCALE, dict(coupled_scale=True)),
    (DSS, R.FLAG_KEEP_ALPHA | R.FLAG_KEEP_BLOCK_SCALE, dict(keep_alpha=True, keep_block_scale=True)),
    (dict(DSS, max_iters=2, n_beta=7, beta_step_pct=4), R.FLAG_KEEP_ALPHA | R.FLAG_KEEP_BLOCK_SCALE,
     dict(keep_alpha=True, keep_block_scale=True)),
])
def test_c_oracle_equals_numpy_restatement_on_the_arms(rows, cols, seed, kw, cfg, flags, npkw):
    w = WL.small_case(rows, cols, seed, **kw)
    a = R.quantize(w, R.RefCfg(flags=flags, **cfg))
    b = N.quantize(w, **cfg, **npkw)
    assert a.iters_run == b["iters_run"] and a.alpha == b["alpha"]
    assert np.array_equal(a.packed, b["packed"]) and np.array_equal(a.scales, b["scales"])
    assert np.allclose(a.trace_sse, b["trace_sse"], rtol=1e-12, atol=0)


def test_coupled_arm_stores_the_scale_it_quantized_with():
    """Sec. 3.2 alone: after any number of updates the stored E4M3 scale is the quantization
    scale, so re-rounding W by alpha * stored scale (Eq. 2, written out here) gives the codes."""
    w = WL.small_case(24, 256, 5, outlier_entry_frac=0.01, outlier_scale=30.0)
    r = R.quantize(w, R.RefCfg(flags=R.FLAG_COUPLED_SCALE, **CJSO))
    a = np.abs(WL.bf16_bits_to_f32(w))
    s = (np.float32(r.alpha) * np.repeat(E4M3[r.scales].astype(np.float32), 16, axis=1)).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        x = (a * (np.float32(1.0) / s).astype(np.float32)).astype(np.float32)
    want = np.minimum(x, np.float32(6)).astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    live = np.repeat(r.scales != 0, 16, axis=1)
    assert np.array_equal(np.where(live, want, 0.0), magnitudes(r.packed))
    # and the global scale moved away from Eq. 1's (Eq. 5 ran)
    assert r.trace_alpha[1] != r.trace_alpha[0]


def test_search_arm_keeps_alpha_and_never_worsens_a_block():
    """Sec. 3.3 alone: alpha stays Eq. 1's; beta = 1 with the stored scale is among the
    candidates of every block, so no block ends above its max-based error."""
    w = WL.small_case(32, 512, 9, dist="gauss_t2mix")
    base = R.quantize(w, R.RefCfg(max_iters=0))
    r = R.quantize(w, R.RefCfg(flags=R.FLAG_KEEP_ALPHA | R.FLAG_KEEP_BLOCK_SCALE, **DSS))
    assert r.alpha == base.alpha and np.all(r.trace_alpha == base.alpha)
    e0 = block_errors(w, base.packed, base.scales, base.alpha)
    e1 = block_errors(w, r.packed, r.scales, r.alpha)
    assert np.all(e1 <= e0 * (1 + 1e-12))
    assert e1.sum() < 0.97 * e0.sum()                # and the search does gain overall
    # the stored scale moved by at most one code upward (candidates: the stored code and the next)
    d = r.scales.astype(int) - base.scales.astype(int)
    assert d.min() >= 0 and d.max() <= 1


def test_full_method_beats_both_arms_on_a_synthetic_tensor():
    """The ordering the paper reports for its ablation (Table 4, Fig. 4), on synthetic weights:
    full SOAR ends at or below each stand-alone arm, and each arm at or below plain NVFP4."""
    w = WL.small_case(64, 512, 13, outlier_cols_frac=0.004, outlier_scale=20.0)
    rtn = R.quantize(w, R.RefCfg(max_iters=0)).trace_sse[-1]
    cjso = R.quantize(w, R.RefCfg(flags=R.FLAG_COUPLED_SCALE, max_iters=15, early_stop_rel=1e-3, n_dq=1, n_beta=1))
    dss = R.quantize(w, R.RefCfg(flags=R.FLAG_KEEP_ALPHA | R.FLAG_KEEP_BLOCK_SCALE, **DSS)).trace_sse[-1]
    full = R.quantize(w, R.RefCfg()).trace_sse[-1]
    assert full <= min(cjso.trace_sse.min(), dss) and max(cjso.trace_sse.min(), dss) <= rtn


def test_two_coupled_candidates_end_where_the_full_search_ends():
    """An observation on synthetic weights, not a claim of the paper: for a fixed dequantization
    scale the best codes are the nearest ones under that same scale, so trying each of the two
    bracketing E4M3 codes with itself as quantization scale (2 candidates per block) reaches the
    error the 202-pair search reaches."""
    for seed, kw in ((13, dict(outlier_cols_frac=0.004, outlier_scale=20.0)),
                     (5, dict(dist="laplace", outlier_entry_frac=0.0005, outlier_scale=50.0)),
                     (7, dict(dist="gauss_t2mix"))):
        w = WL.small_case(96, 1024, seed, **kw)
        full = R.quantize(w, R.RefCfg()).trace_sse[-1]
        pair = R.quantize(w, R.RefCfg(flags=R.FLAG_COUPLED_SCALE, n_dq=2, n_beta=1)).trace_sse[-1]
        assert pair <= full * 1.003
