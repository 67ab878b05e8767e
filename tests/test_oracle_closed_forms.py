"""Pins for the oracle's closed-form steps (Eq. 5 and Eq. 6 of the paper) and for the
block-level search (Eq. 8): each is compared with a brute-force minimisation written here
from the objective of Eq. 4, not with the oracle's own formula."""
import numpy as np
import pytest

from oracle import soar_ref as R
from paper_2605_12245_b200 import workloads as WL

GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def bf16_block(rng, scale=0.02, n=16):
    return WL.f32_to_bf16_bits((rng.standard_t(4, n) * scale).astype(np.float32))


def objective(wmag, m, alpha, delta):
    """Eq. 4 for one block, in binary64: sum (|W| - m * alpha*delta)^2."""
    return float(np.sum((wmag - m * (alpha * delta)) ** 2))


def test_round_block_sums_match_definition():
    rng = np.random.default_rng(0)
    for _ in range(50):
        w = bf16_block(rng)
        wm = np.abs(WL.bf16_bits_to_f32(w)).astype(np.float64)
        alpha = float(np.float32(wm.max() / 2688.0))
        dq = float(np.float32(rng.uniform(50, 448)))
        m, A, B = R.round_block(w, alpha, dq)
        assert set(np.unique(m)) <= set(GRID)
        assert A == pytest.approx(float(np.sum(wm * m)), rel=1e-15)
        assert B == float(np.sum(m * m))
        # nearest grid point of |W|/(alpha*dq), up to the binary32 rounding of the quotient
        x = wm / (alpha * dq)
        near = GRID[np.argmin(np.abs(GRID[None, :] - np.minimum(x, 6.0)[:, None]), axis=1)]
        clear = np.min(np.abs(np.minimum(x, 6.0)[:, None] - np.array([.25, .75, 1.25, 1.75, 2.5, 3.5, 5.0])[None, :]), axis=1) > 1e-5
        assert np.array_equal(near[clear], m[clear])


def test_eq5_global_scale_minimises_objective():
    """With codes and block scales fixed, alpha* of Eq. 5 is the minimiser of Eq. 4."""
    rng = np.random.default_rng(1)
    blocks = [bf16_block(rng) for _ in range(64)]
    alpha0 = float(np.float32(max(np.abs(WL.bf16_bits_to_f32(b)).max() for b in blocks) / 2688.0))
    ms, ds, wms = [], [], []
    num = den = 0.0
    for b in blocks:
        wm = np.abs(WL.bf16_bits_to_f32(b)).astype(np.float64)
        d = max(1, R.e4m3_encode(float(np.float32(wm.max() / (6 * alpha0)))))
        m, A, B = R.round_block(b, alpha0, R.e4m3_decode(d))
        v = R.e4m3_decode(d)
        num += A * v
        den += B * v * v
        ms.append(m); ds.append(v); wms.append(wm)
    a_star = num / den

    def total(a):
        return sum(objective(wm, m, a, v) for wm, m, v in zip(wms, ms, ds))

    base = total(a_star)
    for rel in (1e-3, 1e-4, -1e-4, -1e-3, 0.05, -0.05):
        assert total(a_star * (1 + rel)) > base
    # stationarity by central difference
    h = a_star * 1e-6
    g = (total(a_star + h) - total(a_star - h)) / (2 * h)
    curv = (total(a_star + h) - 2 * base + total(a_star - h)) / h ** 2
    assert abs(g) < 1e-6 * curv * a_star
    # and against a dense scan of alpha
    scan = np.linspace(0.8, 1.2, 4001) * a_star
    assert abs(scan[np.argmin([total(a) for a in scan])] / a_star - 1) < 2e-4


def test_eq6_block_scale_and_e4m3_bracket():
    """With codes and alpha fixed, Eq. 6 minimises the block objective over real scales,
    and over all E4M3 codes the best one is one of the two codes bracketing Eq. 6."""
    rng = np.random.default_rng(2)
    vals = np.array([R.e4m3_decode(c) for c in range(1, 0x7F)])
    for _ in range(200):
        w = bf16_block(rng, scale=10 ** rng.uniform(-3, 0))
        wm = np.abs(WL.bf16_bits_to_f32(w)).astype(np.float64)
        alpha = float(np.float32(wm.max() / 2688.0 * rng.uniform(0.5, 30)))
        dq = float(np.float32(wm.max() / (6 * alpha) * rng.uniform(0.6, 1.5)))
        m, A, B = R.round_block(w, alpha, dq)
        if B == 0:
            continue
        center = R.block_scale(A, B, alpha, 1)
        exact = A / (alpha * B)
        assert center == pytest.approx(exact, rel=3e-7)
        assert objective(wm, m, alpha, exact) <= objective(wm, m, alpha, exact * 1.001)
        assert objective(wm, m, alpha, exact) <= objective(wm, m, alpha, exact * 0.999)
        errs = np.array([objective(wm, m, alpha, v) for v in vals])
        best_code = 1 + int(np.argmin(errs))
        cands = R.dq_candidates(center, 2)
        assert best_code in cands, (center, best_code, cands)
        assert len(cands) <= 2 and all(1 <= c <= 0x7E for c in cands)
        if 2.0 ** -9 <= center < 448:
            assert R.e4m3_decode(cands[0]) <= center
            if len(cands) == 2:
                assert cands[1] == cands[0] + 1 and R.e4m3_decode(cands[1]) > center
        # the error the oracle reports for a code is the objective
        for c in cands:
            assert R.block_error(w, m, alpha, c) == pytest.approx(objective(wm, m, alpha, R.e4m3_decode(c)), rel=1e-12, abs=1e-300)


def test_dq_candidate_sets():
    assert R.dq_candidates(1.0, 2) == [0x38, 0x39]                # 1.0 is E4M3: {1.0, next above}
    assert R.dq_candidates(1.06, 2) == [0x38, 0x39]
    assert R.dq_candidates(1.0, 1) == [0x38]
    assert R.dq_candidates(1.07, 1) == [0x39]                     # nearest of 1.0 / 1.125
    assert R.dq_candidates(1.06, 4) == [0x37, 0x38, 0x39, 0x3A]
    assert R.dq_candidates(1e-9, 2) == [0x01]                     # below the smallest code
    assert R.dq_candidates(2.0 ** -9, 2) == [0x01, 0x02]
    assert R.dq_candidates(500.0, 2) == [0x7E]                    # above 448
    assert R.dq_candidates(447.0, 2) == [0x7D, 0x7E]
    assert R.dq_candidates(447.0, 4) == [0x7C, 0x7D, 0x7E]
    assert R.dq_candidates(1e-9, 1) == [0x01]


def test_search_winner_is_brute_force_argmin():
    """Eq. 8: enumerate every (beta, neighbour) pair here, with the objective written out,
    and compare with the block the oracle returns after one iteration on a 1-block tensor."""
    rng = np.random.default_rng(3)
    cfg = R.RefCfg(max_iters=1, early_stop_rel=0.0)
    for trial in range(40):
        w = bf16_block(rng, scale=10 ** rng.uniform(-3, 0)).reshape(1, 16)
        ref = R.quantize(w, cfg)
        wm = np.abs(WL.bf16_bits_to_f32(w[0])).astype(np.float64)
        # state before the iteration (Eq. 1)
        alpha0 = float(np.float32(np.float32(wm.max()) / np.float32(2688.0)))
        assert ref.trace_alpha[0] == alpha0
        d0 = R.e4m3_encode(float(np.float32(np.float32(wm.max()) / np.float32(np.float32(alpha0) * np.float32(6)))))
        m0, A0, B0 = R.round_block(w[0], alpha0, R.e4m3_decode(d0))
        v0 = R.e4m3_decode(d0)
        alpha1 = float(np.float32((A0 * v0) / (B0 * v0 * v0)))
        assert ref.trace_alpha[1] == alpha1
        center = R.block_scale(A0, B0, alpha1, d0)
        best = (np.inf, None, None)
        for k in range(cfg.n_beta):
            dq = float(np.float32(np.float32(center) * np.float32(R.beta(k, cfg.n_beta, 1))))
            m, _, _ = R.round_block(w[0], alpha1, dq)
            for c in R.dq_candidates(center, 2):
                L = objective(wm, m, alpha1, R.e4m3_decode(c))
                if L < best[0] * (1 - 1e-12):
                    best = (L, m.copy(), c)
        L, m, c = best
        assert ref.scales[0, 0] == c
        codes = np.concatenate([[b & 0xF, b >> 4] for b in ref.packed[0]])
        assert np.array_equal(GRID[codes & 7], m)
        assert ref.trace_sse[1] == pytest.approx(L, rel=1e-10)
        # never worse than beta = 1 with the nearest E4M3 code (that pair, or one at least as good, is in the grid)
        m1, _, _ = R.round_block(w[0], alpha1, center)
        near = R.dq_candidates(center, 1)[0]
        assert L <= objective(wm, m1, alpha1, R.e4m3_decode(near)) * (1 + 1e-12)
