"""Pins for the oracle's number formats (Sec. 3.1 of the paper: E2M1 elements, E4M3 block
scales).  Each check compares the C oracle with something it does not contain: the
constants the paper prints, a brute-force nearest-grid search, or a library cast."""
import itertools

import ml_dtypes
import numpy as np
import pytest
import torch

from oracle import soar_ref as R


def read_golden(golden_dir):
    out = {}
    with open(f"{golden_dir}/nvfp4_constants.txt") as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = [s.strip() for s in line.split("=")]
                out[k] = v
    return out


def test_constants_match_paper(golden_dir):
    g = read_golden(golden_dir)
    grid = [float(v) for v in g["e2m1_grid"].split()]
    # every grid value is a fixed point of the rounding and maps to consecutive codes
    for i, v in enumerate(grid):
        assert R.e2m1_round(v) == v
        assert R.e2m1_code(v) == i
    assert R.e2m1_round(1e9) == float(g["m_fp4"])
    assert R.e4m3_decode(0x7E) == float(g["m_fp8"])
    assert R.e4m3_encode(1e9) == 0x7E
    cfg = R.RefCfg()
    assert cfg.max_iters == int(g["max_iters"])
    assert cfg.early_stop_rel == float(g["early_stop_rel"])
    assert cfg.n_dq == int(g["n_dq"])
    assert R.beta(0, cfg.n_beta, cfg.beta_step_pct) == np.float32(float(g["beta_min"]))
    assert R.beta(cfg.n_beta - 1, cfg.n_beta, cfg.beta_step_pct) == np.float32(float(g["beta_max"]))
    steps = [R.beta(k, cfg.n_beta, cfg.beta_step_pct) for k in range(cfg.n_beta)]
    assert np.allclose(np.diff(steps), float(g["beta_step"]), atol=1e-6)
    assert R.beta(cfg.n_beta // 2, cfg.n_beta, cfg.beta_step_pct) == 1.0


def test_e2m1_round_is_nearest_grid_point(golden_dir):
    grid = np.array([float(v) for v in read_golden(golden_dir)["e2m1_grid"].split()])
    xs = np.concatenate([np.linspace(0, 7.5, 30001), np.float32(np.random.default_rng(0).random(20000) * 8)])
    for x in xs:
        d = np.abs(grid - x)
        best = d.min()
        winners = grid[d == best]
        got = R.e2m1_round(float(x))
        if len(winners) == 1:
            assert got == winners[0], x
        else:  # exact midpoint: the neighbour with the even code wins
            even = [w for w in winners if R.e2m1_code(w) % 2 == 0]
            assert got == even[0], x


def test_e2m1_midpoints_half_even():
    # midpoints of the grid and the value they must round to (even code)
    expect = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for x, m in expect.items():
        assert R.e2m1_round(x) == m
        lo = float(np.nextafter(np.float32(x), np.float32(0)))
        hi = float(np.nextafter(np.float32(x), np.float32(10)))
        assert R.e2m1_round(lo) < R.e2m1_round(hi)
        assert R.e2m1_round(lo) <= m <= R.e2m1_round(hi)


def test_e2m1_matches_library_cast():
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        rng.random(50000).astype(np.float32) * 6.0,
        np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 0.0], np.float32),
    ])
    xs = np.concatenate([xs, np.nextafter(xs, np.float32(-1)).clip(0), np.nextafter(xs, np.float32(10)).clip(0, 6)])
    lib = xs.astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    got = np.array([R.e2m1_round(float(x)) for x in xs])
    assert np.array_equal(lib, got)


def test_e4m3_decode_all_codes():
    codes = np.arange(0x7F, dtype=np.uint8)
    lib = codes.view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    tor = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = np.array([R.e4m3_decode(int(c)) for c in codes])
    assert np.array_equal(lib, got)
    assert np.array_equal(tor, got)
    assert np.all(np.diff(got) > 0)          # positive codes are monotone in value
    assert got[1] == 2.0 ** -9 and got[8] == 2.0 ** -6 and got[0x7E] == 448.0


def test_e4m3_encode_round_trip_and_midpoints():
    vals = [R.e4m3_decode(c) for c in range(0x7F)]
    for c, v in enumerate(vals):
        assert R.e4m3_encode(v) == c
    for c in range(0x7E):
        mid = 0.5 * (vals[c] + vals[c + 1])           # exact in binary32
        assert float(np.float32(mid)) == mid
        even = c if c % 2 == 0 else c + 1
        assert R.e4m3_encode(mid) == even
        assert R.e4m3_encode(float(np.nextafter(np.float32(mid), np.float32(0)))) == c
        assert R.e4m3_encode(float(np.nextafter(np.float32(mid), np.float32(1e9)))) == c + 1


def test_e4m3_encode_matches_library_casts():
    rng = np.random.default_rng(2)
    v = np.exp(rng.uniform(np.log(2.0 ** -12), np.log(448.0), 40000)).astype(np.float32)
    lib = v.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    tor = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([R.e4m3_encode(float(x)) for x in v], np.uint8)
    assert np.array_equal(lib, got)
    assert np.array_equal(tor, got)


def test_e4m3_saturates_at_448():
    for v in (448.0, 449.0, 463.9, 464.0, 480.0, 1e4, 3e38):
        assert R.e4m3_encode(v) == 0x7E
    assert R.e4m3_encode(0.0) == 0
    assert R.e4m3_encode(2.0 ** -11) == 0        # below half the smallest subnormal
    assert R.e4m3_encode(2.0 ** -10) == 0        # tie between 0 and 2^-9 goes to the even code 0
    assert R.e4m3_encode(float(np.nextafter(np.float32(2.0 ** -10), np.float32(1)))) == 1


def test_bf16_decode_is_exact():
    lib = R.lib()
    for bits in itertools.chain(range(0, 0x7F80, 97), [0x3F80, 0x0001, 0x7F7F]):
        f = np.array([bits], np.uint16).view(ml_dtypes.bfloat16).astype(np.float32)[0]
        assert lib.soar_ref_bf16_to_f32(bits) == f
