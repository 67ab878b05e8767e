"""Seeded random sweep of shapes, settings, magnitudes and weights: the CUDA path against the
oracle on cases nobody picked by hand (tiny and huge tensor maxima, blocks far below the tensor
maximum, odd strides, wide candidate windows, extreme column weights)."""
import numpy as np
import pytest
import torch

from oracle import soar_ref as R
from paper_2605_12245_b200 import api
from paper_2605_12245_b200 import workloads as WL
from tests import parity as P

pytestmark = pytest.mark.gpu


def random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    rows = int(rng.integers(1, 70))
    cols = 16 * int(rng.integers(1, 40))
    ld = cols + 8 * int(rng.integers(0, 3))
    dist = ["student_t4", "laplace", "gauss_t2mix"][seed % 3]
    w = WL.small_case(rows, cols, seed, dist=dist, outlier_entry_frac=float(rng.choice([0.0, 0.01, 0.05])),
                      outlier_scale=float(rng.choice([10.0, 100.0, 1000.0])))
    f = WL.bf16_bits_to_f32(w)
    # tensor-wide magnitude anywhere in the accepted range, some rows pushed far below the maximum,
    # some blocks zeroed
    f = f * np.float32(2.0 ** int(rng.integers(-80, 80)))
    low = rng.random(rows) < 0.2
    f[low] *= np.float32(2.0 ** -int(rng.integers(8, 30)))
    zero_blocks = rng.random((rows, cols // 16)) < 0.05
    f = np.where(np.repeat(zero_blocks, 16, axis=1), np.float32(0.0), f)
    w = WL.f32_to_bf16_bits(f.astype(np.float32))
    cfgkw = dict(max_iters=int(rng.integers(0, 4)), early_stop_rel=float(rng.choice([0.0, 1e-3])),
                 n_dq=int(rng.choice([1, 2, 2, 2, 3, 4])), n_beta=int(rng.choice([1, 1, 3, 7, 21, 101])),
                 beta_step_pct=int(rng.choice([1, 2, 5])))
    if 100 - (cfgkw["n_beta"] // 2) * cfgkw["beta_step_pct"] <= 0:
        cfgkw["beta_step_pct"] = 1
    if seed % 5 == 0:
        cfgkw["flags"] = R.FLAG_COUPLED_SCALE
    elif seed % 7 == 0:
        cfgkw["flags"] = R.FLAG_KEEP_ALPHA | R.FLAG_KEEP_BLOCK_SCALE
    h = None
    if seed % 2:
        h = np.exp2(rng.uniform(-20, 20, cols) if seed % 4 == 1 else rng.normal(0, 2, cols)).astype(np.float32)
        h = np.clip(h, 2.0 ** -20, 2.0 ** 20)
        h[rng.random(cols) < 0.1] = 0.0
    return w, ld, cfgkw, h


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("SOAR_FUZZ_CASES", "96"))))
def test_random_case(seed):
    w, ld, cfgkw, h = random_case(seed)
    if not w.any():
        pytest.skip("all-zero draw")
    cfg, ref_cfg = P.cfg_pair(**cfgkw)
    if h is None:
        gpu = P.run_gpu(w, cfg, ld)
    else:
        W = P.to_device(w, ld)
        out = api.soar_quantize_weighted(W, torch.from_numpy(h).cuda(), cfg)
        torch.cuda.synchronize()
        gpu = P.GpuOut(out.packed.cpu().numpy(), out.scales.cpu().numpy(), float(out.alpha.cpu()[0]),
                       out.read_result(), out)
    ref = R.quantize(w, ref_cfg, h=h)
    assert ref.status == 0
    # Tiny tensors, and weights that leave one element in charge of a block's error, make flagged near-ties
    # common; a few of them decided the other way are already far above 0.01 % of the blocks.  Outside the
    # flagged blocks nothing may differ, and the total error must still agree to 1e-5.
    ties = int(ref.tie_flags.sum())
    P.assert_parity(gpu, ref, mismatch_cap=max(2, ties // 10))
