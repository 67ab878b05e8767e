"""GPU parity at the benchmark's full tensor sizes, in the launch configuration bench.py times
(whole tensors, contiguous rows, persistent grids).  Where the CPU oracle finishes a whole
tensor in seconds the comparison is element by element; for the largest tensor the paper's
full candidate grid is checked through properties that hold at any size (the oracle's
error evaluation of the GPU's outputs equals the error the GPU reports; the search never ends
above its starting error), and the one-candidate shape is compared element by element."""
import math

import numpy as np
import pytest
import torch

from oracle import soar_ref as R
from paper_2605_12245_b200 import api
from paper_2605_12245_b200 import workloads as WL
from tests import parity as P

pytestmark = pytest.mark.gpu


def test_config1_whole_tensor_paper_preset():
    wl = WL.config1()
    w = WL.generate(wl, 0)
    cfg, ref_cfg = P.cfg_pair()
    rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
    print("config1:", rep)


@pytest.mark.parametrize("tensor", [1, 0])          # k (1024 x 8192), q (8192 x 8192) of the Llama-3-70B layer
def test_config4_whole_tensors_paper_preset(tensor):
    wl = WL.config4()
    w = WL.generate(wl, tensor)
    cfg, ref_cfg = P.cfg_pair()
    rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
    print(wl.tensors[tensor].name, rep)


def test_config2_whole_tensors_paper_preset():
    """The Qwen3-8B-shaped layer (outlier input columns x20): down (4096 x 12288, long rows) and v (1024 x 4096)."""
    wl = WL.config2()
    cfg, ref_cfg = P.cfg_pair()
    for tensor in (6, 2):
        w = WL.generate(wl, tensor)
        rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
        print(wl.tensors[tensor].name, rep)


def test_config3_last_layer_tensor_paper_preset():
    """Layer 35 of the 36-layer model (its own seed): o (4096 x 4096)."""
    wl = WL.config3_layer(35)
    w = WL.generate(wl, 3)
    cfg, ref_cfg = P.cfg_pair()
    rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
    print(wl.name, wl.tensors[3].name, rep)


def test_config5_distribution_candidate_sweep_points():
    """Config 5's Gaussian / Student-t(2) mix at the sweep's candidate counts, on the first 1024 rows of the
    28672 x 8192 matrix (the whole matrix takes the oracle minutes per point)."""
    w = WL.generate(WL.config5(), 0, 0, 1024)
    for pairs in (1, 4, 8, 16, 32):
        n_dq = min(2, pairs)
        cfg, ref_cfg = P.cfg_pair(max_iters=1, early_stop_rel=0.0, n_dq=n_dq, n_beta=pairs // n_dq)
        rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
        print("config5 rows 0..1023, pairs", pairs, rep)


def test_config4_whole_tensor_coupled_pair_preset():
    """q (8192 x 8192) with two coupled candidates per block: several HBM-bound iterations."""
    wl = WL.config4()
    w = WL.generate(wl, 0)
    cfg = api.soar_default_cfg(api.PRESET_COUPLED_PAIR)
    ref_cfg = R.RefCfg(n_dq=2, n_beta=1, flags=R.FLAG_COUPLED_SCALE)
    rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
    print("q, coupled pair:", rep)


def test_config4_largest_tensor():
    """gate: 28672 x 8192 (470 MB, several times the L2)."""
    wl = WL.config4()
    w = WL.generate(wl, 4)
    # one-candidate shape: whole-tensor comparison
    cfg, ref_cfg = P.cfg_pair(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1)
    gpu = P.run_gpu(w, cfg)
    rep = P.assert_parity(gpu, R.quantize(w, ref_cfg))
    print("gate, single pass:", rep)
    del gpu
    torch.cuda.empty_cache()
    # the paper's grid: properties
    cfg, _ = P.cfg_pair()
    gpu = P.run_gpu(w, cfg)
    res = gpu.result
    assert res.status == 0 and 1 <= res.iters_run <= 15
    sse, sumsq = R.dequant_error(w, gpu.packed, gpu.scales, gpu.alpha)     # oracle's Eq. 3-4 on the GPU's outputs
    assert res.sse == pytest.approx(sse, rel=1e-9)
    # the oracle adds 2.3e8 terms one after another, which costs it about 1e-10 of relative accuracy
    # at this size; an exactly rounded sum of the same squares pins the tighter figure
    assert res.sumsq == pytest.approx(sumsq, rel=1e-9)
    f = WL.bf16_bits_to_f32(w).astype(np.float64)
    assert res.sumsq == pytest.approx(math.fsum((f * f).sum(axis=1)), rel=1e-13)
    del f
    assert res.sse <= res.sse_init
    ts = np.array(res.trace_sse[: res.iters_run + 1])
    assert np.all(np.diff(ts)[:-1] < 0)                                     # every executed iteration but the last gained
    # sign bits of the codes are the inputs' sign bits
    lo, hi = (gpu.packed >> 3) & 1, (gpu.packed >> 7) & 1
    assert np.array_equal(lo, (w[:, 0::2] >> 15).astype(np.uint8))
    assert np.array_equal(hi, (w[:, 1::2] >> 15).astype(np.uint8))
    W = P.to_device(w)
    e = api.soar_dequant_error(W, gpu.buffers.packed, gpu.buffers.scales, gpu.buffers.alpha).cpu().numpy()
    assert e[0] == pytest.approx(sse, rel=1e-9) and e[1] == pytest.approx(res.sumsq, rel=1e-13)
