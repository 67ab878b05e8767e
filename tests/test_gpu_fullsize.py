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


# ---- the launch shape the benchmark times: one batched call, CTAs walking from tensor to tensor

def _batch_against_oracle(wl_name, ws, names, cfg, ref_cfg):
    got = P.run_gpu_batch(ws, cfg)
    for name, w, g in zip(names, ws, got):          # the oracle per tensor, so that a failure names it
        g.buffers = None
        rep = P.assert_parity(g, R.quantize(w, ref_cfg))
        print(wl_name, name, rep)


def test_config4_whole_layer_in_one_batched_call_paper_preset_and_single_pass():
    """All seven tensors of the Llama-3-70B-shaped layer through soar_quantize_batch, exactly as
    bench.py launches them, every tensor element by element against the oracle."""
    wl = WL.config4()
    ws = [WL.generate(wl, i) for i in range(len(wl.tensors))]
    names = [t.name for t in wl.tensors]
    cfg, ref_cfg = P.cfg_pair()
    _batch_against_oracle("config4 paper", ws, names, cfg, ref_cfg)
    torch.cuda.empty_cache()
    cfg, ref_cfg = P.cfg_pair(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1)
    _batch_against_oracle("config4 single pass", ws, names, cfg, ref_cfg)


@pytest.mark.parametrize("cfgkw", [
    dict(),                                                   # the paper's preset
    dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1),  # single pass
    dict(max_iters=0),                                        # Eq. 1-3 only
    dict(max_iters=2, early_stop_rel=0.0, n_dq=4, n_beta=1),  # several codes on one rounding
])
def test_batch_of_mid_size_tensors_hands_over_inside_every_kernel(cfgkw):
    """Nineteen matrices, sixteen of them several hundred tiles long: the first launch group has
    thousands of tiles, far more than any kernel's grid, so in every pass (forward and backward)
    each CTA leaves one matrix and enters the next in mid-sequence.  Same bytes as separate calls,
    and the oracle's."""
    shapes = [(520 + 24 * i, 4096) if i % 2 == 0 else (1040 + 8 * i, 2064) for i in range(16)] + \
             [(1, 16), (300, 4096), (5, 48)]
    ws = [WL.small_case(r, c, 700 + i, dist=("laplace" if i % 3 == 0 else "student_t4"),
                        outlier_entry_frac=0.002 * (i % 2), outlier_scale=40.0) for i, (r, c) in enumerate(shapes)]
    ws.insert(3, WL.small_case(1, 16, 777))                  # a one-block matrix between two long ones
    ws[7] = np.zeros_like(ws[7])                             # an all-zero matrix in mid-sequence
    cfg, ref_cfg = P.cfg_pair(**cfgkw)
    lds = [w.shape[1] + (40 if i == 5 else 0) for i, w in enumerate(ws)]
    got = P.run_gpu_batch(ws, cfg, lds)
    for i, (w, g) in enumerate(zip(ws, got)):
        one = P.run_gpu(w, cfg, lds[i])
        assert g.result.status == one.result.status and g.result.iters_run == one.result.iters_run, i
        assert np.array_equal(g.packed, one.packed) and np.array_equal(g.scales, one.scales), i
        assert g.alpha == one.alpha, i
        assert g.result.sse == pytest.approx(one.result.sse, rel=1e-12), i
        if g.result.status == 0:
            P.assert_parity(g, R.quantize(w, ref_cfg))
        else:
            assert g.result.status == api.STATUS_ZERO_TENSOR and not g.scales.any()


def test_config3_whole_layer_batched_and_tensors_of_the_first_and_last_layer():
    """Layer 17 of the 36-layer Qwen3-8B-shaped model through the batched call, all seven tensors against
    the oracle; k of layer 0 and of layer 35 (each layer has its own seed) through single calls."""
    wl = WL.config3_layer(17)
    ws = [WL.generate(wl, i) for i in range(len(wl.tensors))]
    cfg, ref_cfg = P.cfg_pair()
    _batch_against_oracle(wl.name, ws, [t.name for t in wl.tensors], cfg, ref_cfg)
    for layer in (0, 35):
        wl = WL.config3_layer(layer)
        w = WL.generate(wl, 1)
        print(wl.name, wl.tensors[1].name, P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg)))


def test_config5_candidate_sweep_points_with_fifteen_iterations():
    """The sweep of config 5 at T = 15 (early stop off), on the first 1024 rows."""
    w = WL.generate(WL.config5(), 0, 0, 1024)
    for pairs in (1, 4, 8, 16, 32):
        n_dq = min(2, pairs)
        cfg, ref_cfg = P.cfg_pair(max_iters=15, early_stop_rel=0.0, n_dq=n_dq, n_beta=pairs // n_dq)
        rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
        print("config5 rows 0..1023, T = 15, pairs", pairs, rep)
