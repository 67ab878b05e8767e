"""GPU parity for the column-weighted objective (soar_quantize_weighted) against the CPU oracle,
element by element on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import soar_ref as R
from paper_2605_12245_b200 import api
from paper_2605_12245_b200 import workloads as WL
from tests import parity as P

pytestmark = pytest.mark.gpu


def run_weighted(w_bits, h, cfg, ld=None):
    W = P.to_device(w_bits, ld)
    hw = torch.from_numpy(np.ascontiguousarray(h, dtype=np.float32)).cuda()
    out = api.soar_quantize_weighted(W, hw, cfg)
    torch.cuda.synchronize()
    res = out.read_result()
    scales = out.scales.cpu().numpy() if out.scales is not None else None
    return P.GpuOut(out.packed.cpu().numpy(), scales, float(out.alpha.cpu()[0]), res, out), W, hw


@pytest.mark.parametrize("rows,cols,ld,seed,kw", [
    (64, 256, None, 0, {}),
    (257, 4096, None, 1, dict(outlier_entry_frac=0.002, outlier_scale=40.0)),   # several tiles, exact multiple
    (37, 1040, 1048, 2, dict(dist="laplace", outlier_cols_frac=0.01, outlier_scale=20.0)),   # ragged tail, padded rows
    (3, 16, 24, 3, {}),
])
@pytest.mark.parametrize("cfgkw", [
    dict(),                                                            # the paper's setting
    dict(max_iters=0),
    dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1),
    dict(max_iters=2, early_stop_rel=0.0, n_dq=4, n_beta=5, beta_step_pct=3),
    dict(max_iters=3, n_dq=2, n_beta=1, flags=R.FLAG_COUPLED_SCALE),
    dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=21, flags=R.FLAG_KEEP_ALPHA | R.FLAG_KEEP_BLOCK_SCALE),
])
def test_weighted_parity(rows, cols, ld, seed, kw, cfgkw):
    if rows * cols > 300_000 and cfgkw.get("n_beta", 101) * cfgkw.get("max_iters", 15) > 200 and cfgkw:
        pytest.skip("oracle time")
    w = WL.small_case(rows, cols, seed, **kw)
    h = WL.column_weights(cols, seed, zero_frac=0.02 if seed % 2 else 0.0)
    cfg, ref_cfg = P.cfg_pair(**cfgkw)
    gpu, _, _ = run_weighted(w, h, cfg, ld)
    ref = R.quantize(w, ref_cfg, h=h)
    rep = P.assert_parity(gpu, ref)
    assert rep.blocks == rows * cols // 16
    assert gpu.result.sumsq == pytest.approx(ref.sumsq, rel=1e-12)


def test_unit_weights_give_exactly_what_the_unweighted_entry_gives():
    w = WL.small_case(200, 2048, 11, outlier_entry_frac=0.001, outlier_scale=30.0)
    for cfgkw in (dict(), dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1)):
        cfg, _ = P.cfg_pair(**cfgkw)
        a = P.run_gpu(w, cfg)
        b, _, _ = run_weighted(w, np.ones(2048, np.float32), cfg)
        assert np.array_equal(a.packed, b.packed) and np.array_equal(a.scales, b.scales)
        assert a.alpha == b.alpha and a.result.iters_run == b.result.iters_run
        assert b.result.sse == pytest.approx(a.result.sse, rel=1e-9)
        assert b.result.sumsq == pytest.approx(a.result.sumsq, rel=1e-12)


def test_weighted_error_report_matches_an_independent_pass_over_the_outputs():
    w = WL.small_case(300, 16 * 33, 5)
    h = WL.column_weights(16 * 33, 5)
    for layout in (api.SCALES_LINEAR, api.SCALES_SWIZZLED):
        cfg = api.soar_default_cfg(api.PRESET_PAPER, scale_layout=layout)
        gpu, W, hw = run_weighted(w, h, cfg)
        sc = gpu.buffers.scales if layout == api.SCALES_LINEAR else gpu.buffers.scales_sw
        e = api.soar_dequant_error_weighted(W, hw, gpu.buffers.packed, sc, gpu.buffers.alpha, layout).cpu().numpy()
        assert e[0] == pytest.approx(gpu.result.sse, rel=1e-9)
        assert e[1] == pytest.approx(gpu.result.sumsq, rel=1e-12)
        if layout == api.SCALES_LINEAR:
            sse, ss = R.dequant_error(w, gpu.packed, gpu.scales, gpu.alpha, h=h)
            assert e[0] == pytest.approx(sse, rel=1e-12) and e[1] == pytest.approx(ss, rel=1e-12)


def test_swizzled_only_layout_and_padded_rows():
    w = WL.small_case(130, 16 * 5, 8)
    h = WL.column_weights(16 * 5, 8)
    lin = api.soar_default_cfg(api.PRESET_PAPER)
    both = api.soar_default_cfg(api.PRESET_PAPER, scale_layout=api.SCALES_SWIZZLED)
    a, _, _ = run_weighted(w, h, lin)
    b, W, hw = run_weighted(w, h, both, ld=16 * 5 + 8)
    assert np.array_equal(a.packed, b.packed) and a.alpha == b.alpha
    sw = b.buffers.scales_sw.cpu().numpy()
    rows, nbc = 130, 5
    ct = (nbc + 3) // 4
    for r in (0, 31, 32, 127, 128, 129):
        for c in range(nbc):
            tile = (r // 128) * ct + c // 4
            off = tile * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + c % 4
            assert sw[off] == a.scales[r, c]


def test_bad_weights_and_degenerate_inputs_are_reported():
    w = WL.small_case(16, 64, 0)
    cfg, ref_cfg = P.cfg_pair(max_iters=2, early_stop_rel=0.0, n_dq=2, n_beta=5)
    for bad in (-1.0, float("inf"), float("nan"), 2.0 ** -30, 2.0 ** 30):
        h = np.ones(64, np.float32)
        h[17] = bad
        gpu, _, _ = run_weighted(w, h, cfg)
        assert gpu.result.status & api.STATUS_BAD_WEIGHT
        assert gpu.result.iters_run == 0
    # all weights zero: nothing to optimise, every candidate ties, the first one wins on both sides
    h = np.zeros(64, np.float32)
    gpu, _, _ = run_weighted(w, h, cfg)
    ref = R.quantize(w, ref_cfg, h=h)
    assert gpu.result.status == 0 == ref.status
    assert np.array_equal(gpu.packed, ref.packed) and np.array_equal(gpu.scales, ref.scales)
    assert gpu.result.sse == 0.0 and gpu.result.sumsq == 0.0
    # zero tensor and non-finite input keep their statuses
    z = np.zeros((4, 32), np.uint16)
    gpu, _, _ = run_weighted(z, np.ones(32, np.float32), cfg)
    assert gpu.result.status == api.STATUS_ZERO_TENSOR and gpu.alpha == 1.0
    n = w.copy()
    n[3, 5] = 0x7FC0
    gpu, _, _ = run_weighted(n, np.ones(64, np.float32), cfg)
    assert gpu.result.status & api.STATUS_NONFINITE


def test_argument_errors_of_the_weighted_entry():
    cfg = api.soar_default_cfg(api.PRESET_PAPER)
    W = torch.zeros((16, 64), dtype=torch.bfloat16, device="cuda")
    h = torch.ones(64, dtype=torch.float32, device="cuda")
    out = api.alloc_buffers(16, 64, cfg, weighted=True)
    L = api.lib()
    import ctypes as C
    args = lambda **o: [o.get("W", W.data_ptr()), 16, 64, 64, o.get("h", h.data_ptr()), C.byref(cfg),  # noqa: E731
                        out.packed.data_ptr(), out.scales.data_ptr(), None, out.alpha.data_ptr(),
                        o.get("ws", out.workspace.data_ptr()), o.get("wsb", out.workspace.numel()),
                        out.result.data_ptr(), None]
    assert L.soar_quantize_weighted(*args(h=None)) == -1
    assert L.soar_quantize_weighted(*args(h=h.data_ptr() + 4)) == -2
    assert L.soar_quantize_weighted(*args(wsb=out.workspace.numel() - 1)) == -3
    assert L.soar_quantize_weighted(*args()) == 0
    torch.cuda.synchronize()
    assert api.soar_weighted_workspace_bytes(16, 64, cfg) == 2048 + 1024 + 256
    # the plain workspace is smaller than the weighted one: it must be refused
    small = api.alloc_buffers(16, 64, cfg)
    assert L.soar_quantize_weighted(*args(ws=small.workspace.data_ptr(), wsb=small.workspace.numel())) == -3


@pytest.mark.parametrize("tensor", [1, 0])          # k (1024 x 8192), q (8192 x 8192) of the Llama-3-70B layer
def test_full_size_tensors_under_the_weighted_objective(tensor):
    """Whole tensors of the benchmark's workload in the launch configuration bench.py times
    (--objective weighted), element by element against the oracle."""
    wl = WL.config4()
    w = WL.generate(wl, tensor)
    h = WL.column_weights(wl.tensors[tensor].cols, 1000 + tensor)
    cfg, ref_cfg = P.cfg_pair()
    gpu, W, hw = run_weighted(w, h, cfg)
    ref = R.quantize(w, ref_cfg, h=h)
    rep = P.assert_parity(gpu, ref)
    print(wl.tensors[tensor].name, "weighted:", rep)
    assert gpu.result.sumsq == pytest.approx(ref.sumsq, rel=1e-9)
    e = api.soar_dequant_error_weighted(W, hw, gpu.buffers.packed, gpu.buffers.scales, gpu.buffers.alpha).cpu().numpy()
    assert e[0] == pytest.approx(gpu.result.sse, rel=1e-9)


def test_host_pipeline_with_column_weights_returns_what_direct_calls_return():
    cfg = api.soar_default_cfg(api.PRESET_PAPER, max_iters=2, n_beta=11)
    shapes = [(64, 256), (130, 1040), (16, 64), (257, 512), (64, 256)]
    ws = [WL.small_case(r, c, 40 + i) for i, (r, c) in enumerate(shapes)]
    hs = [torch.from_numpy(WL.column_weights(c, 40 + i)).cuda() for i, (r, c) in enumerate(shapes)]
    pipe = api.HostPipeline(shapes, cfg, depth=2, weighted=True)
    hosts = []
    for w, (r, c) in zip(ws, shapes):
        hb = api.alloc_host_buffers(r, c, cfg)
        hb.W.copy_(torch.from_numpy(w.view(np.int16)).view(torch.bfloat16))
        hosts.append(hb)
    pipe.run(hosts, hs)
    pipe.run(hosts, hs)          # a second list right behind the first
    pipe.synchronize()
    for w, h, hb in zip(ws, hs, hosts):
        direct = api.soar_quantize_weighted(P.to_device(w), h, cfg)
        torch.cuda.synchronize()
        assert np.array_equal(hb.packed.numpy(), direct.packed.cpu().numpy())
        assert np.array_equal(hb.scales.numpy(), direct.scales.cpu().numpy())
        assert float(hb.alpha[0]) == float(direct.alpha.cpu()[0])
        assert hb.read_result().iters_run == direct.read_result().iters_run
    with pytest.raises(api.SoarError):
        api.HostPipeline(shapes, cfg, depth=2).run(hosts, hs)


def test_the_weighted_call_and_the_staged_calls_replay_from_a_cuda_graph():
    """Neither entry point synchronizes or allocates: both can be captured once and replayed."""
    w = WL.small_case(128, 2048, 83, outlier_cols_frac=0.002, outlier_scale=20.0)
    h = WL.column_weights(2048, 83)
    cfg, ref_cfg = P.cfg_pair()
    W = P.to_device(w)
    hw = torch.from_numpy(h).cuda()
    side = torch.cuda.Stream()
    # weighted objective
    out = api.alloc_buffers(*w.shape, cfg, weighted=True)
    api.soar_quantize_weighted(W, hw, cfg, out, side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        api.soar_quantize_weighted(W, hw, cfg, out, side)
    out.packed.zero_(); out.scales.zero_(); out.alpha.zero_()
    g.replay()
    torch.cuda.synchronize()
    gpu = P.GpuOut(out.packed.cpu().numpy(), out.scales.cpu().numpy(), float(out.alpha.cpu()[0]),
                   out.read_result(), out)
    P.assert_parity(gpu, R.quantize(w, ref_cfg, h=h))
    # the stages of the plain call, one by one
    from paper_2605_12245_b200 import row_sharded as RS
    out2 = api.alloc_buffers(*w.shape, cfg)
    g2 = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(g2, stream=side):
        for stage in RS.stages(cfg.max_iters):
            api.soar_quantize_stage([W], cfg, [out2], out2.workspace, stage, side)
    g2.replay()
    torch.cuda.synchronize()
    gpu2 = P.GpuOut(out2.packed.cpu().numpy(), out2.scales.cpu().numpy(), float(out2.alpha.cpu()[0]),
                    out2.read_result(), out2)
    P.assert_parity(gpu2, R.quantize(w, ref_cfg))


def test_weighted_batch_gives_each_matrix_what_a_single_call_gives():
    """Nineteen matrices with their own weight vectors through soar_quantize_weighted_batch (two launch groups,
    one block to hundreds of tiles, a matrix with zero weights, one all zero, one with a bad weight): the same
    bytes as separate soar_quantize_weighted calls, and the oracle's."""
    shapes = [(1, 16), (3, 48), (37, 1040), (300, 4096), (64, 4096), (5, 16), (257, 512), (8, 8192), (600, 2064)] * 2 + \
             [(96, 1024)]
    ws = [WL.small_case(r, c, 500 + i, dist=("laplace" if i % 3 == 0 else "student_t4"),
                        outlier_entry_frac=0.004 * (i % 2), outlier_scale=40.0) for i, (r, c) in enumerate(shapes)]
    hs = [WL.column_weights(c, 600 + i, zero_frac=(0.1 if i == 4 else 0.0)) for i, (r, c) in enumerate(shapes)]
    ws[5][:] = 0
    hs[7] = hs[7].copy(); hs[7][3] = -1.0                     # a bad weight: that matrix alone is rejected
    cfg, ref_cfg = P.cfg_pair()
    dev = [P.to_device(w) for w in ws]
    dh = [torch.from_numpy(h).cuda() for h in hs]
    outs = [api.alloc_buffers(w.shape[0], w.shape[1], cfg) for w in ws]
    api.soar_quantize_weighted_batch(dev, dh, cfg, outs)
    torch.cuda.synchronize()
    for i, (w, h, W, H, o) in enumerate(zip(ws, hs, dev, dh, outs)):
        one = api.soar_quantize_weighted(W, H, cfg)
        torch.cuda.synchronize()
        r1, rb = one.read_result(), o.read_result()
        assert rb.status == r1.status and rb.iters_run == r1.iters_run, i
        if rb.status & api.STATUS_BAD_WEIGHT:
            assert i == 7
            continue
        assert torch.equal(o.packed, one.packed) and torch.equal(o.scales, one.scales) and torch.equal(o.alpha, one.alpha), i
        assert rb.sse == pytest.approx(r1.sse, rel=1e-12), i
        if rb.status == 0 and i % 3 == 0:
            g = P.GpuOut(o.packed.cpu().numpy(), o.scales.cpu().numpy(), float(o.alpha.cpu()[0]), rb, o)
            P.assert_parity(g, R.quantize(w, ref_cfg, h=h), mismatch_cap=(0 if w.size < 16 * 20000 else None))
