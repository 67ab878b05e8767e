"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded bytes.  Shapes span several CTAs' worth of blocks, ragged tails and padded row
strides; settings cover the paper's preset and the smaller candidate grids."""
import ml_dtypes
import numpy as np
import pytest
import torch

from oracle import soar_ref as R
from paper_2605_12245_b200 import api
from paper_2605_12245_b200 import workloads as WL
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols,ld,seed,kw", [
    (1, 16, None, 0, {}),
    (3, 48, 64, 1, {}),
    (37, 1040, None, 2, dict(outlier_entry_frac=0.01, outlier_scale=50.0)),
    (130, 2064, 2072, 3, dict(dist="laplace", outlier_cols_frac=0.01, outlier_scale=20.0)),
    (257, 4096, None, 4, dict(dist="gauss_t2mix")),
])
@pytest.mark.parametrize("cfgkw", [
    dict(),                                                   # the paper's preset
    dict(max_iters=0),                                        # Eq. 1-3 only
    dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1),  # single pass
    dict(max_iters=3, early_stop_rel=0.0, n_dq=1, n_beta=1),  # CJSO with the nearest scale
    dict(max_iters=2, early_stop_rel=0.0, n_dq=4, n_beta=6, beta_step_pct=3),
    dict(flags=1, n_dq=1, n_beta=1),                                        # Sec. 3.2 alone (coupled scale)
    dict(flags=1, n_dq=2, n_beta=1),                                        # both bracketing codes, coupled
    dict(flags=1, max_iters=2, early_stop_rel=0.0, n_dq=2, n_beta=3, beta_step_pct=5),
    dict(flags=6, max_iters=1, early_stop_rel=0.0),                          # Sec. 3.3 alone (2 x 101 search)
    dict(flags=6, max_iters=2, early_stop_rel=0.0, n_dq=4, n_beta=7, beta_step_pct=4),
])
def test_parity_small(rows, cols, ld, seed, kw, cfgkw):
    w = WL.small_case(rows, cols, seed, **kw)
    cfg, ref_cfg = P.cfg_pair(**cfgkw)
    gpu = P.run_gpu(w, cfg, ld)
    ref = R.quantize(w, ref_cfg)
    P.assert_parity(gpu, ref)
    assert gpu.result.sumsq == pytest.approx(ref.sumsq, rel=1e-12)


def test_parity_medium_paper_preset():
    """512 x 2048 with outlier columns: 65 536 blocks, full 15 x 202 search."""
    w = WL.small_case(512, 2048, 11, outlier_cols_frac=0.001, outlier_scale=20.0)
    cfg, ref_cfg = P.cfg_pair()
    rep = P.assert_parity(P.run_gpu(w, cfg), R.quantize(w, ref_cfg))
    print("medium:", rep)


def test_rounding_ties_e2m1_and_e4m3():
    """Inputs built so that |W|/(alpha*scale) lands exactly on E2M1 midpoints and
    bmax/(6 alpha) exactly on E4M3 midpoints: both sides must break the ties alike."""
    e4 = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    unit = 2.0 ** -10                       # alpha0 = amax/2688 = 2^-10 exactly
    rows = []
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 0.0, 5.5])
    for c in range(0x28, 0x7E, 3):          # block scales with exact products in bf16
        s = e4[c]
        blk = mids * s * unit
        blk[7] = 6.0 * s * unit             # block max pins the scale to code c
        rows.append(blk)
    for c in range(0x30, 0x7D):             # block max on the midpoint between codes c and c+1
        mid = 0.5 * (e4[c] + e4[c + 1])
        blk = np.zeros(16)
        blk[0] = 6.0 * mid * unit
        blk[1:8] = mids[:7] * e4[c] * unit
        rows.append(blk)
    top = np.zeros(16); top[0] = 2688.0 * unit
    rows.append(top)
    w = np.array(rows, np.float32)
    w = np.concatenate([w, -w], axis=0)
    bits = WL.f32_to_bf16_bits(w)
    assert np.array_equal(WL.bf16_bits_to_f32(bits), w), "test values must be exact in bf16"
    for cfgkw in (dict(max_iters=0), dict(max_iters=2, early_stop_rel=0.0)):
        cfg, ref_cfg = P.cfg_pair(**cfgkw)
        P.assert_parity(P.run_gpu(bits, cfg), R.quantize(bits, ref_cfg))


def test_degenerate_blocks_and_tensors():
    w = WL.small_case(8, 256, 20)
    w[1, 16:32] = 0
    w[1, 20] = 0x8000                                        # negative zero inside a zero block
    w[2, 32:48] = WL.f32_to_bf16_bits(np.full(16, 1e-12, np.float32))
    cfg, ref_cfg = P.cfg_pair(max_iters=3)
    gpu = P.run_gpu(w, cfg)
    P.assert_parity(gpu, R.quantize(w, ref_cfg))
    assert gpu.result.zero_blocks == 1
    z = np.zeros((4, 64), np.uint16); z[0, 5] = 0x8000
    gz, rz = P.run_gpu(z, cfg), R.quantize(z, ref_cfg)
    assert gz.result.status == api.STATUS_ZERO_TENSOR == rz.status
    assert gz.alpha == 1.0 and np.array_equal(gz.packed, rz.packed) and not gz.scales.any()
    bad = w.copy(); bad[3, 7] = 0x7FC0
    assert P.run_gpu(bad, cfg).result.status & api.STATUS_NONFINITE
    bad[3, 7] = 0xFF80
    assert P.run_gpu(bad, cfg).result.status & api.STATUS_NONFINITE
    tiny = WL.f32_to_bf16_bits(np.full((2, 32), 1e-35, np.float32))
    assert P.run_gpu(tiny, cfg).result.status & api.STATUS_RANGE


def test_wide_candidates_take_the_exact_path():
    """One element 200x above the rest of its block: candidates with a scale fit to the
    small elements saturate the large one far beyond 32 and must still be scored exactly."""
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((16, 256)) * 0.01).astype(np.float32)
    w[:, ::16] *= 300.0
    bits = WL.f32_to_bf16_bits(w)
    cfg, ref_cfg = P.cfg_pair(max_iters=2, early_stop_rel=0.0, n_dq=2, n_beta=101, beta_step_pct=1)
    gpu = P.run_gpu(bits, cfg)
    P.assert_parity(gpu, R.quantize(bits, ref_cfg))


def test_presets_of_the_stand_alone_arms_match_the_oracle():
    w = WL.small_case(96, 1024, 61, outlier_cols_frac=0.004, outlier_scale=20.0)
    for preset, ref_cfg in (
            (api.PRESET_CJSO_ONLY, R.RefCfg(n_dq=1, n_beta=1, flags=R.FLAG_COUPLED_SCALE)),
            (api.PRESET_COUPLED_PAIR, R.RefCfg(n_dq=2, n_beta=1, flags=R.FLAG_COUPLED_SCALE)),
            (api.PRESET_DSS_ONLY, R.RefCfg(max_iters=1, early_stop_rel=0.0,
                                           flags=R.FLAG_KEEP_ALPHA | R.FLAG_KEEP_BLOCK_SCALE))):
        P.assert_parity(P.run_gpu(w, api.soar_default_cfg(preset)), R.quantize(w, ref_cfg))


def test_fast_reciprocal_equals_the_correctly_rounded_one_everywhere_it_is_used():
    """All 2^23 significands of every exponent the shortcut is allowed on: 2.1e9 inputs."""
    assert api.soar_selftest_reciprocal(2, 252) == 0
    with pytest.raises(api.SoarError):
        api.soar_selftest_reciprocal(1, 252)


@pytest.mark.parametrize("cfgkw", [
    dict(),                                                   # the paper's preset: tensors stop after different iterations
    dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1),  # single pass
    dict(max_iters=0),
])
def test_batch_gives_each_matrix_what_a_single_call_gives(cfgkw):
    """20 matrices (more than one launch group), from one block to several tiles, one all zero,
    one with a NaN, one with a padded row stride: same bytes as 20 separate calls, and the oracle's."""
    shapes = [(1, 16), (3, 48), (37, 1040), (130, 2064), (64, 4096), (5, 16), (257, 512), (8, 8192)] * 2 + \
             [(16, 64), (96, 1024), (33, 272), (512, 256)]
    ws = [WL.small_case(r, c, 100 + i, dist=("laplace" if i % 3 == 0 else "student_t4"),
                        outlier_entry_frac=0.005 * (i % 2), outlier_scale=40.0)
          for i, (r, c) in enumerate(shapes)]
    ws[5][:] = 0
    ws[9] = ws[9].copy(); ws[9][1, 3] = 0x7FC0
    cfg, ref_cfg = P.cfg_pair(**cfgkw)
    dev = [P.to_device(w, ld=(w.shape[1] + 24 if i == 3 else None)) for i, w in enumerate(ws)]
    outs = [api.alloc_buffers(w.shape[0], w.shape[1], cfg) for w in ws]
    api.soar_quantize_batch(dev, cfg, outs)
    torch.cuda.synchronize()
    for i, (w, W, o) in enumerate(zip(ws, dev, outs)):
        one = api.soar_quantize(W, cfg)
        torch.cuda.synchronize()
        r1, rb = one.read_result(), o.read_result()
        assert rb.status == r1.status and rb.iters_run == r1.iters_run, i
        if rb.status & api.STATUS_NONFINITE:
            continue
        assert np.array_equal(o.packed.cpu().numpy(), one.packed.cpu().numpy()), i
        assert np.array_equal(o.scales.cpu().numpy(), one.scales.cpu().numpy()), i
        assert float(o.alpha.cpu()[0]) == float(one.alpha.cpu()[0]), i
        assert rb.sse == pytest.approx(r1.sse, rel=1e-12), i
        if rb.status == 0 and i % 4 == 0:
            g = P.GpuOut(o.packed.cpu().numpy(), o.scales.cpu().numpy(), float(o.alpha.cpu()[0]), rb, o)
            P.assert_parity(g, R.quantize(w, ref_cfg))


def test_a_wait_that_runs_out_is_reported_and_leaves_the_library_usable():
    """The kernels' waits are bounded.  With the test hook on, no tile is ever fetched, every consumer
    wait runs to its poll limit, the kernels return, and the report says so; a normal call on the
    same buffers right afterwards gives the right bytes."""
    w = WL.small_case(300, 2048, 95, outlier_entry_frac=0.002, outlier_scale=30.0)
    cfg, ref_cfg = P.cfg_pair(max_iters=3)
    W = P.to_device(w)
    out = api.alloc_buffers(300, 2048, cfg)
    api.soar_debug_fail_waits(True)
    try:
        api.soar_quantize(W, cfg, out)
        e = api.soar_dequant_error(W, out.packed, out.scales, out.alpha)
        torch.cuda.synchronize()
    finally:
        api.soar_debug_fail_waits(False)
    res = out.read_result()
    assert res.status & api.STATUS_INTERNAL and res.iters_run == 0
    assert bool(torch.isnan(e).all())
    api.soar_quantize(W, cfg, out)                                  # same workspace, right after
    torch.cuda.synchronize()
    g = P.GpuOut(out.packed.cpu().numpy(), out.scales.cpu().numpy(), float(out.alpha.cpu()[0]), out.read_result(), out)
    P.assert_parity(g, R.quantize(w, ref_cfg))


def test_deterministic_mode_repeats_bit_for_bit():
    """With SOAR_FLAG_DETERMINISTIC the tensor-wide sums are added in a fixed order: twenty runs of a
    tensor of a thousand tiles (every CTA of every pass contributes) and of a batch give the same
    bits in every output and every reported number; and they are the oracle's results."""
    w = WL.small_case(2048, 2048, 301, outlier_entry_frac=0.0005, outlier_scale=50.0)
    small = [WL.small_case(r, c, 310 + i) for i, (r, c) in enumerate([(300, 1024), (1, 16), (77, 4096)])]
    cfg, ref_cfg = P.cfg_pair()
    cfg.flags |= api.FLAG_DETERMINISTIC
    assert api.soar_workspace_bytes(2048, 2048, cfg) >= api.soar_workspace_bytes(2048, 2048, P.cfg_pair()[0]) + 56 * 1024
    W = P.to_device(w)
    dev = [P.to_device(x) for x in small]
    first = None
    for rep in range(20):
        out = api.soar_quantize(W, cfg)
        outs = [api.alloc_buffers(x.shape[0], x.shape[1], cfg) for x in small]
        api.soar_quantize_batch(dev, cfg, outs)
        torch.cuda.synchronize()
        got = []
        for o in [out] + outs:
            r = o.read_result()
            got.append((o.packed.cpu().numpy().tobytes(), o.scales.cpu().numpy().tobytes(), o.alpha.cpu().numpy().tobytes(),
                        r.iters_run, r.sse, r.sse_init, r.sumsq, tuple(r.trace_sse), tuple(r.trace_alpha)))
        if first is None:
            first = got
            g = P.GpuOut(out.packed.cpu().numpy(), out.scales.cpu().numpy(), float(out.alpha.cpu()[0]),
                         out.read_result(), out)
            P.assert_parity(g, R.quantize(w, ref_cfg))
            for x, o in zip(small, outs):
                g = P.GpuOut(o.packed.cpu().numpy(), o.scales.cpu().numpy(), float(o.alpha.cpu()[0]), o.read_result(), o)
                P.assert_parity(g, R.quantize(x, ref_cfg), mismatch_cap=0)
        else:
            assert got == first, rep
    # settings without iterations, and the one-candidate shape
    for kw in (dict(max_iters=0), dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1)):
        c, rc = P.cfg_pair(**kw)
        c.flags |= api.FLAG_DETERMINISTIC
        a, b = P.run_gpu(w, c), P.run_gpu(w, c)
        assert (a.result.sse, a.result.sumsq, a.alpha) == (b.result.sse, b.result.sumsq, b.alpha)
        assert np.array_equal(a.packed, b.packed)
        P.assert_parity(a, R.quantize(w, rc))
    # the staged and the weighted entry points do not take the flag
    with pytest.raises(api.SoarError):
        o = api.alloc_buffers(2048, 2048, cfg)
        api.soar_quantize_stage([W], cfg, [o], o.workspace, api.STAGE_AMAX)
    with pytest.raises(api.SoarError):
        api.soar_quantize_weighted(W, torch.ones(2048, device="cuda"), cfg)


def test_calls_on_two_streams_with_their_own_workspaces_do_not_disturb_each_other():
    w1 = WL.small_case(300, 2048, 81, outlier_entry_frac=0.003, outlier_scale=30.0)
    w2 = WL.small_case(200, 4096, 82, dist="laplace")
    cfg, _ = P.cfg_pair(max_iters=3)
    W1, W2 = P.to_device(w1), P.to_device(w2)
    want1, want2 = api.soar_quantize(W1, cfg), api.soar_quantize(W2, cfg)
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    o1, o2 = api.alloc_buffers(*w1.shape, cfg), api.alloc_buffers(*w2.shape, cfg)
    for _ in range(3):
        api.soar_quantize(W1, cfg, o1, s1)
        api.soar_quantize(W2, cfg, o2, s2)
    torch.cuda.synchronize()
    for got, want in ((o1, want1), (o2, want2)):
        assert torch.equal(got.packed, want.packed) and torch.equal(got.scales, want.scales)
        assert torch.equal(got.alpha, want.alpha)


def test_a_call_replays_from_a_cuda_graph():
    """Nothing in a call synchronizes or allocates, so it can be captured once and replayed."""
    w = WL.small_case(128, 2048, 83, outlier_cols_frac=0.002, outlier_scale=20.0)
    cfg, ref_cfg = P.cfg_pair()
    W = P.to_device(w)
    out = api.alloc_buffers(*w.shape, cfg)
    side = torch.cuda.Stream()
    api.soar_quantize(W, cfg, out, side)                  # first call outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        api.soar_quantize(W, cfg, out, side)
    out.packed.zero_(); out.scales.zero_(); out.alpha.zero_()
    g.replay()
    torch.cuda.synchronize()
    gpu = P.GpuOut(out.packed.cpu().numpy(), out.scales.cpu().numpy(), float(out.alpha.cpu()[0]),
                   out.read_result(), out)
    P.assert_parity(gpu, R.quantize(w, ref_cfg))


def test_host_entry_point_and_launch_trace():
    """soar_quantize_host (copies in, quantizes, copies out on one stream) against a direct call;
    the launch trace names every kernel of the call."""
    w = WL.small_case(130, 2064, 91, outlier_entry_frac=0.003, outlier_scale=30.0)
    cfg, _ = P.cfg_pair(max_iters=2, early_stop_rel=0.0)
    want = P.run_gpu(w, cfg)
    hb = api.alloc_host_buffers(w.shape[0], w.shape[1], cfg)
    hb.W.copy_(torch.from_numpy(w.view(np.int16)).view(torch.bfloat16))
    dev_W = torch.empty(w.shape, dtype=torch.bfloat16, device="cuda")
    dev = api.alloc_buffers(w.shape[0], w.shape[1], cfg)
    api.soar_trace_begin()
    api.soar_quantize_host(hb, cfg, dev_W, dev)
    torch.cuda.synchronize()
    trace = api.soar_trace_end()
    assert np.array_equal(hb.packed.numpy(), want.packed) and np.array_equal(hb.scales.numpy(), want.scales)
    assert float(hb.alpha[0]) == want.alpha and hb.read_result().iters_run == 2
    assert {k: v[0] for k, v in trace.items()} == {"amax_kernel": 1, "init_kernel": 1, "iterate_kernel": 2,
                                                   "finalize_kernel": 1}
    assert sum(v[0] for v in trace.values()) == api.soar_quantize_launches(cfg)
    assert all(v[1] > 0 for v in trace.values())


def test_host_entry_point_enqueues_nothing_on_an_argument_error():
    """A workspace that is too small is refused before the copy of W into the staging buffer starts."""
    w = WL.small_case(64, 512, 92)
    cfg, _ = P.cfg_pair(max_iters=2)
    hb = api.alloc_host_buffers(64, 512, cfg)
    hb.W.copy_(torch.from_numpy(w.view(np.int16)).view(torch.bfloat16))
    dev_W = torch.full((64, 512), 7.0, dtype=torch.bfloat16, device="cuda")
    dev = api.alloc_buffers(64, 512, cfg)
    dev.workspace = dev.workspace[:1024]
    with pytest.raises(api.SoarError, match="workspace"):
        api.soar_quantize_host(hb, cfg, dev_W, dev)
    torch.cuda.synchronize()
    assert bool((dev_W == 7.0).all())


def test_host_pipeline_returns_what_direct_calls_return():
    """Seven matrices through three staging slots: every slot is reused, sizes differ."""
    shapes = [(64, 1024), (16, 256), (300, 512), (8, 4096), (130, 2064), (1, 16), (257, 1024)]
    ws = [WL.small_case(r, c, 200 + i, outlier_entry_frac=0.004, outlier_scale=30.0) for i, (r, c) in enumerate(shapes)]
    cfg, _ = P.cfg_pair(max_iters=3)
    hosts = []
    for w in ws:
        hb = api.alloc_host_buffers(w.shape[0], w.shape[1], cfg)
        hb.W.copy_(torch.from_numpy(w.view(np.int16)).view(torch.bfloat16))
        hosts.append(hb)
    pipe = api.HostPipeline(shapes, cfg, depth=3)
    for _ in range(2):                                   # the second round reuses everything once more
        pipe.run(hosts)
    pipe.synchronize()
    for w, hb in zip(ws, hosts):
        want = P.run_gpu(w, cfg)
        assert np.array_equal(hb.packed.numpy(), want.packed)
        assert np.array_equal(hb.scales.numpy(), want.scales)
        assert float(hb.alpha[0]) == want.alpha
        assert hb.read_result().iters_run == want.result.iters_run


def test_host_pipeline_weighted_objective_and_slot_capacity():
    """The pipeline with column weights equals direct soar_quantize_weighted calls; a matrix that does not fit
    the slots is refused before anything is enqueued."""
    shapes = [(64, 1024), (130, 2064), (16, 256)]
    ws = [WL.small_case(r, c, 230 + i, outlier_entry_frac=0.004, outlier_scale=30.0) for i, (r, c) in enumerate(shapes)]
    hs = [torch.from_numpy(WL.column_weights(c, 240 + i)).cuda() for i, (r, c) in enumerate(shapes)]
    cfg, _ = P.cfg_pair(max_iters=3)
    hosts = []
    for w in ws:
        hb = api.alloc_host_buffers(w.shape[0], w.shape[1], cfg)
        hb.W.copy_(torch.from_numpy(w.view(np.int16)).view(torch.bfloat16))
        hosts.append(hb)
    pipe = api.HostPipeline(shapes, cfg, depth=2, weighted=True)
    pipe.run(hosts, hs)
    pipe.synchronize()
    for w, h, hb in zip(ws, hs, hosts):
        want = api.soar_quantize_weighted(P.to_device(w), h, cfg)
        torch.cuda.synchronize()
        assert np.array_equal(hb.packed.numpy(), want.packed.cpu().numpy())
        assert np.array_equal(hb.scales.numpy(), want.scales.cpu().numpy())
        assert float(hb.alpha[0]) == float(want.alpha.cpu()[0])
    big = api.alloc_host_buffers(512, 4096, cfg)             # larger than the slots
    big.W.zero_()
    marker = hosts[0].packed.clone()
    with pytest.raises(api.SoarError, match="pipeline slot"):
        pipe.run([hosts[0], big])
    pipe.synchronize()
    assert torch.equal(hosts[0].packed, marker)
    pipe.close()


def test_argument_errors_are_reported_on_the_host():
    w = P.to_device(WL.small_case(4, 64, 0))
    cfg = api.soar_default_cfg()
    with pytest.raises(api.SoarError):
        api.soar_quantize(w[:, :40], cfg)                      # cols % 16 != 0
    bad = api.soar_default_cfg(block=32)
    with pytest.raises(api.SoarError):
        api.soar_quantize(w, bad)
    with pytest.raises(api.SoarError):
        api.soar_quantize(w, api.soar_default_cfg(flags=16))   # unknown flag bit
    out = api.alloc_buffers(4, 64, cfg)
    out.workspace = out.workspace[:16]
    with pytest.raises(api.SoarError):
        api.soar_quantize(w, cfg, out)
    with pytest.raises(api.SoarError):
        api.soar_quantize(w.cpu(), cfg)


def swizzle_reference(lin: np.ndarray) -> np.ndarray:
    """128x4-tiled scale layout written with array reshapes (independent of the kernel's
    index formula): pad to (128k, 4m); a tile is stored as [32 rows][4 row-groups][4 cols]."""
    rows, nbc = lin.shape
    rt, ct = -(-rows // 128), -(-nbc // 4)
    pad = np.zeros((rt * 128, ct * 4), np.uint8)
    pad[:rows, :nbc] = lin
    t = pad.reshape(rt, 4, 32, ct, 4)          # [row tile][row group][row in group][col tile][col]
    return t.transpose(0, 3, 2, 1, 4).reshape(-1)


@pytest.mark.parametrize("rows,cols", [(128, 64), (130, 16 * 5), (300, 16 * 33)])
def test_swizzled_scale_layout(rows, cols):
    w = WL.small_case(rows, cols, 31)
    both = api.soar_default_cfg(api.PRESET_SINGLE_PASS, scale_layout=api.SCALES_LINEAR | api.SCALES_SWIZZLED)
    g = P.run_gpu(w, both)
    sw = g.buffers.scales_sw.cpu().numpy()
    assert sw.size == api.soar_swizzled_scale_bytes(rows, cols)
    assert np.array_equal(sw, swizzle_reference(g.scales))
    only = api.soar_default_cfg(api.PRESET_SINGLE_PASS, scale_layout=api.SCALES_SWIZZLED)
    W = P.to_device(w)
    o = api.soar_quantize(W, only)
    torch.cuda.synchronize()
    assert o.scales is None
    assert np.array_equal(o.scales_sw.cpu().numpy(), sw)
    assert np.array_equal(o.packed.cpu().numpy(), g.packed)
    # the error kernel reads either layout
    e_lin = api.soar_dequant_error(W, g.buffers.packed, g.buffers.scales, g.buffers.alpha).cpu().numpy()
    e_sw = api.soar_dequant_error(W, o.packed, o.scales_sw, o.alpha, api.SCALES_SWIZZLED).cpu().numpy()
    assert e_lin[0] == pytest.approx(e_sw[0], rel=1e-12)
    assert e_lin[0] == pytest.approx(g.result.sse, rel=1e-9)


@pytest.mark.parametrize("M,K,N", [(256, 512, 128), (128, 2048, 256)])
def test_outputs_feed_the_hardware_block_scaled_gemm(M, K, N):
    """The packed codes and the 128x4-tiled scales go, as they are, into the library's block-scaled FP4
    matrix product (Blackwell's block-scaled MMA underneath); the result must equal the product with
    the matrix dequantized by Eq. 3 on the host.  This pins the nibble order and the tiled scale
    layout against the consumer they are meant for.  The other operand is made of exact E2M1 values
    with unit scales, so the only rounding is the product's binary32 accumulation."""
    if not hasattr(torch, "float4_e2m1fn_x2"):
        pytest.skip("this torch has no packed FP4 dtype")
    w = WL.small_case(M, K, 7, outlier_entry_frac=0.002, outlier_scale=20.0)
    cfg = api.soar_default_cfg(api.PRESET_PAPER, scale_layout=api.SCALES_LINEAR | api.SCALES_SWIZZLED)
    g = P.run_gpu(w, cfg)
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
    codes = np.stack([g.packed & 0xF, g.packed >> 4], axis=-1).reshape(M, K)
    e4 = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    Wd = grid[codes & 7] * np.where(codes & 8, -1.0, 1.0) * np.repeat(e4[g.scales], 16, axis=1)   # Eq. 3 without alpha
    rng = np.random.default_rng(0)
    xc = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    X = grid[xc & 7] * np.where(xc & 8, -1.0, 1.0)
    xp = (xc[:, 0::2] | (xc[:, 1::2] << 4)).astype(np.uint8)
    ones = swizzle_reference(np.full((N, K // 16), 0x38, np.uint8))                               # E4M3 1.0
    a = torch.from_numpy(xp).cuda().view(torch.float4_e2m1fn_x2)
    b = g.buffers.packed.view(torch.float4_e2m1fn_x2)
    sa = torch.from_numpy(ones).cuda().view(torch.float8_e4m3fn)
    sb = g.buffers.scales_sw.view(torch.float8_e4m3fn)
    try:
        out = torch._scaled_mm(a, b.t(), sa, sb, out_dtype=torch.float32)
    except (RuntimeError, NotImplementedError) as e:      # no block-scaled FP4 product on this device / build
        pytest.skip(f"block-scaled FP4 product unavailable: {str(e)[:80]}")
    ref = X @ Wd.T
    assert np.abs(out.double().cpu().numpy() - ref).max() <= 1e-6 * np.abs(ref).max()


def test_dequant_error_matches_oracle():
    w = WL.small_case(96, 1024, 41, outlier_entry_frac=0.002, outlier_scale=50.0)
    cfg, ref_cfg = P.cfg_pair(max_iters=2)
    g = P.run_gpu(w, cfg, ld=1040)
    W = P.to_device(w, 1040)
    e = api.soar_dequant_error(W, g.buffers.packed, g.buffers.scales, g.buffers.alpha).cpu().numpy()
    sse, ss = R.dequant_error(w, g.packed, g.scales, g.alpha)
    assert e[0] == pytest.approx(sse, rel=1e-12)
    assert e[1] == pytest.approx(ss, rel=1e-12)
    assert g.result.sse == pytest.approx(sse, rel=1e-9)


def test_two_calls_share_a_workspace_and_repeat_exactly():
    w1, w2 = WL.small_case(64, 512, 50), WL.small_case(64, 512, 51)
    cfg, _ = P.cfg_pair(max_iters=2)
    out = api.alloc_buffers(64, 512, cfg)
    a = api.soar_quantize(P.to_device(w1), cfg, out); torch.cuda.synchronize()
    p1, s1, al1 = a.packed.cpu().numpy().copy(), a.scales.cpu().numpy().copy(), float(a.alpha.cpu()[0])
    api.soar_quantize(P.to_device(w2), cfg, out)
    api.soar_quantize(P.to_device(w1), cfg, out); torch.cuda.synchronize()
    assert np.array_equal(out.packed.cpu().numpy(), p1)
    assert np.array_equal(out.scales.cpu().numpy(), s1)
    assert float(out.alpha.cpu()[0]) == al1
