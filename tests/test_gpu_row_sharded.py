"""One tensor split by rows into parts that run stage by stage (soar_quantize_stage) with the
workspace-header fields combined between stages: what several GPUs would do with an all-reduce,
emulated here on one GPU by running the parts one after another and combining their headers
locally with the same schedule.  The concatenated outputs must be those of the unsplit tensor
and must pass the oracle's parity bar."""
import numpy as np
import pytest
import torch

from oracle import soar_ref as R
from paper_2605_12245_b200 import api
from paper_2605_12245_b200 import row_sharded as RS
from paper_2605_12245_b200 import workloads as WL
from tests import parity as P

pytestmark = pytest.mark.gpu


def combine_locally(headers, stage, max_iters):
    """What combine_header's all-reduce does over ranks, over a list of headers on one device."""
    for name, idx, how in RS.fields_written(stage, max_iters):
        views = [RS.header_view(h, name, idx) for h in headers]
        vals = torch.stack([v.to(torch.float64) for v in views])
        red = vals.max(0).values if how == RS.MAX else vals.sum(0)
        for v in views:
            v.copy_(red.to(v.dtype))


def run_parts(w_bits, cuts, cfg):
    """Quantize the row ranges [cuts[i], cuts[i+1]) as separate parts; returns per-part buffers."""
    Ws = [P.to_device(np.ascontiguousarray(w_bits[a:b])) for a, b in zip(cuts[:-1], cuts[1:])]
    outs = [api.alloc_buffers(W.shape[0], W.shape[1], cfg) for W in Ws]
    headers = [o.workspace[:api.WORKSPACE_HEADER_BYTES] for o in outs]
    for stage in RS.stages(cfg.max_iters):
        for W, o in zip(Ws, outs):
            api.soar_quantize_stage([W], cfg, [o], o.workspace, stage)
        combine_locally(headers, stage, cfg.max_iters)
    torch.cuda.synchronize()
    return outs


def joined(outs):
    packed = np.concatenate([o.packed.cpu().numpy() for o in outs])
    scales = np.concatenate([o.scales.cpu().numpy() for o in outs])
    return packed, scales


@pytest.mark.parametrize("cfgkw", [dict(), dict(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1), dict(max_iters=0)])
def test_stages_in_order_on_one_part_are_the_whole_call(cfgkw):
    w = WL.small_case(130, 1040, 4, outlier_entry_frac=0.002, outlier_scale=30.0)
    cfg, _ = P.cfg_pair(**cfgkw)
    whole = P.run_gpu(w, cfg)
    (part,) = run_parts(w, [0, 130], cfg)
    assert np.array_equal(part.packed.cpu().numpy(), whole.packed)
    assert np.array_equal(part.scales.cpu().numpy(), whole.scales)
    a, b = part.read_result(), whole.result
    # (tensor sums are atomic additions in arrival order: their last bits vary from run to run)
    assert (a.status, a.iters_run, a.alpha, a.amax, a.zero_blocks) == (b.status, b.iters_run, b.alpha, b.amax, b.zero_blocks)
    assert a.sse == pytest.approx(b.sse, rel=1e-12) and a.sumsq == pytest.approx(b.sumsq, rel=1e-13)


@pytest.mark.parametrize("cuts", [[0, 128, 384, 500], [0, 1, 500], [0, 250, 500]])
@pytest.mark.parametrize("cfgkw", [dict(), dict(max_iters=2, early_stop_rel=0.0, n_dq=2, n_beta=1)])
def test_row_parts_with_combined_headers_give_the_unsplit_tensor(cuts, cfgkw):
    w = WL.small_case(500, 2048, 9, outlier_cols_frac=0.01, outlier_scale=20.0)
    cfg, ref_cfg = P.cfg_pair(**cfgkw)
    whole = P.run_gpu(w, cfg)
    outs = run_parts(w, cuts, cfg)
    packed, scales = joined(outs)
    results = [o.read_result() for o in outs]
    alphas = [float(o.alpha.cpu()[0]) for o in outs]
    # every part ends with the whole tensor's alpha, iteration count and report
    assert len(set(alphas)) == 1 and alphas[0] == whole.alpha
    for r in results:
        assert r.iters_run == whole.result.iters_run and r.status == 0
        assert r.sse == pytest.approx(whole.result.sse, rel=1e-12)
        assert r.sumsq == pytest.approx(whole.result.sumsq, rel=1e-13)
        assert r.zero_blocks == whole.result.zero_blocks and r.wide_candidates == whole.result.wide_candidates
    assert np.array_equal(packed, whole.packed) and np.array_equal(scales, whole.scales)
    # and the oracle's bar on the joined outputs
    gpu = P.GpuOut(packed, scales, alphas[0], results[0], outs[0])
    P.assert_parity(gpu, R.quantize(w, ref_cfg))


def test_a_zero_part_and_a_part_with_a_nan():
    w = WL.small_case(256, 512, 12)
    w[:128] = 0                                           # the first part is all zero, the tensor is not
    cfg, ref_cfg = P.cfg_pair(max_iters=2, early_stop_rel=0.0, n_dq=2, n_beta=5)
    outs = run_parts(w, [0, 128, 256], cfg)
    packed, scales = joined(outs)
    res = [o.read_result() for o in outs]
    assert res[0].status == 0 and res[1].status == 0      # not a zero tensor: the other part has data
    assert not scales[:128].any() and res[0].zero_blocks == 128 * 32
    gpu = P.GpuOut(packed, scales, float(outs[0].alpha.cpu()[0]), res[0], outs[0])
    P.assert_parity(gpu, R.quantize(w, ref_cfg))
    w[200, 17] = 0x7FC0                                   # NaN in the second part: every part must report it
    outs = run_parts(w, [0, 128, 256], cfg)
    assert all(o.read_result().status & api.STATUS_NONFINITE for o in outs)
    assert all(o.read_result().iters_run == 0 for o in outs)


def test_swizzled_scales_of_128_row_parts_are_slices_of_the_whole():
    w = WL.small_case(384, 16 * 12, 3)
    cfg = api.soar_default_cfg(api.PRESET_PAPER, scale_layout=api.SCALES_LINEAR | api.SCALES_SWIZZLED)
    whole = P.run_gpu(w, cfg)
    outs = run_parts(w, [0, 128, 384], cfg)
    sw = np.concatenate([o.scales_sw.cpu().numpy() for o in outs])
    assert np.array_equal(sw, whole.buffers.scales_sw.cpu().numpy())


def test_stage_argument_errors():
    cfg = api.soar_default_cfg(api.PRESET_PAPER, max_iters=3)
    W = torch.zeros((16, 64), dtype=torch.bfloat16, device="cuda")
    out = api.alloc_buffers(16, 64, cfg)
    for bad in (3, 64, -4):
        with pytest.raises(api.SoarError):
            api.soar_quantize_stage([W], cfg, [out], out.workspace, bad)
    api.soar_quantize_stage([W], cfg, [out], out.workspace, api.STAGE_AMAX)
    torch.cuda.synchronize()
