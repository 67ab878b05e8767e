"""soar_quantize_static: the entry point for callers that cannot allocate device memory (code
living inside another framework's memory pool, plugins that receive only their input and
output buffers).  It keeps its scratch in an array built into the library, so it must give
exactly what soar_quantize gives with a caller-provided workspace, also when the array
still holds a previous call's leftovers.  Collected last on purpose."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import soar_ref as R
from paper_2605_12245_b200 import api
from paper_2605_12245_b200 import workloads as WL
from tests import parity as P

pytestmark = pytest.mark.gpu


def _outputs(buf):
    torch.cuda.synchronize()
    res = buf.read_result()
    return (buf.packed.cpu().numpy(), buf.scales.cpu().numpy(), buf.alpha.cpu().numpy(),
            res.iters_run, res.sse, res.status)


def test_static_scratch_entry_point_matches_workspace_entry_point_twice_in_a_row():
    cfg = api.soar_default_cfg(api.PRESET_PAPER, max_iters=3)
    cases = [WL.small_case(96, 1024, 71, outlier_entry_frac=0.002, outlier_scale=50.0),
             WL.small_case(33, 2064, 72, dist="laplace")]
    for w in cases:                                  # two calls in a row share the built-in array
        W = P.to_device(w)
        rows, cols = w.shape
        want = _outputs(api.soar_quantize(W, cfg, api.alloc_buffers(rows, cols, cfg)))
        out = api.alloc_buffers(rows, cols, cfg)
        out.workspace = None                         # not used by this entry point
        got = _outputs(api.soar_quantize_static(W, cfg, out))
        assert np.array_equal(got[0], want[0])       # codes, bit-exact
        assert np.array_equal(got[1], want[1])       # scale bytes, bit-exact
        assert got[2][0] == want[2][0]               # alpha
        assert got[3] == want[3] and got[5] == want[5] == 0
        assert got[4] == pytest.approx(want[4], rel=P.SSE_RTOL)
        # and what the oracle gives for the same bytes
        P.assert_parity(P.GpuOut(got[0], got[1], float(got[2][0]), out.read_result(), out),
                        R.quantize(w, R.RefCfg(max_iters=3)), mismatch_cap=0)


def test_static_scratch_entry_point_takes_no_device_memory_and_fits_its_largest_matrix():
    """The largest accepted matrix with the settings that need the most scratch (iterations on, no
    row-major scale output, so the scale bytes live in the scratch too): the need then equals
    the built-in array exactly.  Device memory in use must be the same after the calls as before."""
    rows = cols = 4096
    assert rows * cols == api.STATIC_MAX_ELEMENTS
    cfg = api.soar_default_cfg(api.PRESET_PAPER, max_iters=3, scale_layout=api.SCALES_SWIZZLED)
    w = WL.small_case(rows, cols, 73, outlier_entry_frac=0.0005, outlier_scale=50.0)
    W = P.to_device(w)
    want = api.soar_quantize(W, cfg, api.alloc_buffers(rows, cols, cfg))
    out = api.alloc_buffers(rows, cols, cfg)
    out.workspace = None
    api.soar_quantize_static(W, cfg, out)                     # the first call on a device looks the array up
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    for _ in range(2):
        api.soar_quantize_static(W, cfg, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
    assert torch.equal(out.packed, want.packed) and torch.equal(out.scales_sw, want.scales_sw)
    assert torch.equal(out.alpha, want.alpha)
    assert out.read_result().iters_run == want.read_result().iters_run == 3


def test_static_scratch_entry_point_refuses_large_matrices():
    cfg = api.soar_default_cfg(api.PRESET_RTN)
    rows, cols = 4096 + 16, 4096                    # just above the stated maximum
    assert rows * cols > api.STATIC_MAX_ELEMENTS
    W = torch.zeros((rows, cols), dtype=torch.bfloat16, device="cuda")
    out = api.alloc_buffers(rows, cols, cfg)
    with pytest.raises(api.SoarError, match="built-in scratch"):
        api.soar_quantize_static(W, cfg, out)
    assert api.lib().soar_status_string(-5).decode().startswith("matrix exceeds")
