"""GPU parity of the MXFP4 entry point (Sec. 4.3, "DSS on MXFP4") against the oracle's MXFP4 mode on
the same seeded bytes: codes and E8M0 scale bytes bit-exact outside the blocks the oracle flags
as ties, the error within 1e-5."""
import numpy as np
import pytest
import torch

from oracle import soar_ref as R
from paper_2605_12245_b200 import api
from paper_2605_12245_b200 import workloads as WL
from tests import parity as P

pytestmark = pytest.mark.gpu


def run(w, ld=None, **kw):
    out = api.soar_mx_quantize(P.to_device(w, ld), **kw)
    torch.cuda.synchronize()
    return out.packed.cpu().numpy(), out.scales.cpu().numpy(), out.read_result()


def check(w, ld=None, **kw):
    packed, scales, res = run(w, ld, **kw)
    ref = R.mx_quantize(w, **kw)
    rows, nb = ref.scales.shape
    bad = (packed != ref.packed).reshape(rows, nb, 16).any(axis=2) | (scales != ref.scales)
    ties = ref.tie_flags.astype(bool)
    assert res.status == ref.status
    assert int((bad & ~ties).sum()) == 0, (int(bad.sum()), int(ties.sum()))
    assert int(bad.sum()) <= max(1e-4 * bad.size, 0), (int(bad.sum()), bad.size)
    assert res.sse == pytest.approx(ref.sse, rel=P.SSE_RTOL)
    assert res.sumsq == pytest.approx(ref.sumsq, rel=1e-12)
    return int(bad.sum()), int(ties.sum()), bad.size


@pytest.mark.parametrize("rows,cols,ld,seed,kw", [
    (1, 32, None, 0, {}),
    (3, 96, 128, 1, {}),
    (37, 1056, None, 2, dict(outlier_entry_frac=0.01, outlier_scale=50.0)),
    (130, 2080, 2088, 3, dict(dist="laplace", outlier_cols_frac=0.01, outlier_scale=20.0)),
    (257, 4096, None, 4, dict(dist="gauss_t2mix")),
])
@pytest.mark.parametrize("cfgkw", [
    dict(n_beta=0),                                   # the format's plain rule
    dict(),                                           # 2 x 101 pairs
    dict(n_dq=1, n_beta=11, beta_step_pct=3),
    dict(n_dq=4, n_beta=21, beta_step_pct=4),
])
def test_mxfp4_parity_small(rows, cols, ld, seed, kw, cfgkw):
    print(check(WL.small_case(rows, cols, seed, **kw), ld, **cfgkw))


def test_mxfp4_degenerate_inputs():
    w = WL.small_case(4, 128, 21)
    w[0, :32] = 0
    w[0, 7] = 0x8000
    w[1, 32:64] = WL.f32_to_bf16_bits(np.full(32, 1e-38, np.float32))
    w[2, 64:96] = WL.f32_to_bf16_bits(np.full(32, 3e30, np.float32))
    for nb in (0, 101):
        check(w, n_beta=nb)
    _, scales, res = run(w)
    assert res.zero_blocks == 2 and scales[0, 0] == 0 and scales[1, 1] == 0
    z = np.zeros((2, 64), np.uint16)
    packed, scales, res = run(z)
    assert res.status == api.STATUS_ZERO_TENSOR and not packed.any() and not scales.any()
    bad = w.copy()
    bad[3, 3] = 0x7F80
    assert run(bad)[2].status & api.STATUS_NONFINITE
    with pytest.raises(api.SoarError):
        api.soar_mx_quantize(P.to_device(WL.small_case(2, 48, 1)))        # cols % 32 != 0


def test_mxfp4_full_size_tensor_and_gain_over_the_plain_rule():
    """k of the Llama-3-70B-shaped layer (1024 x 8192) whole; the search ends below the plain rule's error."""
    w = WL.generate(WL.config4(), 1)
    print("mxfp4 dss, config 4 k:", check(w))
    print("mxfp4 plain, config 4 k:", check(w, n_beta=0))
    plain, dss = run(w, n_beta=0)[2], run(w)[2]
    assert dss.sse < 0.9 * plain.sse
