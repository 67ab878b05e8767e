"""NumPy restatement of SOAR for tiny inputs.  TEST INFRASTRUCTURE ONLY.

A second, independently written CPU implementation of Algorithm 1 of the SOAR paper
(Sec. 3.1-3.4, App. B.3).  It exists to pin ``soar_ref.c``: the two are written
separately, use different rounding routes (this file rounds with the ``ml_dtypes`` casts
to ``float4_e2m1fn`` and ``float8_e4m3fn``; the C file evaluates Eq. 2 literally) and must
agree bit for bit on small tensors.  The search is a flat enumeration of every
(beta, E4M3 neighbour) pair of every block, held in arrays, so it only suits a few
thousand blocks.

Same arithmetic convention as the C file: binary32 round-to-nearest steps for whatever
feeds a rounding decision, binary64 for sums and errors.
"""
from __future__ import annotations

import math

import ml_dtypes
import numpy as np

F32 = np.float32
E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])  # Sec. 3.1 / Eq. 2 grid
M_FP4 = 6.0
M_FP8 = 448.0


def e4m3_values() -> np.ndarray:
    """Values of the 127 non-negative finite E4M3 codes 0x00..0x7E (ascending)."""
    return np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)


def e4m3_encode(v: np.ndarray) -> np.ndarray:
    """Eq. 16: nearest E4M3 code (ties to even), clipped to 448."""
    v = np.minimum(np.asarray(v, dtype=F32), F32(M_FP8))
    return v.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)


def e2m1_round(x: np.ndarray) -> np.ndarray:
    """Eq. 2 via the library cast; magnitudes above 6 saturate."""
    x = np.minimum(np.asarray(x, dtype=F32), F32(M_FP4))
    return x.astype(ml_dtypes.float4_e2m1fn).astype(np.float64)


def reround(mag: np.ndarray, alpha: F32, dq: np.ndarray) -> np.ndarray:
    """Eq. 2 under scales (alpha, dq): magnitudes of the codes, shape of ``mag``.

    mag: float32 [..., 16]; dq: float32 [...]."""
    s = (F32(alpha) * dq.astype(F32)).astype(F32)
    with np.errstate(divide="ignore", invalid="ignore"):
        r = (F32(1.0) / s).astype(F32)
        x = (mag * r[..., None]).astype(F32)
    return e2m1_round(x)


def seq_sum(a: np.ndarray) -> np.ndarray:
    """Left-to-right binary64 sum over the last axis (the order the C file uses)."""
    acc = np.zeros(a.shape[:-1], np.float64)
    for j in range(a.shape[-1]):
        acc = acc + a[..., j]
    return acc


def betas(n_beta: int, step_pct: int) -> np.ndarray:
    k = np.arange(n_beta)
    return ((100.0 + (k - n_beta // 2) * step_pct) / 100.0).astype(F32)


def dq_candidates(center: np.ndarray, n: int, vals: np.ndarray) -> np.ndarray:
    """E4M3 codes around ``center`` (App. B.3), int array [nblk, n], clipped to [1, 0x7E].

    Duplicates created by the clipping stay in the array: the later copy can never win
    under a strict comparison, so they do not change the argmin."""
    if n <= 1:
        c = e4m3_encode(center).astype(np.int64)[:, None]
    else:
        cf = np.searchsorted(vals, center.astype(np.float64), side="right") - 1
        offs = np.arange(-(n // 2 - 1), n // 2 + 1)
        c = cf[:, None] + offs[None, :]
    return np.clip(c, 1, 0x7E)


def quantize(w_bits: np.ndarray, max_iters=15, early_stop_rel=1e-3, n_dq=2, n_beta=101,
             beta_step_pct=1, coupled_scale=False, keep_alpha=False, keep_block_scale=False, h=None):
    """Algorithm 1 on uint16 bf16 bit patterns [rows, cols]; returns a dict.

    The three switches give the paper's stand-alone arms: ``coupled_scale`` is Sec. 3.2's
    scheme (one block scale quantizes and dequantizes: a candidate's quantization scale is its
    own E4M3 value times beta); ``keep_alpha`` and ``keep_block_scale`` together are Sec. 3.3
    alone (no Eq. 5, no Eq. 6: the search runs around the max-based start).

    ``h`` (float32, one per column, optional) weights every element's term of the objective:
    the diagonal form of the output-distortion objective of Sec. 5."""
    rows, cols = w_bits.shape
    hb = (np.ones(cols) if h is None else np.asarray(h, np.float32).astype(np.float64))
    hb = np.tile(hb.reshape(-1, 16), (rows, 1))           # [nblk, 16] weights of each block's columns
    wf = (w_bits.astype(np.uint32) << np.uint32(16)).view(F32)
    sign = (w_bits >> 15).astype(np.uint8).reshape(-1, 16)
    mag = np.abs(wf).reshape(-1, 16).astype(F32)
    mag64 = mag.astype(np.float64)
    nblk = mag.shape[0]
    vals = e4m3_values()

    amax = F32(mag.max())
    assert amax > 0
    alpha = F32(amax / F32(2688.0))                       # Eq. 1
    bmax = mag.max(axis=1)
    live = bmax > 0
    t = (bmax / F32(alpha * F32(6.0))).astype(F32)
    dd = e4m3_encode(t).astype(np.int64)
    dd[live & (dd == 0)] = 1
    dd[~live] = 0
    dq = vals[dd].astype(F32)                             # dq0 = dd0 (Sec. 3.3 (i))

    def err(m, a, d):
        s = np.float64(a) * vals[d]
        e = mag64 - m * s[:, None]
        return seq_sum(hb * (e * e))

    m = reround(mag, alpha, dq)
    m[~live] = 0
    trace_alpha = [float(alpha)]
    trace_sse = [math.fsum(err(m, alpha, dd)[live])]
    bet = betas(n_beta, beta_step_pct)
    iters = 0
    for t_it in range(max_iters):
        m = reround(mag, alpha, dq)
        m[~live] = 0
        A = seq_sum((hb * mag64) * m)
        B = seq_sum(hb * (m * m))
        num = math.fsum((A * vals[dd])[live])
        den = math.fsum((B * vals[dd] ** 2)[live])
        alpha_new = F32(num / den) if den > 0 else alpha  # Eq. 5
        if keep_alpha:
            alpha_new = alpha
        # Eq. 6
        with np.errstate(divide="ignore", invalid="ignore"):
            center = (A.astype(F32) / (alpha_new * B.astype(F32)).astype(F32)).astype(F32)
        center = np.where(B > 0, center, vals[dd].astype(F32)).astype(F32)
        if keep_block_scale:
            center = vals[dd].astype(F32)
        cand_d = dq_candidates(center, n_dq, vals)         # [nblk, nd]
        nd = cand_d.shape[1]
        if coupled_scale:                                  # quantization scale = the candidate's own E4M3 value
            base = vals[cand_d].astype(F32)                # [nblk, nd]
        else:                                              # quantization scale around the unrounded solution
            base = np.repeat(center[:, None], nd, axis=1)
        cand_q = (base[:, None, :] * bet[None, :, None]).astype(F32)   # [nblk, nb, nd]
        mk = reround(mag[:, None, None, :], alpha_new, cand_q)         # [nblk, nb, nd, 16]
        best = np.full(nblk, np.inf)
        bk = np.zeros(nblk, np.int64)
        bd = np.zeros(nblk, np.int64)
        for k in range(n_beta):                            # beta ascending, then d ascending
            for j in range(nd):
                L = err(mk[:, k, j, :], alpha_new, cand_d[:, j])
                better = L < best                          # strict: first minimum wins
                best = np.where(better, L, best)
                bk = np.where(better, k, bk)
                bd = np.where(better, j, bd)
        ar = np.arange(nblk)
        dq = np.where(live, cand_q[ar, bk, bd], dq).astype(F32)
        dd = np.where(live, cand_d[ar, bd], dd)
        alpha = alpha_new
        sse_new = math.fsum(best[live])
        trace_alpha.append(float(alpha))
        prev = trace_sse[-1]
        trace_sse.append(sse_new)
        iters = t_it + 1
        if early_stop_rel > 0 and (prev == 0 or (prev - sse_new) / prev < early_stop_rel):
            break

    m = reround(mag, alpha, dq)
    m[~live] = 0
    code = np.searchsorted(E2M1_VALUES, m).astype(np.uint8) | (sign << 3)
    packed = (code[:, 0::2] | (code[:, 1::2] << 4)).astype(np.uint8).reshape(rows, cols // 2)
    return dict(packed=packed, scales=dd.astype(np.uint8).reshape(rows, cols // 16),
                alpha=float(alpha), iters_run=iters, trace_alpha=np.array(trace_alpha),
                trace_sse=np.array(trace_sse))
