"""ctypes loader for the CPU reference oracle (oracle/soar_ref.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this module.
It builds ``libsoar_ref.so`` beside the source with gcc when the object is missing or
older than the source, and marshals NumPy arrays into the C calls.  It holds none of the
method's arithmetic: that lives in the C file, which follows the SOAR paper
(Sec. 3.1-3.4, App. B.3, Algorithm 1).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "soar_ref.c")
_LIB = os.path.join(_HERE, "libsoar_ref.so")

STATUS_ZERO_TENSOR = 1
STATUS_NONFINITE = 2
STATUS_RANGE = 4
STATUS_BAD_WEIGHT = 16

FLAG_COUPLED_SCALE, FLAG_KEEP_ALPHA, FLAG_KEEP_BLOCK_SCALE = 1, 2, 4

GCC_FLAGS = ["-O2", "-msse4.1", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *GCC_FLAGS, _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [
        ("max_iters", C.c_int32),
        ("early_stop_rel", C.c_float),
        ("n_dq", C.c_int32),
        ("n_beta", C.c_int32),
        ("beta_step_pct", C.c_int32),
        ("flags", C.c_int32),
    ]


@dataclass
class RefCfg:
    """Search settings; the defaults are the paper's (Sec. 4.1, App. B.3)."""

    max_iters: int = 15
    early_stop_rel: float = 1e-3
    n_dq: int = 2
    n_beta: int = 101
    beta_step_pct: int = 1
    flags: int = 0            # FLAG_* bits: the paper's stand-alone arms (Sec. 3.2, Sec. 3.3)

    def c(self) -> _Cfg:
        return _Cfg(self.max_iters, self.early_stop_rel, self.n_dq, self.n_beta, self.beta_step_pct,
                    self.flags)


@dataclass
class RefResult:
    packed: np.ndarray        # uint8 [rows, cols/2]
    scales: np.ndarray        # uint8 [rows, cols/16]
    alpha: float              # binary32 value
    iters_run: int
    trace_alpha: np.ndarray   # float64 [iters_run+1]
    trace_sse: np.ndarray     # float64 [iters_run+1]
    tie_flags: np.ndarray     # uint8 [rows, cols/16]
    sumsq: float
    status: int


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u16p, u8p = C.POINTER(C.c_uint16), C.POINTER(C.c_uint8)
        dp = C.POINTER(C.c_double)
        L.soar_ref_bf16_to_f32.restype = C.c_float
        L.soar_ref_bf16_to_f32.argtypes = [C.c_uint16]
        L.soar_ref_e2m1_round.restype = C.c_double
        L.soar_ref_e2m1_round.argtypes = [C.c_double]
        L.soar_ref_e2m1_code.restype = C.c_int
        L.soar_ref_e2m1_code.argtypes = [C.c_double]
        L.soar_ref_e4m3_decode.restype = C.c_float
        L.soar_ref_e4m3_decode.argtypes = [C.c_uint8]
        L.soar_ref_e4m3_encode.restype = C.c_uint8
        L.soar_ref_e4m3_encode.argtypes = [C.c_float]
        L.soar_ref_round_block.restype = None
        L.soar_ref_round_block.argtypes = [u16p, C.c_float, C.c_float, dp, dp, dp]
        L.soar_ref_block_error.restype = C.c_double
        L.soar_ref_block_error.argtypes = [u16p, dp, C.c_float, C.c_uint8]
        fp = C.POINTER(C.c_float)
        L.soar_ref_round_block_w.restype = None
        L.soar_ref_round_block_w.argtypes = [u16p, fp, C.c_float, C.c_float, dp, dp, dp]
        L.soar_ref_block_error_w.restype = C.c_double
        L.soar_ref_block_error_w.argtypes = [u16p, fp, dp, C.c_float, C.c_uint8]
        L.soar_ref_block_scale.restype = C.c_float
        L.soar_ref_block_scale.argtypes = [C.c_double, C.c_double, C.c_float, C.c_uint8]
        L.soar_ref_dq_candidates.restype = C.c_int
        L.soar_ref_dq_candidates.argtypes = [C.c_float, C.c_int, u8p]
        L.soar_ref_beta.restype = C.c_float
        L.soar_ref_beta.argtypes = [C.c_int, C.c_int, C.c_int]
        L.soar_ref_quantize.restype = C.c_int
        L.soar_ref_quantize.argtypes = [
            u16p, C.c_int64, C.c_int64, C.c_int64, C.POINTER(_Cfg), u8p, u8p,
            C.POINTER(C.c_float), C.POINTER(C.c_int32), dp, dp, u8p, C.c_double, dp,
        ]
        L.soar_ref_dequant_error.restype = None
        L.soar_ref_dequant_error.argtypes = [
            u16p, C.c_int64, C.c_int64, C.c_int64, u8p, u8p, C.c_float, dp, dp,
        ]
        L.soar_ref_quantize_weighted.restype = C.c_int
        L.soar_ref_quantize_weighted.argtypes = [
            u16p, C.c_int64, C.c_int64, C.c_int64, fp, C.POINTER(_Cfg), u8p, u8p,
            C.POINTER(C.c_float), C.POINTER(C.c_int32), dp, dp, u8p, C.c_double, dp,
        ]
        L.soar_ref_dequant_error_weighted.restype = None
        L.soar_ref_dequant_error_weighted.argtypes = [
            u16p, C.c_int64, C.c_int64, C.c_int64, fp, u8p, u8p, C.c_float, dp, dp,
        ]
        L.soar_ref_e8m0_decode.restype = C.c_double
        L.soar_ref_e8m0_decode.argtypes = [C.c_uint8]
        L.soar_ref_mx_plain_code.restype = C.c_uint8
        L.soar_ref_mx_plain_code.argtypes = [C.c_float]
        L.soar_ref_mx_candidates.restype = C.c_int
        L.soar_ref_mx_candidates.argtypes = [C.c_float, C.c_int, u8p]
        L.soar_ref_mx_round_block.restype = None
        L.soar_ref_mx_round_block.argtypes = [u16p, C.c_float, dp]
        L.soar_ref_mx_block_error.restype = C.c_double
        L.soar_ref_mx_block_error.argtypes = [u16p, dp, C.c_uint8]
        L.soar_ref_mx_quantize.restype = C.c_int
        L.soar_ref_mx_quantize.argtypes = [u16p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int,
                                           u8p, u8p, dp, dp, u8p, C.c_double]
        L.soar_ref_num_threads.restype = C.c_int
        _lib = L
    return _lib


def _u16(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_uint16))


def _u8(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_uint8))


def num_threads() -> int:
    return int(lib().soar_ref_num_threads())


def _f32(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _weights(h, cols: int):
    """Column weights as a contiguous float32 array of ``cols`` entries (None stays None)."""
    if h is None:
        return None
    h = np.ascontiguousarray(h, dtype=np.float32)
    assert h.shape == (cols,)
    return h


def quantize(w_bits: np.ndarray, cfg: RefCfg, tie_rel: float = 1e-6, h=None) -> RefResult:
    """Run Algorithm 1 on a 2-D uint16 array of bf16 bit patterns (row stride = shape[1]).

    ``h``: optional float32 column weights of the objective (Sec. 5, diagonal form)."""
    assert w_bits.dtype == np.uint16 and w_bits.ndim == 2
    rows, cols = w_bits.shape
    assert cols % 16 == 0
    h = _weights(h, cols)
    w = np.ascontiguousarray(w_bits)
    packed = np.zeros((rows, cols // 2), np.uint8)
    scales = np.zeros((rows, cols // 16), np.uint8)
    ties = np.zeros((rows, cols // 16), np.uint8)
    ta = np.zeros(cfg.max_iters + 1, np.float64)
    ts = np.zeros(cfg.max_iters + 1, np.float64)
    alpha = C.c_float(0.0)
    iters = C.c_int32(0)
    sumsq = C.c_double(0.0)
    c = cfg.c()
    tail = (C.byref(c), _u8(packed), _u8(scales), C.byref(alpha), C.byref(iters),
            ta.ctypes.data_as(C.POINTER(C.c_double)), ts.ctypes.data_as(C.POINTER(C.c_double)),
            _u8(ties), tie_rel, C.byref(sumsq))
    if h is None:
        st = lib().soar_ref_quantize(_u16(w), rows, cols, cols, *tail)
    else:
        st = lib().soar_ref_quantize_weighted(_u16(w), rows, cols, cols, _f32(h), *tail)
    n = iters.value + 1
    return RefResult(packed, scales, float(alpha.value), int(iters.value), ta[:n].copy(),
                     ts[:n].copy(), ties, float(sumsq.value), int(st))


def dequant_error(w_bits: np.ndarray, packed: np.ndarray, scales: np.ndarray, alpha: float, h=None):
    """Sum of (column-weighted) squared reconstruction error (Eq. 3-4) and sum of squares of W."""
    rows, cols = w_bits.shape
    w = np.ascontiguousarray(w_bits)
    p = np.ascontiguousarray(packed, dtype=np.uint8)
    s = np.ascontiguousarray(scales, dtype=np.uint8)
    h = _weights(h, cols)
    sse, ss = C.c_double(0.0), C.c_double(0.0)
    if h is None:
        lib().soar_ref_dequant_error(_u16(w), rows, cols, cols, _u8(p), _u8(s), C.c_float(alpha),
                                     C.byref(sse), C.byref(ss))
    else:
        lib().soar_ref_dequant_error_weighted(_u16(w), rows, cols, cols, _f32(h), _u8(p), _u8(s),
                                              C.c_float(alpha), C.byref(sse), C.byref(ss))
    return float(sse.value), float(ss.value)


# ---- single-step wrappers used by the pins -------------------------------------------------

def e2m1_round(x: float) -> float:
    return float(lib().soar_ref_e2m1_round(float(x)))


def e2m1_code(m: float) -> int:
    return int(lib().soar_ref_e2m1_code(float(m)))


def e4m3_decode(code: int) -> float:
    return float(lib().soar_ref_e4m3_decode(int(code)))


def e4m3_encode(v: float) -> int:
    return int(lib().soar_ref_e4m3_encode(C.c_float(v)))


def round_block(w16: np.ndarray, alpha: float, dq: float, h=None):
    """Returns (m[16], A, B) for one block of bf16 bit patterns (``h``: its 16 column weights)."""
    w = np.ascontiguousarray(w16, dtype=np.uint16)
    assert w.size == 16
    m = np.zeros(16, np.float64)
    A, B = C.c_double(0.0), C.c_double(0.0)
    mp = m.ctypes.data_as(C.POINTER(C.c_double))
    if h is None:
        lib().soar_ref_round_block(_u16(w), C.c_float(alpha), C.c_float(dq), mp, C.byref(A), C.byref(B))
    else:
        hh = _weights(h, 16)
        lib().soar_ref_round_block_w(_u16(w), _f32(hh), C.c_float(alpha), C.c_float(dq), mp,
                                     C.byref(A), C.byref(B))
    return m, float(A.value), float(B.value)


def block_error(w16: np.ndarray, m: np.ndarray, alpha: float, d: int, h=None) -> float:
    w = np.ascontiguousarray(w16, dtype=np.uint16)
    mm = np.ascontiguousarray(m, dtype=np.float64)
    mp = mm.ctypes.data_as(C.POINTER(C.c_double))
    if h is None:
        return float(lib().soar_ref_block_error(_u16(w), mp, C.c_float(alpha), C.c_uint8(d)))
    hh = _weights(h, 16)
    return float(lib().soar_ref_block_error_w(_u16(w), _f32(hh), mp, C.c_float(alpha), C.c_uint8(d)))


def block_scale(A: float, B: float, alpha: float, d_cur: int) -> float:
    return float(lib().soar_ref_block_scale(A, B, C.c_float(alpha), C.c_uint8(d_cur)))


def dq_candidates(center: float, n: int):
    out = np.zeros(32, np.uint8)
    k = lib().soar_ref_dq_candidates(C.c_float(center), n, _u8(out))
    return [int(v) for v in out[:k]]


def beta(k: int, n_beta: int, step_pct: int) -> float:
    return float(lib().soar_ref_beta(k, n_beta, step_pct))


# ---- MXFP4 (Sec. 4.3 "DSS on MXFP4") ------------------------------------------------------

@dataclass
class RefMxResult:
    packed: np.ndarray        # uint8 [rows, cols/2]
    scales: np.ndarray        # uint8 [rows, cols/32], E8M0 codes
    sse: float
    sumsq: float
    tie_flags: np.ndarray     # uint8 [rows, cols/32]
    status: int


def mx_quantize(w_bits: np.ndarray, n_dq: int = 2, n_beta: int = 101, beta_step_pct: int = 1,
                tie_rel: float = 1e-6) -> RefMxResult:
    """MXFP4 of a 2-D uint16 array of bf16 bit patterns; ``n_beta == 0`` is the format's plain rule."""
    assert w_bits.dtype == np.uint16 and w_bits.ndim == 2 and w_bits.shape[1] % 32 == 0
    rows, cols = w_bits.shape
    w = np.ascontiguousarray(w_bits)
    packed = np.zeros((rows, cols // 2), np.uint8)
    scales = np.zeros((rows, cols // 32), np.uint8)
    ties = np.zeros((rows, cols // 32), np.uint8)
    sse, ss = C.c_double(0.0), C.c_double(0.0)
    st = lib().soar_ref_mx_quantize(_u16(w), rows, cols, cols, n_dq, n_beta, beta_step_pct, _u8(packed), _u8(scales),
                                    C.byref(sse), C.byref(ss), _u8(ties), tie_rel)
    return RefMxResult(packed, scales, float(sse.value), float(ss.value), ties, int(st))


def e8m0_decode(code: int) -> float:
    return float(lib().soar_ref_e8m0_decode(int(code)))


def mx_plain_code(bmax: float) -> int:
    return int(lib().soar_ref_mx_plain_code(C.c_float(bmax)))


def mx_candidates(center: float, n: int):
    out = np.zeros(32, np.uint8)
    k = lib().soar_ref_mx_candidates(C.c_float(center), n, _u8(out))
    return [int(v) for v in out[:k]]


def mx_round_block(w32: np.ndarray, dq: float) -> np.ndarray:
    w = np.ascontiguousarray(w32, dtype=np.uint16)
    assert w.size == 32
    m = np.zeros(32, np.float64)
    lib().soar_ref_mx_round_block(_u16(w), C.c_float(dq), m.ctypes.data_as(C.POINTER(C.c_double)))
    return m


def mx_block_error(w32: np.ndarray, m: np.ndarray, code: int) -> float:
    w = np.ascontiguousarray(w32, dtype=np.uint16)
    mm = np.ascontiguousarray(m, dtype=np.float64)
    return float(lib().soar_ref_mx_block_error(_u16(w), mm.ctypes.data_as(C.POINTER(C.c_double)), C.c_uint8(code)))
