"""Thin Python binding of the C ABI in include/soar.h.

Argument marshalling only: every step of the quantizer runs in the CUDA kernels of
libsoar.so.  torch is used for device memory and streams.  There is no CPU path; importing
works without a GPU (so that symbols can be inspected), but every compute call requires
CUDA tensors, and a missing library raises instead of falling back to anything.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsoar.so")

SOAR_OK = 0
STATUS_ZERO_TENSOR, STATUS_NONFINITE, STATUS_RANGE, STATUS_INTERNAL = 1, 2, 4, 8
STATUS_BAD_WEIGHT = 16
SCALES_LINEAR, SCALES_SWIZZLED = 1, 2
PRESET_PAPER, PRESET_SINGLE_PASS, PRESET_RTN, PRESET_CJSO_ONLY, PRESET_DSS_ONLY, PRESET_COUPLED_PAIR = 0, 1, 2, 3, 4, 5
FLAG_COUPLED_SCALE, FLAG_KEEP_ALPHA, FLAG_KEEP_BLOCK_SCALE, FLAG_DETERMINISTIC = 1, 2, 4, 8
MAX_ITERS = 64

EXPORTS = (
    "soar_default_cfg", "soar_workspace_bytes", "soar_swizzled_scale_bytes", "soar_quantize",
    "soar_dequant_error", "soar_quantize_launches", "soar_status_string", "soar_quantize_host",
    "soar_trace_begin", "soar_trace_end", "soar_quantize_static", "soar_selftest_reciprocal",
    "soar_batch_workspace_bytes", "soar_quantize_batch",
    "soar_weighted_workspace_bytes", "soar_quantize_weighted", "soar_dequant_error_weighted",
    "soar_quantize_stage", "soar_pipeline_create", "soar_pipeline_run", "soar_pipeline_synchronize",
    "soar_pipeline_destroy", "soar_debug_fail_waits", "soar_mx_quantize",
    "soar_weighted_batch_workspace_bytes", "soar_quantize_weighted_batch",
)


class SoarCfg(C.Structure):
    """Mirror of ``soar_cfg``."""

    _fields_ = [
        ("struct_size", C.c_uint32), ("block", C.c_int32), ("max_iters", C.c_int32),
        ("early_stop_rel", C.c_float), ("n_dq", C.c_int32), ("n_beta", C.c_int32),
        ("beta_step_pct", C.c_int32), ("scale_layout", C.c_int32), ("flags", C.c_int32),
    ]


class SoarResult(C.Structure):
    """Mirror of ``soar_result``."""

    _fields_ = [
        ("status", C.c_int32), ("iters_run", C.c_int32), ("alpha", C.c_float), ("amax", C.c_float),
        ("sse", C.c_double), ("sse_init", C.c_double), ("sumsq", C.c_double),
        ("zero_blocks", C.c_int64), ("wide_candidates", C.c_int64),
        ("trace_alpha", C.c_double * (MAX_ITERS + 1)), ("trace_sse", C.c_double * (MAX_ITERS + 1)),
    ]


class SoarMxResult(C.Structure):
    """Mirror of ``soar_mx_result``."""

    _fields_ = [
        ("status", C.c_int32), ("amax_bits", C.c_uint32), ("amax", C.c_float), ("pad_", C.c_int32),
        ("sse", C.c_double), ("sumsq", C.c_double), ("reserved", C.c_double),
        ("zero_blocks", C.c_int64), ("wide_candidates", C.c_int64),
    ]


class SoarTensorDesc(C.Structure):
    """Mirror of ``soar_tensor_desc``."""

    _fields_ = [
        ("W_bf16", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
        ("out_fp4_packed", C.c_void_p), ("out_e4m3_scales", C.c_void_p), ("out_e4m3_scales_sw", C.c_void_p),
        ("out_global_fp32", C.c_void_p), ("out_result", C.c_void_p),
    ]


class SoarStaging(C.Structure):
    """Mirror of ``soar_staging``."""

    _fields_ = [
        ("W", C.c_void_p), ("packed", C.c_void_p), ("scales", C.c_void_p), ("scales_sw", C.c_void_p),
        ("alpha", C.c_void_p), ("result", C.c_void_p), ("workspace", C.c_void_p),
        ("workspace_bytes", C.c_size_t),
    ]


class SoarTraceEntry(C.Structure):
    """Mirror of ``soar_trace_entry``."""

    _fields_ = [("kernel", C.c_char * 32), ("launches", C.c_int64), ("total_ms", C.c_double)]


class SoarError(RuntimeError):
    pass


_lib = None


def lib() -> C.CDLL:
    """Load libsoar.so (built in-tree by ``paper_2605_12245_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SoarError(f"{LIB_PATH} is missing: run `python -m paper_2605_12245_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i64 = C.c_void_p, C.c_int64
        L.soar_default_cfg.restype = C.c_int
        L.soar_default_cfg.argtypes = [C.POINTER(SoarCfg), C.c_int]
        L.soar_workspace_bytes.restype = C.c_size_t
        L.soar_workspace_bytes.argtypes = [i64, i64, C.POINTER(SoarCfg)]
        L.soar_swizzled_scale_bytes.restype = C.c_size_t
        L.soar_swizzled_scale_bytes.argtypes = [i64, i64]
        L.soar_quantize.restype = C.c_int
        L.soar_quantize.argtypes = [vp, i64, i64, i64, C.POINTER(SoarCfg), vp, vp, vp, vp, vp,
                                    C.c_size_t, vp, vp]
        L.soar_dequant_error.restype = C.c_int
        L.soar_dequant_error.argtypes = [vp, i64, i64, i64, vp, vp, C.c_int, vp, vp, vp, vp]
        L.soar_quantize_launches.restype = C.c_int
        L.soar_quantize_launches.argtypes = [C.POINTER(SoarCfg)]
        L.soar_quantize_host.restype = C.c_int
        L.soar_quantize_host.argtypes = [vp, i64, i64, i64, C.POINTER(SoarCfg), vp, vp, vp, vp, vp,
                                         C.POINTER(SoarStaging), vp]
        L.soar_quantize_static.restype = C.c_int
        L.soar_quantize_static.argtypes = [vp, i64, i64, i64, C.POINTER(SoarCfg), vp, vp, vp, vp, vp, vp]
        L.soar_batch_workspace_bytes.restype = C.c_size_t
        L.soar_batch_workspace_bytes.argtypes = [C.POINTER(SoarTensorDesc), C.c_int, C.POINTER(SoarCfg)]
        L.soar_quantize_batch.restype = C.c_int
        L.soar_quantize_batch.argtypes = [C.POINTER(SoarTensorDesc), C.c_int, C.POINTER(SoarCfg), vp, C.c_size_t, vp]
        L.soar_weighted_workspace_bytes.restype = C.c_size_t
        L.soar_weighted_workspace_bytes.argtypes = [i64, i64, C.POINTER(SoarCfg)]
        L.soar_quantize_weighted.restype = C.c_int
        L.soar_quantize_weighted.argtypes = [vp, i64, i64, i64, vp, C.POINTER(SoarCfg), vp, vp, vp, vp, vp,
                                             C.c_size_t, vp, vp]
        L.soar_weighted_batch_workspace_bytes.restype = C.c_size_t
        L.soar_weighted_batch_workspace_bytes.argtypes = [C.POINTER(SoarTensorDesc), C.c_int, C.POINTER(SoarCfg)]
        L.soar_quantize_weighted_batch.restype = C.c_int
        L.soar_quantize_weighted_batch.argtypes = [C.POINTER(SoarTensorDesc), C.POINTER(C.c_void_p), C.c_int,
                                                   C.POINTER(SoarCfg), vp, C.c_size_t, vp]
        L.soar_dequant_error_weighted.restype = C.c_int
        L.soar_dequant_error_weighted.argtypes = [vp, i64, i64, i64, vp, vp, vp, C.c_int, vp, vp, vp, vp]
        L.soar_quantize_stage.restype = C.c_int
        L.soar_quantize_stage.argtypes = [C.POINTER(SoarTensorDesc), C.c_int, C.POINTER(SoarCfg), vp, C.c_size_t,
                                          C.c_int, vp]
        L.soar_pipeline_create.restype = C.c_int
        L.soar_pipeline_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(SoarSlot), C.c_int, vp, vp, vp]
        L.soar_pipeline_run.restype = C.c_int
        L.soar_pipeline_run.argtypes = [vp, C.POINTER(SoarHostMatrix), C.c_int, C.POINTER(SoarCfg),
                                        C.POINTER(C.c_void_p)]
        L.soar_pipeline_synchronize.restype = C.c_int
        L.soar_pipeline_synchronize.argtypes = [vp]
        L.soar_pipeline_destroy.restype = None
        L.soar_pipeline_destroy.argtypes = [vp]
        L.soar_mx_quantize.restype = C.c_int
        L.soar_mx_quantize.argtypes = [vp, i64, i64, i64, C.c_int, C.c_int, C.c_int, vp, vp, vp, vp]
        L.soar_debug_fail_waits.restype = C.c_int
        L.soar_debug_fail_waits.argtypes = [C.c_int]
        L.soar_selftest_reciprocal.restype = C.c_int
        L.soar_selftest_reciprocal.argtypes = [C.c_int, C.c_int, vp, vp]
        L.soar_trace_begin.restype = C.c_int
        L.soar_trace_begin.argtypes = []
        L.soar_trace_end.restype = C.c_int
        L.soar_trace_end.argtypes = [C.POINTER(SoarTraceEntry), C.c_int, C.POINTER(C.c_int)]
        L.soar_status_string.restype = C.c_char_p
        L.soar_status_string.argtypes = [C.c_int]
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != SOAR_OK:
        raise SoarError(f"{what}: {lib().soar_status_string(rc).decode()} ({rc})")


def soar_default_cfg(preset: int = PRESET_PAPER, **overrides) -> SoarCfg:
    cfg = SoarCfg()
    _check(lib().soar_default_cfg(C.byref(cfg), preset), "soar_default_cfg")
    for k, v in overrides.items():
        if not hasattr(cfg, k):
            raise AttributeError(k)
        setattr(cfg, k, v)
    return cfg


def soar_workspace_bytes(rows: int, cols: int, cfg: SoarCfg) -> int:
    return int(lib().soar_workspace_bytes(rows, cols, C.byref(cfg)))


def soar_swizzled_scale_bytes(rows: int, cols: int) -> int:
    return int(lib().soar_swizzled_scale_bytes(rows, cols))


def soar_quantize_launches(cfg: SoarCfg) -> int:
    return int(lib().soar_quantize_launches(C.byref(cfg)))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    if s.device.index != torch.cuda.current_device():
        raise SoarError(f"stream belongs to cuda:{s.device.index} but the current device is "
                        f"cuda:{torch.cuda.current_device()}")
    return C.c_void_p(s.cuda_stream)


def _require_cuda(*tensors):
    """Every tensor must live on the current CUDA device: the library launches there, on a stream of that
    device, and a pointer into another GPU's memory would reach kernels that cannot address it."""
    cur = torch.cuda.current_device() if torch.cuda.is_available() else None
    for t in tensors:
        if t is None:
            continue
        if not t.is_cuda:
            raise SoarError("device pointers required: tensor is not on a CUDA device")
        if t.device.index != cur:
            raise SoarError(f"tensor lives on cuda:{t.device.index} but the current device is cuda:{cur}: "
                            "make the tensor's device current (torch.cuda.device) before the call")


@dataclass
class QuantBuffers:
    """Device buffers of one quantized matrix; allocate once, reuse across calls."""

    packed: torch.Tensor            # uint8 [rows, cols/2]
    scales: torch.Tensor | None     # uint8 [rows, cols/16] (linear layout)
    scales_sw: torch.Tensor | None  # uint8 [soar_swizzled_scale_bytes]
    alpha: torch.Tensor             # float32 [1]
    result: torch.Tensor            # uint8 [sizeof(soar_result)]
    workspace: torch.Tensor         # uint8

    def read_result(self) -> SoarResult:
        """Synchronizing copy of the device report to the host."""
        raw = self.result.cpu().numpy().tobytes()
        return SoarResult.from_buffer_copy(raw)


def soar_weighted_workspace_bytes(rows: int, cols: int, cfg: SoarCfg) -> int:
    return int(lib().soar_weighted_workspace_bytes(rows, cols, C.byref(cfg)))


def alloc_buffers(rows: int, cols: int, cfg: SoarCfg, device="cuda", weighted: bool = False) -> QuantBuffers:
    """Output buffers and workspace for one matrix (``weighted``: sized for soar_quantize_weighted)."""
    u8 = dict(dtype=torch.uint8, device=device)
    lin = torch.empty((rows, cols // 16), **u8) if cfg.scale_layout & SCALES_LINEAR else None
    sw = (torch.empty(soar_swizzled_scale_bytes(rows, cols), **u8)
          if cfg.scale_layout & SCALES_SWIZZLED else None)
    ws_bytes = (soar_weighted_workspace_bytes if weighted else soar_workspace_bytes)(rows, cols, cfg)
    if ws_bytes == 0:
        raise SoarError("soar_workspace_bytes rejected the shape or cfg")
    return QuantBuffers(
        packed=torch.empty((rows, cols // 2), **u8), scales=lin, scales_sw=sw,
        alpha=torch.empty(1, dtype=torch.float32, device=device),
        result=torch.empty(C.sizeof(SoarResult), **u8),
        workspace=torch.empty(ws_bytes, **u8),
    )


def soar_quantize(W: torch.Tensor, cfg: SoarCfg, out: QuantBuffers | None = None, stream=None,
                  ld: int | None = None) -> QuantBuffers:
    """Enqueue ``soar_quantize`` for a bf16 CUDA matrix (2-D, unit column stride)."""
    _require_cuda(W)
    if W.dtype != torch.bfloat16 or W.dim() != 2 or W.stride(1) != 1:
        raise SoarError("W must be a 2-D bf16 tensor with unit column stride")
    rows, cols = W.shape
    ld = W.stride(0) if ld is None else ld
    if out is None:
        out = alloc_buffers(rows, cols, cfg, W.device)
    _require_cuda(out.packed, out.scales, out.scales_sw, out.alpha, out.result, out.workspace)
    rc = lib().soar_quantize(
        _ptr(W), rows, cols, ld, C.byref(cfg), _ptr(out.packed), _ptr(out.scales),
        _ptr(out.scales_sw), _ptr(out.alpha), _ptr(out.workspace), out.workspace.numel(),
        _ptr(out.result), _stream_ptr(stream))
    _check(rc, "soar_quantize")
    return out


def soar_quantize_weighted(W: torch.Tensor, col_weight: torch.Tensor, cfg: SoarCfg,
                           out: QuantBuffers | None = None, stream=None) -> QuantBuffers:
    """Enqueue ``soar_quantize_weighted``: ``col_weight`` is a float32 CUDA vector of W.shape[1] entries."""
    _require_cuda(W, col_weight)
    if W.dtype != torch.bfloat16 or W.dim() != 2 or W.stride(1) != 1:
        raise SoarError("W must be a 2-D bf16 tensor with unit column stride")
    rows, cols = W.shape
    if col_weight.dtype != torch.float32 or col_weight.shape != (cols,) or not col_weight.is_contiguous():
        raise SoarError("col_weight must be a contiguous float32 vector with one entry per column")
    if out is None:
        out = alloc_buffers(rows, cols, cfg, W.device, weighted=True)
    _require_cuda(out.packed, out.scales, out.scales_sw, out.alpha, out.result, out.workspace)
    rc = lib().soar_quantize_weighted(
        _ptr(W), rows, cols, W.stride(0), _ptr(col_weight), C.byref(cfg), _ptr(out.packed), _ptr(out.scales),
        _ptr(out.scales_sw), _ptr(out.alpha), _ptr(out.workspace), out.workspace.numel(),
        _ptr(out.result), _stream_ptr(stream))
    _check(rc, "soar_quantize_weighted")
    return out


def _descs(Ws, outs):
    d = (SoarTensorDesc * len(Ws))()
    for i, (W, o) in enumerate(zip(Ws, outs)):
        _require_cuda(W, o.packed, o.scales, o.scales_sw, o.alpha, o.result)
        if W.dtype != torch.bfloat16 or W.dim() != 2 or W.stride(1) != 1:
            raise SoarError("W must be a 2-D bf16 tensor with unit column stride")
        nul = lambda t: None if t is None else t.data_ptr()  # noqa: E731
        d[i] = SoarTensorDesc(W.data_ptr(), W.shape[0], W.shape[1], W.stride(0), o.packed.data_ptr(),
                              nul(o.scales), nul(o.scales_sw), o.alpha.data_ptr(), nul(o.result))
    return d


def soar_batch_workspace_bytes(Ws, outs, cfg: SoarCfg) -> int:
    d = _descs(Ws, outs)
    return int(lib().soar_batch_workspace_bytes(d, len(Ws), C.byref(cfg)))


def soar_quantize_batch(Ws, cfg: SoarCfg, outs, workspace: torch.Tensor | None = None, stream=None):
    """Enqueue ``soar_quantize_batch`` for a list of bf16 CUDA matrices; ``outs`` are their
    ``QuantBuffers`` (their own ``workspace`` fields are not used), ``workspace`` one uint8 CUDA
    tensor of ``soar_batch_workspace_bytes`` (allocated here when omitted).  Returns it."""
    d = _descs(Ws, outs)
    if workspace is None:
        need = int(lib().soar_batch_workspace_bytes(d, len(Ws), C.byref(cfg)))
        if need == 0:
            raise SoarError("soar_batch_workspace_bytes rejected the shapes or cfg")
        workspace = torch.empty(need, dtype=torch.uint8, device=Ws[0].device)
    _require_cuda(workspace)
    rc = lib().soar_quantize_batch(d, len(Ws), C.byref(cfg), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    _check(rc, "soar_quantize_batch")
    return workspace


def soar_quantize_weighted_batch(Ws, col_weights, cfg: SoarCfg, outs, workspace: torch.Tensor | None = None,
                                 stream=None):
    """Enqueue ``soar_quantize_weighted_batch``: a list of bf16 CUDA matrices, one float32 CUDA weight vector per
    matrix, their ``QuantBuffers`` (own ``workspace`` fields unused) and one uint8 CUDA ``workspace`` of
    ``soar_weighted_batch_workspace_bytes`` (allocated here when omitted).  Returns the workspace."""
    d = _descs(Ws, outs)
    n = len(Ws)
    for W, h in zip(Ws, col_weights):
        _require_cuda(h)
        if h.dtype != torch.float32 or h.shape != (W.shape[1],) or not h.is_contiguous():
            raise SoarError("each col_weight must be a contiguous float32 vector with one entry per column")
    if workspace is None:
        need = int(lib().soar_weighted_batch_workspace_bytes(d, n, C.byref(cfg)))
        if need == 0:
            raise SoarError("soar_weighted_batch_workspace_bytes rejected the shapes or cfg")
        workspace = torch.empty(need, dtype=torch.uint8, device=Ws[0].device)
    _require_cuda(workspace)
    hp = (C.c_void_p * n)(*[h.data_ptr() for h in col_weights])
    rc = lib().soar_quantize_weighted_batch(d, hp, n, C.byref(cfg), _ptr(workspace), workspace.numel(),
                                            _stream_ptr(stream))
    _check(rc, "soar_quantize_weighted_batch")
    return workspace


STATIC_MAX_ELEMENTS = 1 << 24


STAGE_AMAX, STAGE_INIT, STAGE_FINALIZE = -3, -2, -1
WORKSPACE_HEADER_BYTES = 2048


class SoarWorkspaceHeader(C.Structure):
    """Mirror of ``soar_workspace_header`` (used for field offsets only)."""

    _fields_ = [
        ("amax_bits", C.c_uint32), ("error", C.c_uint32), ("zero_blocks", C.c_uint64), ("wide", C.c_uint64),
        ("sumsq", C.c_double), ("num", C.c_double * (MAX_ITERS + 1)), ("den", C.c_double * (MAX_ITERS + 1)),
        ("gsum", C.c_double * (MAX_ITERS + 1)),
    ]


def soar_quantize_stage(Ws, cfg: SoarCfg, outs, workspace: torch.Tensor, stage: int, stream=None) -> None:
    """Enqueue one stage of ``soar_quantize_batch`` (``STAGE_AMAX``, ``STAGE_INIT``, iteration ``t >= 0``,
    ``STAGE_FINALIZE``) for the matrices ``Ws`` with output buffers ``outs`` and a shared ``workspace``."""
    d = _descs(Ws, outs)
    _require_cuda(workspace)
    rc = lib().soar_quantize_stage(d, len(Ws), C.byref(cfg), _ptr(workspace), workspace.numel(), int(stage),
                                   _stream_ptr(stream))
    _check(rc, "soar_quantize_stage")


def soar_quantize_static(W: torch.Tensor, cfg: SoarCfg, out: QuantBuffers, stream=None) -> QuantBuffers:
    """Enqueue ``soar_quantize_static``: the quantizer for callers that cannot allocate device
    memory.  ``out`` supplies the output tensors only; its ``workspace`` is not passed on (the
    library uses its built-in scratch), and matrices above ``STATIC_MAX_ELEMENTS`` are refused."""
    _require_cuda(W, out.packed, out.scales, out.scales_sw, out.alpha, out.result)
    if W.dtype != torch.bfloat16 or W.dim() != 2 or W.stride(1) != 1:
        raise SoarError("W must be a 2-D bf16 tensor with unit column stride")
    rows, cols = W.shape
    rc = lib().soar_quantize_static(
        _ptr(W), rows, cols, W.stride(0), C.byref(cfg), _ptr(out.packed), _ptr(out.scales),
        _ptr(out.scales_sw), _ptr(out.alpha), _ptr(out.result), _stream_ptr(stream))
    _check(rc, "soar_quantize_static")
    return out


@dataclass
class MxBuffers:
    """Device outputs of one MXFP4 call."""

    packed: torch.Tensor      # uint8 [rows, cols/2]
    scales: torch.Tensor      # uint8 [rows, cols/32], E8M0 codes
    result: torch.Tensor      # uint8 [sizeof(soar_mx_result)]

    def read_result(self) -> SoarMxResult:
        return SoarMxResult.from_buffer_copy(self.result.cpu().numpy().tobytes())


def soar_mx_quantize(W: torch.Tensor, n_dq: int = 2, n_beta: int = 101, beta_step_pct: int = 1,
                     out: MxBuffers | None = None, stream=None) -> MxBuffers:
    """Enqueue ``soar_mx_quantize`` (MXFP4, blocks of 32; ``n_beta == 0``: the format's plain rule)."""
    _require_cuda(W)
    if W.dtype != torch.bfloat16 or W.dim() != 2 or W.stride(1) != 1:
        raise SoarError("W must be a 2-D bf16 tensor with unit column stride")
    rows, cols = W.shape
    if out is None:
        u8 = dict(dtype=torch.uint8, device=W.device)
        out = MxBuffers(torch.empty((rows, cols // 2), **u8), torch.empty((rows, max(cols // 32, 1)), **u8),
                        torch.empty(C.sizeof(SoarMxResult), **u8))
    _require_cuda(out.packed, out.scales, out.result)
    rc = lib().soar_mx_quantize(_ptr(W), rows, cols, W.stride(0), n_dq, n_beta, beta_step_pct, _ptr(out.packed),
                                _ptr(out.scales), _ptr(out.result), _stream_ptr(stream))
    _check(rc, "soar_mx_quantize")
    return out


def soar_dequant_error(W: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor,
                       alpha: torch.Tensor, scale_layout: int = SCALES_LINEAR, stream=None,
                       out: torch.Tensor | None = None) -> torch.Tensor:
    """Enqueue ``soar_dequant_error``; returns a float64 CUDA tensor [sse, sumsq]."""
    _require_cuda(W, packed, scales, alpha)
    rows, cols = W.shape
    if out is None:
        out = torch.empty(2, dtype=torch.float64, device=W.device)
    rc = lib().soar_dequant_error(
        _ptr(W), rows, cols, W.stride(0), _ptr(packed), _ptr(scales), scale_layout, _ptr(alpha),
        C.c_void_p(out.data_ptr()), C.c_void_p(out.data_ptr() + 8), _stream_ptr(stream))
    _check(rc, "soar_dequant_error")
    return out


def soar_dequant_error_weighted(W: torch.Tensor, col_weight: torch.Tensor, packed: torch.Tensor,
                                scales: torch.Tensor, alpha: torch.Tensor, scale_layout: int = SCALES_LINEAR,
                                stream=None, out: torch.Tensor | None = None) -> torch.Tensor:
    """Enqueue ``soar_dequant_error_weighted``; returns a float64 CUDA tensor [sse, sumsq]."""
    _require_cuda(W, col_weight, packed, scales, alpha)
    rows, cols = W.shape
    if out is None:
        out = torch.empty(2, dtype=torch.float64, device=W.device)
    rc = lib().soar_dequant_error_weighted(
        _ptr(W), rows, cols, W.stride(0), _ptr(col_weight), _ptr(packed), _ptr(scales), scale_layout,
        _ptr(alpha), C.c_void_p(out.data_ptr()), C.c_void_p(out.data_ptr() + 8), _stream_ptr(stream))
    _check(rc, "soar_dequant_error_weighted")
    return out


@dataclass
class HostBuffers:
    """Page-locked host buffers for one matrix, inputs and outputs of soar_quantize_host."""

    W: torch.Tensor                  # bf16 [rows, cols], pinned
    packed: torch.Tensor             # uint8 [rows, cols/2], pinned
    scales: torch.Tensor | None
    scales_sw: torch.Tensor | None
    alpha: torch.Tensor              # float32 [1], pinned
    result: torch.Tensor             # uint8 [sizeof(soar_result)], pinned

    def read_result(self) -> SoarResult:
        return SoarResult.from_buffer_copy(self.result.numpy().tobytes())


def alloc_host_buffers(rows: int, cols: int, cfg: SoarCfg) -> HostBuffers:
    pin = dict(pin_memory=True)
    lin = torch.empty((rows, cols // 16), dtype=torch.uint8, **pin) if cfg.scale_layout & SCALES_LINEAR else None
    sw = (torch.empty(soar_swizzled_scale_bytes(rows, cols), dtype=torch.uint8, **pin)
          if cfg.scale_layout & SCALES_SWIZZLED else None)
    return HostBuffers(
        W=torch.empty((rows, cols), dtype=torch.bfloat16, **pin),
        packed=torch.empty((rows, cols // 2), dtype=torch.uint8, **pin), scales=lin, scales_sw=sw,
        alpha=torch.empty(1, dtype=torch.float32, **pin),
        result=torch.empty(C.sizeof(SoarResult), dtype=torch.uint8, **pin))


def soar_quantize_host(host: HostBuffers, cfg: SoarCfg, dev_W: torch.Tensor, dev: QuantBuffers,
                       stream=None) -> None:
    """Enqueue ``soar_quantize_host``: H2D copy of ``host.W``, the quantizer, D2H copies of
    every output, in order on ``stream``.  ``dev_W``/``dev`` are the device staging buffers."""
    _require_cuda(dev_W, dev.packed, dev.scales, dev.scales_sw, dev.alpha, dev.result, dev.workspace)
    rows, cols = host.W.shape
    if tuple(dev_W.shape) != (rows, cols) or dev_W.dtype != torch.bfloat16 or not dev_W.is_contiguous():
        raise SoarError("dev_W must be a contiguous bf16 tensor of the host matrix's shape")
    st = SoarStaging(dev_W.data_ptr(), dev.packed.data_ptr(),
                     dev.scales.data_ptr() if dev.scales is not None else None,
                     dev.scales_sw.data_ptr() if dev.scales_sw is not None else None,
                     dev.alpha.data_ptr(), dev.result.data_ptr(), dev.workspace.data_ptr(),
                     dev.workspace.numel())
    rc = lib().soar_quantize_host(
        _ptr(host.W), rows, cols, cols, C.byref(cfg), _ptr(host.packed), _ptr(host.scales),
        _ptr(host.scales_sw), _ptr(host.alpha), _ptr(host.result), C.byref(st), _stream_ptr(stream))
    _check(rc, "soar_quantize_host")


class SoarSlot(C.Structure):
    """Mirror of ``soar_slot``."""

    _fields_ = [("dev", SoarStaging), ("W_bytes", C.c_size_t), ("packed_bytes", C.c_size_t),
                ("scales_bytes", C.c_size_t), ("scales_sw_bytes", C.c_size_t)]


class SoarHostMatrix(C.Structure):
    """Mirror of ``soar_host_matrix``."""

    _fields_ = [("W_host", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
                ("out_fp4_packed_host", C.c_void_p), ("out_e4m3_scales_host", C.c_void_p),
                ("out_e4m3_scales_sw_host", C.c_void_p), ("out_global_host", C.c_void_p),
                ("out_result_host", C.c_void_p)]


class HostPipeline:
    """``soar_pipeline_*`` of the C ABI: quantizes matrices that live in pinned host memory with the
    copies in, the quantizer and the copies out overlapped on three streams over ``depth`` device
    staging slots sized for the largest matrix.  This class allocates the slots and the streams and
    marshals the lists; the chaining is the library's."""

    def __init__(self, shapes, cfg: SoarCfg, depth: int = 3, device="cuda", weighted: bool = False):
        self.cfg = cfg
        self.weighted = weighted
        rows, cols = max(shapes, key=lambda rc: rc[0] * rc[1])
        sw_bytes = max(soar_swizzled_scale_bytes(r, c) for r, c in shapes) if cfg.scale_layout & SCALES_SWIZZLED else 0
        ws_bytes = max((soar_weighted_workspace_bytes if weighted else soar_workspace_bytes)(r, c, cfg)
                       for r, c in shapes)
        self._keep = []                                  # the slots' tensors
        slots = (SoarSlot * depth)()
        for i in range(depth):
            W = torch.empty(rows * cols, dtype=torch.bfloat16, device=device)
            out = alloc_buffers(rows, cols, cfg, device, weighted=weighted)
            if out.scales_sw is not None and out.scales_sw.numel() < sw_bytes:
                out.scales_sw = torch.empty(sw_bytes, dtype=torch.uint8, device=device)
            if out.workspace.numel() < ws_bytes:
                out.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
            _require_cuda(W, out.packed, out.scales, out.scales_sw, out.alpha, out.result, out.workspace)
            self._keep.append((W, out))
            nul = lambda t: None if t is None else t.data_ptr()  # noqa: E731
            slots[i] = SoarSlot(
                SoarStaging(W.data_ptr(), out.packed.data_ptr(), nul(out.scales), nul(out.scales_sw),
                            out.alpha.data_ptr(), out.result.data_ptr(), out.workspace.data_ptr(),
                            out.workspace.numel()),
                W.numel() * 2, out.packed.numel(), 0 if out.scales is None else out.scales.numel(),
                0 if out.scales_sw is None else out.scales_sw.numel())
        self.h2d, self.compute, self.d2h = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        self._handle = C.c_void_p()
        _check(lib().soar_pipeline_create(C.byref(self._handle), slots, depth, _stream_ptr(self.h2d),
                                          _stream_ptr(self.compute), _stream_ptr(self.d2h)), "soar_pipeline_create")

    def run(self, hosts, col_weights=None) -> None:
        """Enqueue the whole list (``HostBuffers`` each); results are in the host buffers once
        ``synchronize()`` returns.  Calls may follow one another without a synchronize in
        between: the copies of the next list then overlap the work on the previous one.
        ``col_weights``: one float32 CUDA vector per matrix for the weighted objective (the
        pipeline must have been built with ``weighted=True``)."""
        if col_weights is not None and not self.weighted:
            raise SoarError("this pipeline's workspaces are not sized for the weighted objective")
        n = len(hosts)
        mats = (SoarHostMatrix * n)()
        nul = lambda t: None if t is None else t.data_ptr()  # noqa: E731
        for i, hb in enumerate(hosts):
            rows, cols = hb.W.shape
            mats[i] = SoarHostMatrix(hb.W.data_ptr(), rows, cols, hb.W.stride(0), hb.packed.data_ptr(), nul(hb.scales),
                                     nul(hb.scales_sw), hb.alpha.data_ptr(), hb.result.data_ptr())
        wp = None
        if col_weights is not None:
            _require_cuda(*col_weights)
            wp = (C.c_void_p * n)(*[h.data_ptr() for h in col_weights])
        _check(lib().soar_pipeline_run(self._handle, mats, n, C.byref(self.cfg), wp), "soar_pipeline_run")

    def synchronize(self) -> None:
        _check(lib().soar_pipeline_synchronize(self._handle), "soar_pipeline_synchronize")

    def close(self) -> None:
        if self._handle:
            lib().soar_pipeline_destroy(self._handle)
            self._handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def soar_selftest_reciprocal(lo_exp: int = 2, hi_exp: int = 252, stream=None) -> int:
    """Runs ``soar_selftest_reciprocal`` and returns the mismatch count (synchronizes)."""
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    _check(lib().soar_selftest_reciprocal(lo_exp, hi_exp, _ptr(out), _stream_ptr(stream)), "soar_selftest_reciprocal")
    return int(out.cpu()[0])


def soar_debug_fail_waits(on: bool) -> None:
    """Test hook: while on, the kernels' waits for tiles run out (see ``soar_debug_fail_waits`` in soar.h)."""
    _check(lib().soar_debug_fail_waits(1 if on else 0), "soar_debug_fail_waits")


def soar_trace_begin() -> None:
    _check(lib().soar_trace_begin(), "soar_trace_begin")


def soar_trace_end() -> dict:
    """Stops tracing; returns {kernel name: (launches, total device ms)}."""
    buf = (SoarTraceEntry * 16)()
    n = C.c_int(0)
    _check(lib().soar_trace_end(buf, 16, C.byref(n)), "soar_trace_end")
    return {buf[i].kernel.decode(): (int(buf[i].launches), float(buf[i].total_ms)) for i in range(min(n.value, 16))}
