"""One tensor split by rows over several GPUs (one process per GPU).

The blocks of a tensor meet in three places only (Algorithm 1): the maximum of Eq. 1, the two
sums of Eq. 5, and the error that Sec. 4.1's early stop watches.  The library keeps those in the
2 KB header of the workspace (``soar_workspace_header``) and can run its kernels one stage at a
time (``soar_quantize_stage``).  So each rank quantizes its own rows, and after every stage the
ranks combine the header fields that stage wrote: one all-reduce with MAX and one with SUM, a
few dozen bytes each, on the stream the kernels run on.  Every rank then holds the whole
tensor's values, so alpha, the iteration at which the search stops and the report are the same
everywhere, and no weight, code or scale ever crosses a link.

This module holds the stage schedule and the header plumbing; it works on CPU tensors too
(gloo), which is how the plumbing is tested without GPUs.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import api

MAX, SUM = "max", "sum"


def stages(max_iters: int) -> list[int]:
    """The stages of one call, in order."""
    return [api.STAGE_AMAX, api.STAGE_INIT, *range(max_iters), api.STAGE_FINALIZE]


def _field(name: str, index: int = 0):
    f = getattr(api.SoarWorkspaceHeader, name)
    dtype = {"amax_bits": torch.int32, "error": torch.int32, "zero_blocks": torch.int64,
             "wide": torch.int64}.get(name, torch.float64)
    size = torch.empty(0, dtype=dtype).element_size()
    return dtype, f.offset + index * size


def fields_written(stage: int, max_iters: int) -> list[tuple[str, int, str]]:
    """(field, index, how to combine) for the header entries to combine after the given stage.

    Each sum is combined once, right after the stage that writes it.  The counter ``wide`` grows
    in the init stage and in every iteration and is only read by the report, so it is combined
    once, after the last stage before the report; ``error`` may be set by any stage and is
    combined with MAX every time (which may be repeated freely)."""
    last_before_report = max_iters - 1 if max_iters > 0 else api.STAGE_INIT
    tail = [("wide", 0, SUM)] if stage == last_before_report else []
    if stage == api.STAGE_AMAX:
        return [("amax_bits", 0, MAX), ("error", 0, MAX), ("sumsq", 0, SUM)]
    if stage == api.STAGE_INIT:
        return [("error", 0, MAX), ("num", 0, SUM), ("den", 0, SUM), ("gsum", 0, SUM),
                ("zero_blocks", 0, SUM)] + tail
    if stage == api.STAGE_FINALIZE:
        return []
    if stage < 0 or stage >= max_iters:
        raise ValueError("unknown stage")
    t = stage + 1
    return [("error", 0, MAX), ("num", t, SUM), ("den", t, SUM), ("gsum", t, SUM)] + tail


def header_view(header: torch.Tensor, name: str, index: int = 0) -> torch.Tensor:
    """A one-element view of a header field inside the uint8 tensor that holds the header."""
    dtype, off = _field(name, index)
    size = torch.empty(0, dtype=dtype).element_size()
    return header[off:off + size].view(dtype)


def combine_header(header: torch.Tensor, stage: int, max_iters: int, all_reduce) -> None:
    """Combine, over all parts of the tensor, the header entries due after ``stage``.

    ``header`` is the uint8 tensor of the first ``WORKSPACE_HEADER_BYTES`` bytes of this part's
    workspace; ``all_reduce(buffer, how)`` reduces a float64 tensor in place over the parts with
    ``how`` in {"max", "sum"}.  Counters and bit patterns travel as float64, which holds them
    exactly (they are below 2^53)."""
    todo = fields_written(stage, max_iters)
    for how in (MAX, SUM):
        views = [header_view(header, n, i) for n, i, h in todo if h == how]
        if not views:
            continue
        buf = torch.cat([v.to(torch.float64) for v in views])
        all_reduce(buf, how)
        for k, v in enumerate(views):
            v.copy_(buf[k:k + 1].to(v.dtype))


def dist_all_reduce(group=None):
    """The ``all_reduce`` argument of ``combine_header`` over a torch.distributed group."""
    def run(buf: torch.Tensor, how: str) -> None:
        dist.all_reduce(buf, op=dist.ReduceOp.MAX if how == MAX else dist.ReduceOp.SUM, group=group)
    return run


def quantize_rows(W_local: torch.Tensor, cfg: api.SoarCfg, out: api.QuantBuffers | None = None,
                  group=None) -> api.QuantBuffers:
    """This rank's rows of a tensor that is split by rows over the ranks of ``group``.

    ``W_local`` is the rank's bf16 slice [rows_local, cols] on its GPU; the outputs are the
    slice's codes and scales, and the whole tensor's alpha and report.  Everything is enqueued
    on the current stream; nothing synchronizes with the host."""
    rows, cols = W_local.shape
    if out is None:
        out = api.alloc_buffers(rows, cols, cfg, W_local.device)
    header = out.workspace[:api.WORKSPACE_HEADER_BYTES]
    reduce = dist_all_reduce(group)
    for stage in stages(cfg.max_iters):
        api.soar_quantize_stage([W_local], cfg, [out], out.workspace, stage)
        combine_header(header, stage, cfg.max_iters, reduce)
    return out
