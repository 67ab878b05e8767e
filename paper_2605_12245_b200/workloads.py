"""Seeded synthetic weight tensors for tests and benchmarks.

This module only draws random numbers and rounds them to bf16; it holds none of the
quantizer's arithmetic and is imported neither by the CUDA binding nor by the CPU
reference.  The tensors stand in for LLM weight matrices (heavy-tailed entries, a few
outlier input channels or entries), which the paper quantizes from trained checkpoints.

Recipe.  A tensor of ``rows x cols`` is drawn in row chunks of about 2**20 elements; chunk
``c`` of tensor ``i`` of a workload with seed ``s`` uses ``PCG64(SeedSequence([s, i, c]))``,
so any chunk can be produced alone and chunks can be drawn in parallel.  Values are drawn
in float32, modified (outliers), then rounded to bf16 with round-to-nearest-even; the
result is returned as uint16 bit patterns, the exact bytes both sides of a parity test use.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
import os

import numpy as np

CHUNK_ELEMS = 1 << 20


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class TensorSpec:
    name: str
    rows: int
    cols: int


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration: a list of tensors that share a distribution."""

    name: str
    seed: int
    dist: str                 # "student_t4" | "laplace" | "gauss_t2mix"
    tensors: tuple
    outlier_cols_frac: float = 0.0   # fraction of input columns scaled by outlier_scale
    outlier_entry_frac: float = 0.0  # Bernoulli fraction of entries scaled by outlier_scale
    outlier_scale: float = 1.0

    @property
    def elements(self) -> int:
        return sum(t.rows * t.cols for t in self.tensors)


def _layer(h: int, kv: int, ffn: int):
    return (
        TensorSpec("q", h, h), TensorSpec("k", kv, h), TensorSpec("v", kv, h),
        TensorSpec("o", h, h), TensorSpec("gate", ffn, h), TensorSpec("up", ffn, h),
        TensorSpec("down", h, ffn),
    )


def config1() -> Workload:
    return Workload("config1_2048x2048_t4", 0, "student_t4", (TensorSpec("w", 2048, 2048),))


def config2(seed: int = 1) -> Workload:
    return Workload("config2_qwen3_8b_layer", seed, "student_t4", _layer(4096, 1024, 12288),
                    outlier_cols_frac=0.001, outlier_scale=20.0)


def config3_layer(layer: int) -> Workload:
    return Workload(f"config3_qwen3_8b_layer{layer}", 1000 + layer, "student_t4",
                    _layer(4096, 1024, 12288), outlier_cols_frac=0.001, outlier_scale=20.0)


def config4() -> Workload:
    return Workload("config4_llama3_70b_layer", 2, "laplace", _layer(8192, 1024, 28672),
                    outlier_entry_frac=0.0005, outlier_scale=50.0)


def config5() -> Workload:
    return Workload("config5_28672x8192_gauss_t2mix", 3, "gauss_t2mix",
                    (TensorSpec("w", 28672, 8192),))


def _draw(rng: np.random.Generator, dist: str, shape) -> np.ndarray:
    if dist == "student_t4":
        # Student-t with nu=4 has variance 2; scale to standard deviation 0.02
        return (rng.standard_t(4.0, size=shape) * (0.02 / np.sqrt(2.0))).astype(np.float32)
    if dist == "laplace":
        return rng.laplace(0.0, 0.015, size=shape).astype(np.float32)
    if dist == "gauss_t2mix":
        g = rng.normal(0.0, 0.02, size=shape).astype(np.float32)
        pick = rng.random(size=shape) < 0.01
        t = (rng.standard_t(2.0, size=shape) * 0.02).astype(np.float32)
        return np.where(pick, t, g)
    raise ValueError(dist)


def _chunk_rows(cols: int) -> int:
    return max(1, CHUNK_ELEMS // cols)


def outlier_columns(wl: Workload, tensor_index: int):
    """Input columns of tensor ``tensor_index`` that carry the outlier scale."""
    if wl.outlier_cols_frac <= 0.0:
        return np.zeros(0, np.int64)
    cols = wl.tensors[tensor_index].cols
    n = max(1, int(round(wl.outlier_cols_frac * cols)))
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([wl.seed, tensor_index, 0xC01])))
    return np.sort(rng.choice(cols, size=n, replace=False))


def _gen_chunk(wl: Workload, ti: int, ci: int, r0: int, r1: int, ocols) -> np.ndarray:
    spec = wl.tensors[ti]
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([wl.seed, ti, ci])))
    x = _draw(rng, wl.dist, (r1 - r0, spec.cols))
    if wl.outlier_entry_frac > 0.0:
        hit = rng.random(size=x.shape) < wl.outlier_entry_frac
        x = np.where(hit, x * np.float32(wl.outlier_scale), x).astype(np.float32)
    if len(ocols):
        x[:, ocols] *= np.float32(wl.outlier_scale)
    return f32_to_bf16_bits(x)


def generate(wl: Workload, tensor_index: int, row_start: int = 0, row_stop: int | None = None,
             workers: int | None = None) -> np.ndarray:
    """bf16 bit patterns (uint16, [rows, cols]) of rows ``row_start:row_stop`` of one tensor.

    ``row_start`` must sit on a chunk boundary (a multiple of ``max(1, 2**20 // cols)``) so
    that the rows returned are the same whether the tensor is drawn whole or in parts.
    """
    spec = wl.tensors[tensor_index]
    row_stop = spec.rows if row_stop is None else min(row_stop, spec.rows)
    cr = _chunk_rows(spec.cols)
    assert row_start % cr == 0, "row_start must be a chunk boundary"
    ocols = outlier_columns(wl, tensor_index)
    jobs = []
    r = row_start
    while r < row_stop:
        r1 = min(r + cr, spec.rows)
        jobs.append((r // cr, r, r1))
        r = r1
    out = np.empty((jobs[-1][2] - row_start if jobs else 0, spec.cols), np.uint16)
    workers = workers or min(32, os.cpu_count() or 1)

    def run(job):
        ci, a, b = job
        out[a - row_start:b - row_start] = _gen_chunk(wl, tensor_index, ci, a, b, ocols)

    if workers > 1 and len(jobs) > 1:
        with ThreadPoolExecutor(workers) as ex:
            list(ex.map(run, jobs))
    else:
        for j in jobs:
            run(j)
    return out[: row_stop - row_start]


def small_case(rows: int, cols: int, seed: int, dist: str = "student_t4",
               outlier_cols_frac: float = 0.0, outlier_entry_frac: float = 0.0,
               outlier_scale: float = 1.0) -> np.ndarray:
    """A single small tensor with the same recipe, for parity tests."""
    wl = Workload(f"small_{rows}x{cols}", seed, dist, (TensorSpec("w", rows, cols),),
                  outlier_cols_frac, outlier_entry_frac, outlier_scale)
    return generate(wl, 0, workers=1)


def column_weights(cols: int, seed: int, samples: int = 128, outlier_frac: float = 0.005,
                   zero_frac: float = 0.0) -> np.ndarray:
    """Synthetic per-column weights for the weighted objective: float32 [cols].

    Stand-in for the diagonal of X X^T / n of a calibration batch: channel ``c`` has standard
    deviation ``sigma_c`` (log-normal, with a fraction ``outlier_frac`` of channels 10-30 times
    larger, as LLM activations show), and ``h_c = sigma_c^2 * chi2(samples) / samples``.  The
    result is scaled to mean 1, clipped to [2^-20, 2^20]; a fraction ``zero_frac`` of the
    columns is then set to zero (channels that never fire)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, cols, 0x5EED])))
    sigma = np.exp(0.5 * rng.standard_normal(cols))
    n_out = int(round(outlier_frac * cols))
    if n_out > 0:
        idx = rng.choice(cols, size=n_out, replace=False)
        sigma[idx] *= rng.uniform(10.0, 30.0, size=n_out)
    h = sigma ** 2 * rng.chisquare(samples, size=cols) / samples
    h = np.clip(h / h.mean(), 2.0 ** -20, 2.0 ** 20)
    if zero_frac > 0.0:
        h[rng.random(cols) < zero_frac] = 0.0
    return h.astype(np.float32)
