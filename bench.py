#!/usr/bin/env python
"""Benchmark of the SOAR NVFP4 quantize pass on B200.

One "step" quantizes every tensor of the workload once (the whole hot path: tensor
maximum, max-based start, the CJSO + DSS iterations, alpha and the report), through the
C-ABI library with all inputs already resident in HBM.  Prints ONE JSON line on stdout.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload config1|config2|config3|config4|config5] [--preset paper|single_pass]

Multi-GPU runs are one rank per GPU under torch.distributed.run (started by the caller, or by
this script itself when --gpus N is given to a plain process); the tensors of a model are
independent, so every rank quantizes its own copy of the workload with no collective on the
data path (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_12245_b200 import workloads as WL  # noqa: E402

SM_COUNT = 148


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, sm_max_mhz=1965.0, source="fallback")


class FlatWorkload:
    """The tensors of one or several workloads as one list (config 3 is 36 layer workloads)."""

    def __init__(self, name, parts):
        self.name = name
        self.sources = [(wl, i) for wl in parts for i in range(len(wl.tensors))]
        self.tensors = tuple(wl.tensors[i] for wl, i in self.sources)

    @property
    def elements(self) -> int:
        return sum(t.rows * t.cols for t in self.tensors)

    def generate(self, i, *a, **kw):
        wl, ti = self.sources[i]
        return WL.generate(wl, ti, *a, **kw)


def pick_workload(name: str, rank: int = 0) -> FlatWorkload:
    """``rank`` > 0 draws the same shapes from a seed of its own (weak scaling: one layer per rank)."""
    from paper_2605_12245_b200 import sharding as SH
    single = {"config1": WL.config1, "config2": WL.config2, "config4": WL.config4, "config5": WL.config5}
    if name in single:
        wl = SH.rank_workload(single[name](), rank)
        return FlatWorkload(wl.name, [wl])
    if name == "config3":
        return FlatWorkload("config3_qwen3_8b_36_layers" + (f"_rank{rank}" if rank else ""),
                            [SH.rank_workload(WL.config3_layer(l), rank) for l in range(36)])
    raise SystemExit(f"unknown workload {name}")


def preset_cfg(api, preset: str, args=None, **over):
    """The preset's settings; ``--pairs K`` and ``--iters T`` override the candidate grid and the
    iteration count (K pairs per block = n_beta x n_dq with n_dq = min(2, K); no early stop)."""
    base = {"paper": api.PRESET_PAPER, "single_pass": api.PRESET_SINGLE_PASS,
            "coupled_pair": api.PRESET_COUPLED_PAIR}[preset]
    if args is not None and args.pairs:
        n_dq = min(2, args.pairs)
        over.update(n_dq=n_dq, n_beta=max(1, args.pairs // n_dq))
    if args is not None and args.iters is not None:
        over.update(max_iters=args.iters, early_stop_rel=0.0)
    cfg = api.soar_default_cfg(base, **over)
    if args is not None and getattr(args, "deterministic", False):
        cfg.flags |= api.FLAG_DETERMINISTIC
    return cfg


def ref_cfg_of(R, cfg):
    return R.RefCfg(max_iters=cfg.max_iters, early_stop_rel=cfg.early_stop_rel, n_dq=cfg.n_dq,
                    n_beta=cfg.n_beta, beta_step_pct=cfg.beta_step_pct, flags=cfg.flags)


def ref_preset_cfg(R, preset: str, args):
    """The oracle's settings for a preset, from the oracle's own defaults (the paper's: Sec. 4.1, App. B.3)
    and the same command-line overrides as ``preset_cfg``; the CUDA library plays no part in it."""
    c = R.RefCfg()
    if preset == "single_pass":
        c = R.RefCfg(max_iters=1, early_stop_rel=0.0, n_dq=2, n_beta=1)
    elif preset == "coupled_pair":
        c = R.RefCfg(n_dq=2, n_beta=1, flags=R.FLAG_COUPLED_SCALE)
    if args.pairs:
        c.n_dq = min(2, args.pairs)
        c.n_beta = max(1, args.pairs // c.n_dq)
    if args.iters is not None:
        c.max_iters, c.early_stop_rel = args.iters, 0.0
    return c


OUT_BYTES = 0.5 + 1.0 / 16          # codes + scale byte per element
STATE_BYTES = 0.5                   # 8 bytes of carried sums per 16-element block


def kernel_bytes_per_elem(name: str, cfg, t: int = 0) -> float:
    """Algorithmic HBM bytes per weight element of one launch (iteration ``t`` for iterate)."""
    if name == "amax_kernel":
        return 2.0                                                   # read W
    if name == "init_kernel":                                        # read W; write state, or the outputs when T = 0
        return 2.0 + (STATE_BYTES if cfg.max_iters > 0 else OUT_BYTES)
    if name == "iterate_kernel":                                     # read W + state; write state unless last; outputs
        last = t == cfg.max_iters - 1
        emits = last or cfg.early_stop_rel > 0
        return 2.0 + STATE_BYTES + (0.0 if last else STATE_BYTES) + (OUT_BYTES if emits else 0.0)
    if name == "dequant_error_kernel":
        return 2.0 + OUT_BYTES
    return 0.0


# DRAM bytes per element (dram__bytes_read.sum + dram__bytes_write.sum of one launch, ncu, config 5:
# profiles/single_pass_kernels_config5.md, profiles/iterate_kernel_paper_config5.md and
# profiles/weighted_iterate_kernel_config5.md).  Traffic grows in
# proportion to the elements, so a launch's traffic is this figure times its elements.  The figures
# belong to one version of the kernels: they are dropped when the device part of the source (everything above
# the host-side section of soar.cu) no longer matches.
NCU_TRAFFIC = {
    "kernel_source_sha256_16": "01bec268fb069bbc",
    "bytes_per_elem": {"amax_kernel": 2.02, "init_kernel": 2.44, "iterate_kernel/single": 3.01,
                       "iterate_kernel/grid": 3.47, "weighted_iterate_kernel": 4.57},
    "inst_per_block": {"amax_kernel": 125, "init_kernel": 218, "iterate_kernel/single": 258,
                       "iterate_kernel/grid": 490, "weighted_iterate_kernel": 1204},
}


HOST_MARKER = b"// ------------------------------------------------------------------ host side"


def kernel_source_hash() -> str | None:
    """sha256 (16 hex digits) of the device part of soar.cu: everything above the host-side section."""
    src = os.path.join(ROOT, "paper_2605_12245_b200", "csrc", "soar.cu")
    import hashlib
    try:
        with open(src, "rb") as f:
            text = f.read()
    except OSError:
        return None
    if HOST_MARKER not in text:
        return None
    return hashlib.sha256(text.split(HOST_MARKER)[0]).hexdigest()[:16]


def _profile_key(name: str, cfg) -> str:
    if name == "iterate_kernel":
        name += "/single" if cfg.n_beta == 1 and not (cfg.n_dq > 2 and cfg.flags & 1) else "/grid"
    return name


def ncu_traffic_per_elem(name: str, cfg):
    if kernel_source_hash() != NCU_TRAFFIC["kernel_source_sha256_16"]:
        return None
    return NCU_TRAFFIC["bytes_per_elem"].get(_profile_key(name, cfg))


def ncu_inst_per_block(name: str, cfg):
    """Executed instructions per 16-element block and launch (ncu, same captures), or None once the kernels changed."""
    if kernel_source_hash() != NCU_TRAFFIC["kernel_source_sha256_16"]:
        return None
    return NCU_TRAFFIC["inst_per_block"].get(_profile_key(name, cfg))


def call_bytes_per_elem(cfg, iters_run: int) -> float:
    """Algorithmic HBM bytes per element of one soar_quantize call that ran ``iters_run`` iterations."""
    return (kernel_bytes_per_elem("amax_kernel", cfg) + kernel_bytes_per_elem("init_kernel", cfg)
            + sum(kernel_bytes_per_elem("iterate_kernel", cfg, t) for t in range(iters_run)))


def oracle_one_thread(R, w, rcfg, h=None):
    """The oracle on one host thread (a per-core figure): the OpenMP runtime's own switch, called from
    here; the oracle is run as it stands.  Returns None when the runtime cannot be reached."""
    import ctypes
    try:
        gomp = ctypes.CDLL("libgomp.so.1")
        before = R.num_threads()
        gomp.omp_set_num_threads(1)
    except (OSError, AttributeError):
        return None
    try:
        t0 = time.perf_counter()
        ref = R.quantize(w, rcfg, h=h)
        dt = time.perf_counter() - t0
    finally:
        gomp.omp_set_num_threads(before)
    return dict(value=2.0 * w.size / dt / 1e9, unit="GB/s", elements_per_s=w.size / dt,
                sample=f"{w.shape[0]} rows x {w.shape[1]} cols, {ref.iters_run} iterations, {dt:.1f} s")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "25"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        # samples under load: the upper half of the observed clocks (idle samples sit far below)
        load = sorted(sm)[len(sm) // 2:] if sm else []
        return dict(sm_mhz=statistics.median(load) if load else None,
                    sm_max_mhz=max(mx) if mx else None, samples=len(sm), reasons=sorted(reasons))


def run_reference(args):
    """The CPU oracle as it stands, on a bounded sample of the same workload and preset."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import soar_ref as R
    wl = pick_workload(args.workload)
    cfg = rcfg = ref_preset_cfg(R, args.preset, args)
    spec = wl.tensors[0]
    rows = min(spec.rows, max(1, args.ref_rows))
    rows = max(1, rows // WL._chunk_rows(spec.cols)) * WL._chunk_rows(spec.cols)
    w = wl.generate(0, 0, rows)
    h = WL.column_weights(spec.cols, 1000) if args.objective == "weighted" else None
    for _ in range(args.warmup):
        R.quantize(w, rcfg, h=h)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        R.quantize(w, rcfg, h=h)
    dt = (time.perf_counter() - t0) / args.steps
    value = 2.0 * w.size / dt / 1e9
    sample = f"{rows} rows x {spec.cols} cols of tensor '{spec.name}' of {wl.name} per step"
    line = dict(
        impl="reference", metric="soar_quantize_bf16_input_throughput", value=value, unit="GB/s",
        n_gpus=args.gpus, steps=args.steps, warmup=args.warmup, ms_per_step=dt * 1e3,
        higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f32", data="synthetic",
        config=dict(workload=wl.name, preset=args.preset, max_iters=cfg.max_iters, n_beta=cfg.n_beta,
                    n_dq=cfg.n_dq, early_stop_rel=cfg.early_stop_rel, sample=sample,
                    **({"objective": "column-weighted"} if h is not None else {})),
        cpu_baseline=dict(value=value, unit="GB/s", cores=R.num_threads(), kind="oracle", sample=sample),
        e2e=dict(value=value, unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0),
        elements_per_s=w.size / dt, gpu_launches=0,
    )
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2605_12245_b200 import api
    from paper_2605_12245_b200 import sharding as SH

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    api.lib()
    peaks = load_peaks()
    wl = pick_workload(args.workload, rank)
    cfg = preset_cfg(api, args.preset, args)

    # ---- inputs: generated on the host (seeded), resident in HBM before timing
    host_w, dev_w, outs = [], [], []
    for i, spec in enumerate(wl.tensors):
        bits = wl.generate(i)
        h = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
        host_w.append(h)
        dev_w.append(h.cuda())
        outs.append(api.alloc_buffers(spec.rows, spec.cols, cfg))
    elements = wl.elements
    stream = torch.cuda.current_stream()

    batch_ws = {}

    def step(c=cfg, st=None):
        """One pass over the workload: one batched call (or one call per tensor with --no-batch)."""
        st = stream if st is None else st
        if args.no_batch:
            for W, o in zip(dev_w, outs):
                api.soar_quantize(W, c, o, st)
            return
        key = (c.max_iters, c.scale_layout, c.flags)
        if key not in batch_ws:
            batch_ws[key] = torch.empty(api.soar_batch_workspace_bytes(dev_w, outs, c), dtype=torch.uint8, device="cuda")
        api.soar_quantize_batch(dev_w, c, outs, batch_ws[key], st)

    eager_step = step
    if args.graph:
        # replay the step's launches from a CUDA graph: takes the host's launch cost out of the picture
        side = torch.cuda.Stream()
        graphs = {}

        def graphed(c):
            key = (c.max_iters, c.n_beta, c.n_dq, c.early_stop_rel)
            if key not in graphs:
                g = torch.cuda.CUDAGraph()
                torch.cuda.synchronize()
                eager_step(c, side)                      # allocate the workspace outside the capture
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=side):
                    eager_step(c, side)
                graphs[key] = g
            return graphs[key]

        def step(c=cfg):  # noqa: F811
            graphed(c).replay()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, trace=True):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if trace:
            api.soar_trace_begin()
        t0 = time.perf_counter()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        host_ms.append((time.perf_counter() - t0) * 1e3 / steps)      # host clock, final synchronize included
        tr = api.soar_trace_end() if trace else {}
        barrier()
        ms = SH.max_over_ranks(e0.elapsed_time(e1) / steps, "cuda")
        return ms, tr

    host_ms = []
    sampler = ClockSampler(local)
    sampler.start()
    # headline: K steps with nothing between the kernels; then the same K steps again with an
    # event pair around every kernel (which costs a few microseconds per launch) for the shares
    ms, _ = timed(step, args.steps, args.warmup, trace=False)
    traced_ms, trace = timed(eager_step if args.graph else step, args.steps, 0, trace=True)
    clocks = sampler.stop()
    results = [o.read_result() for o in outs]
    iters = [r.iters_run for r in results]
    value = world * 2.0 * elements / (ms * 1e-3) / 1e9
    launches = sum(v[0] for v in trace.values())

    # ---- the timed batch's outputs against one soar_quantize call per tensor (same bytes expected)
    bad = []
    for i, (W, o) in enumerate(zip(dev_w, outs)):
        one = api.soar_quantize(W, cfg)
        torch.cuda.synchronize()
        if not (torch.equal(one.packed, o.packed) and torch.equal(one.scales, o.scales) and torch.equal(one.alpha, o.alpha)
                and one.read_result().iters_run == iters[i]):
            bad.append(i)
        del one
    outputs_checked = dict(tensors=len(outs), differing_from_single_calls=bad)
    packed0 = outs[0].packed.cpu()            # the later sections reuse the output buffers
    if bad:
        raise SystemExit(f"batched outputs differ from per-tensor calls for tensors {bad}")

    # ---- roofline of the dominant kernel: its algorithmic bytes over its measured device time, against the
    # measured HBM copy bandwidth; beside it the issue-slot side from the committed profile
    dom = max(trace, key=lambda k: trace[k][1])
    n_launch, tot_ms = trace[dom]
    if args.no_batch:
        active = sum(iters) if dom == "iterate_kernel" else len(wl.tensors)
    else:      # one launch serves a group of up to 16 tensors; an iteration launch works while any of them runs
        groups = [iters[i:i + 16] for i in range(0, len(iters), 16)]
        active = sum(max(g) for g in groups) if dom == "iterate_kernel" else len(groups)
    tpe = ncu_traffic_per_elem(dom, cfg)
    work_elems = (sum(s.rows * s.cols * it for s, it in zip(wl.tensors, iters)) if dom == "iterate_kernel"
                  else elements)
    traffic = None if tpe is None or active == 0 else tpe * work_elems / active
    if dom == "iterate_kernel":
        byts = sum(s.rows * s.cols * kernel_bytes_per_elem(dom, cfg, t)
                   for s, it in zip(wl.tensors, iters) for t in range(it)) * args.steps
    else:
        byts = elements * args.steps * kernel_bytes_per_elem(dom, cfg)
    achieved = byts / (tot_ms * 1e-3) / 1e9
    ipb = ncu_inst_per_block(dom, cfg)
    issue = None
    if ipb is not None and dom == "iterate_kernel":
        warp_inst = ipb * (work_elems / 16) / 32 * args.steps
        issue_peak = SM_COUNT * 4 * peaks["sm_max_mhz"] * 1e6            # one warp instruction per scheduler and clock
        issue = dict(instructions_per_block=ipb, frac_of_issue_peak=warp_inst / (tot_ms * 1e-3) / issue_peak,
                     peak="148 SMs x 4 schedulers x clocks.max.sm", source="ncu, profiles/ (same kernel source)")
    roofline = dict(bound="hbm", kernel=dom, achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], traffic=traffic, launches=n_launch,
                    active_launches=active * args.steps, kernel_ms_per_step=tot_ms / args.steps,
                    peak_source=peaks["source"], frac_of_nominal_8000=achieved / 8000.0, issue=issue)
    call_bytes = sum(s.rows * s.cols * call_bytes_per_elem(cfg, it) for s, it in zip(wl.tensors, iters))
    call_gbs = world * call_bytes / (ms * 1e-3) / 1e9
    whole_call = dict(algorithmic_bytes_per_step=call_bytes, achieved_gbs=call_gbs,
                      frac_of_measured_hbm=call_gbs / world / peaks["hbm_gbs"],
                      frac_of_nominal_8000=call_gbs / world / 8000.0)
    kernels = {k: dict(launches=v[0], ms_per_step=v[1] / args.steps, share=v[1] / sum(x[1] for x in trace.values()))
               for k, v in trace.items()}

    # ---- the HBM-bound shape of the same path (T=1, beta={1}, 2 neighbours), for the bandwidth bar
    extra = {}
    if args.preset == "paper" and not args.no_single_pass:
        sp = preset_cfg(api, "single_pass")
        sp_ms, _ = timed(lambda: step(sp), max(args.steps, 5), 3, trace=False)
        _, sp_tr = timed(lambda: (eager_step if args.graph else step)(sp), max(args.steps, 5), 0, trace=True)
        sp_bytes = elements * call_bytes_per_elem(sp, sp.max_iters)
        gbs = sp_bytes / (sp_ms * 1e-3) / 1e9
        extra["single_pass"] = dict(
            ms_per_step=sp_ms, value=world * 2.0 * elements / (sp_ms * 1e-3) / 1e9, unit="GB/s",
            algorithmic_bytes_per_step=sp_bytes, achieved_gbs=gbs, frac_of_measured_hbm=gbs / peaks["hbm_gbs"],
            frac_of_nominal_8000=gbs / 8000.0,
            kernels={k: dict(launches=v[0], ms_per_step=v[1] / max(args.steps, 5),
                             achieved_gbs=(elements * kernel_bytes_per_elem(k, sp, 0) * max(args.steps, 5)
                                           / (v[1] * 1e-3) / 1e9) if v[1] > 0 else None,
                             traffic_bytes_per_elem=ncu_traffic_per_elem(k, sp))
                     for k, v in sp_tr.items()})

    # ---- the error check of Eq. 3-4 on the outputs just produced (its own entry point, not part of a step)
    err_out = torch.empty(2, dtype=torch.float64, device="cuda")

    def err_step():
        for W, o in zip(dev_w, outs):
            api.soar_dequant_error(W, o.packed, o.scales, o.alpha, stream=stream, out=err_out)

    err_ms, _ = timed(err_step, max(args.steps, 5), 3, trace=False)
    err_bytes = elements * kernel_bytes_per_elem("dequant_error_kernel", cfg)
    extra["dequant_error"] = dict(ms_per_step=err_ms, achieved_gbs=err_bytes / (err_ms * 1e-3) / 1e9,
                                  frac_of_measured_hbm=err_bytes / (err_ms * 1e-3) / 1e9 / peaks["hbm_gbs"])

    # ---- candidate-count sweep (config 5's purpose: where the search loop overtakes HBM); one iteration each
    if args.sweep:
        rows_out = []
        for K in [int(x) for x in args.sweep.split(",")]:
            n_dq = min(2, K)
            c = api.soar_default_cfg(api.PRESET_SINGLE_PASS, n_dq=n_dq, n_beta=max(1, K // n_dq))
            k_ms, _ = timed(lambda: step(c), max(args.steps, 5), 3, trace=False)
            k_bytes = elements * call_bytes_per_elem(c, 1)
            rows_out.append(dict(pairs=c.n_dq * c.n_beta, n_beta=c.n_beta, n_dq=c.n_dq, ms_per_step=k_ms,
                                 value=world * 2.0 * elements / (k_ms * 1e-3) / 1e9, unit="GB/s",
                                 achieved_gbs=k_bytes / (k_ms * 1e-3) / 1e9,
                                 frac_of_measured_hbm=k_bytes / (k_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]))
        extra["sweep"] = rows_out
    if args.sweep_dq:      # the other axis: one quantization scale (beta = 1), K E4M3 codes around it
        rows_out = []
        for K in [int(x) for x in args.sweep_dq.split(",")]:
            c = api.soar_default_cfg(api.PRESET_SINGLE_PASS, n_dq=K, n_beta=1)
            k_ms, _ = timed(lambda: step(c), max(args.steps, 5), 3, trace=False)
            k_bytes = elements * call_bytes_per_elem(c, 1)
            rows_out.append(dict(n_dq=K, n_beta=1, ms_per_step=k_ms, value=world * 2.0 * elements / (k_ms * 1e-3) / 1e9,
                                 unit="GB/s", achieved_gbs=k_bytes / (k_ms * 1e-3) / 1e9,
                                 frac_of_measured_hbm=k_bytes / (k_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]))
        extra["sweep_dq"] = rows_out

    # ---- end to end through the C ABI's host-buffer pipeline (soar_pipeline_run): pinned host buffers in and out,
    # every copy inside the timed region
    import ctypes
    ctypes_sizeof_result = ctypes.sizeof(api.SoarResult)
    e2e = None
    if not args.no_e2e:
        # config 3 would pin 18 GB: its 36 layers go through a ring of four layers' worth of pinned buffers
        # (36 x 7 copies in and out per step all the same; layer l reads the ring's layer l mod 4)
        per_layer = 7 if args.workload == "config3" else len(wl.tensors)
        ring_layers = 4 if args.workload == "config3" else 1
        pipe = api.HostPipeline([(s.rows, s.cols) for s in wl.tensors[:per_layer]], cfg, depth=6)
        hosts = []
        for h, spec in zip(host_w[:per_layer * ring_layers], wl.tensors):
            hb = api.alloc_host_buffers(spec.rows, spec.cols, cfg)
            hb.W.copy_(h)
            hosts.append(hb)
        order = [hosts[i % len(hosts)] for i in range(len(wl.tensors))]

        def e2e_step():
            pipe.run(order)

        for _ in range(2):
            e2e_step()
        pipe.synchronize()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            e2e_step()
        pipe.synchronize()
        dt = (time.perf_counter() - t0) / args.steps
        dt = SH.max_over_ranks(dt, "cuda")
        # results must equal the resident-input run
        r_last = hosts[(len(wl.tensors) - 1) % len(hosts)].read_result()
        assert r_last.status == 0 and hosts[0].read_result().iters_run == iters[0]
        assert torch.equal(hosts[0].packed, packed0)
        e2e = dict(value=world * 2.0 * elements / dt / 1e9, unit="GB/s", ms_per_step=dt * 1e3,
                   h2d_bytes_per_step=2 * elements,
                   d2h_bytes_per_step=elements // 2 + elements // 16 + len(wl.tensors) * (4 + ctypes_sizeof_result),
                   api="soar_pipeline_run (C ABI): pinned host buffers, copy-in / soar_quantize / copy-out on three "
                       "streams over 6 device slots",
                   host_buffers=("%d distinct pinned layers reused in turn" % ring_layers) if ring_layers > 1
                   else "one pinned buffer set per tensor")
        pipe.close()

    # ---- the oracle on the host cores, bounded sample (rank 0, single GPU only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        from oracle import soar_ref as R
        spec = wl.tensors[0]
        rows = max(1, min(spec.rows, args.cpu_rows) // WL._chunk_rows(spec.cols)) * WL._chunk_rows(spec.cols)
        w = host_w[0][:rows].view(torch.int16).numpy().view(np.uint16)
        t0 = time.perf_counter()
        ref = R.quantize(w, ref_cfg_of(R, cfg))
        dt = time.perf_counter() - t0
        cpu = dict(value=2.0 * w.size / dt / 1e9, unit="GB/s", cores=R.num_threads(), kind="oracle",
                   sample=f"first {rows} rows x {spec.cols} cols of tensor '{spec.name}', {ref.iters_run} iterations, {dt:.1f} s",
                   elements_per_s=w.size / dt,
                   one_thread=oracle_one_thread(R, w[: max(1, rows // 16)], ref_cfg_of(R, cfg)))

    if rank == 0:
        line = dict(
            metric="soar_quantize_bf16_input_throughput", value=value, unit="GB/s", n_gpus=world,
            steps=args.steps, warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak",
            vs_baseline=None, dtype="f32", data="synthetic",
            config=dict(workload=wl.name, preset=args.preset, max_iters=cfg.max_iters, n_beta=cfg.n_beta,
                        n_dq=cfg.n_dq, early_stop_rel=cfg.early_stop_rel, tensors=len(wl.tensors),
                        elements=elements, iters_run=iters,
                        l2="inputs (%.2f GB per step) exceed the 126 MB L2" % (2 * elements / 1e9),
                        parallelism=f"{world} rank(s), one layer of these shapes each, no collective"),
            elements_per_s=world * elements / (ms * 1e-3), host_clock_ms_per_step=host_ms[0],
            hbm_frac_end_to_end_of_measured=value / peaks["hbm_gbs"],
            traced_ms_per_step=traced_ms, cuda_graph=bool(args.graph), batched=not args.no_batch, roofline=roofline,
            whole_call=whole_call, kernels=kernels, outputs_checked=outputs_checked, cpu_baseline=cpu, e2e=e2e,
            gpu_launches=launches, clocks=clocks, **extra)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


WEIGHTED_STATE_BYTES = 17.0 / 16    # {A, B} in binary64 and the scale code per 16-element block


def weighted_kernel_bytes_per_elem(name: str, cfg, t: int = 0) -> float:
    if name == "weighted_amax_kernel":
        return 2.0
    if name == "weighted_init_kernel":
        return 2.0 + (WEIGHTED_STATE_BYTES if cfg.max_iters > 0 else OUT_BYTES)
    if name == "weighted_iterate_kernel":
        last = t == cfg.max_iters - 1
        emits = last or cfg.early_stop_rel > 0
        return 2.0 + WEIGHTED_STATE_BYTES + (0.0 if last else WEIGHTED_STATE_BYTES) + (OUT_BYTES if emits else 0.0)
    return 0.0


def run_weighted(args):
    """The same step under the column-weighted objective: one soar_quantize_weighted_batch call over the
    workload's tensors, W and the column weights resident in HBM."""
    import torch
    from ctypes import byref as ctypes_byref

    from paper_2605_12245_b200 import api
    from paper_2605_12245_b200 import sharding as SH

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    api.lib()
    peaks = load_peaks()
    wl = pick_workload(args.workload, rank)
    cfg = preset_cfg(api, args.preset, args)
    host_w, host_h, dev_w, dev_h, outs = [], [], [], [], []
    for i, spec in enumerate(wl.tensors):
        bits = wl.generate(i)
        hw = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
        hh = torch.from_numpy(WL.column_weights(spec.cols, 1000 * (rank + 1) + i))
        host_w.append(hw)
        host_h.append(hh)
        dev_w.append(hw.cuda())
        dev_h.append(hh.cuda())
        outs.append(api.alloc_buffers(spec.rows, spec.cols, cfg, weighted=True))
    elements = wl.elements
    stream = torch.cuda.current_stream()

    batch_ws = torch.empty(int(api.lib().soar_weighted_batch_workspace_bytes(api._descs(dev_w, outs), len(dev_w),
                                                                             ctypes_byref(cfg))),
                           dtype=torch.uint8, device="cuda")

    def step():
        """One batched call over the workload's tensors (one call per tensor with --no-batch)."""
        if args.no_batch:
            for W, h, o in zip(dev_w, dev_h, outs):
                api.soar_quantize_weighted(W, h, cfg, o, stream)
        else:
            api.soar_quantize_weighted_batch(dev_w, dev_h, cfg, outs, batch_ws, stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, trace):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if trace:
            api.soar_trace_begin()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        tr = api.soar_trace_end() if trace else {}
        barrier()
        return SH.max_over_ranks(e0.elapsed_time(e1) / steps, "cuda"), tr

    sampler = ClockSampler(local)
    sampler.start()
    ms, _ = timed(step, args.steps, args.warmup, False)
    traced_ms, trace = timed(step, args.steps, 0, True)
    clocks = sampler.stop()
    results = [o.read_result() for o in outs]
    iters = [r.iters_run for r in results]
    value = world * 2.0 * elements / (ms * 1e-3) / 1e9
    launches = sum(v[0] for v in trace.values())
    dom = max(trace, key=lambda k: trace[k][1])
    n_launch, tot_ms = trace[dom]
    it_bytes = sum(s.rows * s.cols * weighted_kernel_bytes_per_elem("weighted_iterate_kernel", cfg, t)
                   for s, it in zip(wl.tensors, iters) for t in range(it)) * args.steps
    byts = it_bytes if dom == "weighted_iterate_kernel" else elements * args.steps * weighted_kernel_bytes_per_elem(dom, cfg)
    achieved = byts / (tot_ms * 1e-3) / 1e9
    tpe = ncu_traffic_per_elem(dom, cfg)
    work_elems = sum(s.rows * s.cols * it for s, it in zip(wl.tensors, iters))
    roofline = dict(bound="hbm", kernel=dom, achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"],
                    traffic=None if tpe is None or sum(iters) == 0 or dom != "weighted_iterate_kernel"
                    else tpe * work_elems / sum(iters),
                    launches=n_launch, active_launches=sum(iters) * args.steps if dom == "weighted_iterate_kernel" else n_launch,
                    kernel_ms_per_step=tot_ms / args.steps, peak_source=peaks["source"],
                    frac_of_nominal_8000=achieved / 8000.0,
                    note="the block sums carry arbitrary weights, so they are binary64 sums in element order: "
                         "the pass is bound by binary64 issue, not by HBM")
    kernels = {k: dict(launches=v[0], ms_per_step=v[1] / args.steps, share=v[1] / sum(x[1] for x in trace.values()))
               for k, v in trace.items()}

    # what the weights buy: weighted error of this run against the weighted error of the unweighted method's output
    gain = None
    if rank == 0:
        plain = api.soar_quantize(dev_w[0], cfg)
        e = api.soar_dequant_error_weighted(dev_w[0], dev_h[0], plain.packed, plain.scales, plain.alpha).cpu().numpy()
        gain = dict(tensor=wl.tensors[0].name, weighted_rel_error=results[0].sse / results[0].sumsq,
                    weighted_rel_error_of_unweighted_run=float(e[0] / e[1]),
                    weighted_rel_error_of_max_based_start=results[0].sse_init / results[0].sumsq)
        del plain

    # ---- end to end: pinned host buffers in and out, copies inside the timed region
    e2e = None
    if not args.no_e2e and args.workload != "config3":
        pipe = api.HostPipeline([(s.rows, s.cols) for s in wl.tensors], cfg, depth=6, weighted=True)
        hosts = []
        for hsrc, spec in zip(host_w, wl.tensors):
            hb = api.alloc_host_buffers(spec.rows, spec.cols, cfg)
            hb.W.copy_(hsrc)
            hosts.append(hb)

        def e2e_step():
            pipe.run(hosts, dev_h)

        for _ in range(2):
            e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            e2e_step()
        torch.cuda.synchronize()
        dt = SH.max_over_ranks((time.perf_counter() - t0) / args.steps, "cuda")
        import ctypes
        e2e = dict(value=world * 2.0 * elements / dt / 1e9, unit="GB/s", ms_per_step=dt * 1e3,
                   h2d_bytes_per_step=2 * elements,
                   d2h_bytes_per_step=elements // 2 + elements // 16 + len(wl.tensors) * (4 + ctypes.sizeof(api.SoarResult)),
                   api="soar_pipeline_run (C ABI): pinned host buffers, copy-in / soar_quantize_weighted / copy-out on "
                       "three streams over 6 device slots (the column weights stay on the device)")
        pipe.close()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        from oracle import soar_ref as R
        spec = wl.tensors[0]
        rows = max(1, min(spec.rows, args.cpu_rows) // WL._chunk_rows(spec.cols)) * WL._chunk_rows(spec.cols)
        w = host_w[0][:rows].view(torch.int16).numpy().view(np.uint16)
        t0 = time.perf_counter()
        ref = R.quantize(w, ref_cfg_of(R, cfg), h=host_h[0].numpy())
        dt = time.perf_counter() - t0
        cpu = dict(value=2.0 * w.size / dt / 1e9, unit="GB/s", cores=R.num_threads(), kind="oracle",
                   sample=f"first {rows} rows x {spec.cols} cols of tensor '{spec.name}', {ref.iters_run} iterations, {dt:.1f} s",
                   elements_per_s=w.size / dt,
                   one_thread=oracle_one_thread(R, w[: max(1, rows // 16)], ref_cfg_of(R, cfg), h=host_h[0].numpy()))

    if rank == 0:
        line = dict(
            metric="soar_quantize_bf16_input_throughput", value=value, unit="GB/s", n_gpus=world,
            steps=args.steps, warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak",
            vs_baseline=None, dtype="f64", data="synthetic",
            config=dict(workload=wl.name, objective="column-weighted", preset=args.preset, max_iters=cfg.max_iters,
                        n_beta=cfg.n_beta, n_dq=cfg.n_dq, early_stop_rel=cfg.early_stop_rel, tensors=len(wl.tensors),
                        elements=elements, iters_run=iters,
                        l2="inputs (%.2f GB per step) exceed the 126 MB L2" % (2 * elements / 1e9),
                        parallelism=f"{world} rank(s), one layer of these shapes each, no collective"),
            elements_per_s=world * elements / (ms * 1e-3), traced_ms_per_step=traced_ms, roofline=roofline,
            kernels=kernels, cpu_baseline=cpu, e2e=e2e, gpu_launches=launches, clocks=clocks, weighting_gain=gain)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_mxfp4(args):
    """The MXFP4 entry point (Sec. 4.3, DSS on MXFP4) on the same workloads: one soar_mx_quantize call per tensor,
    W resident in HBM; one pass over W per call."""
    import torch

    from paper_2605_12245_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    api.lib()
    peaks = load_peaks()
    wl = pick_workload(args.workload)
    n_beta = 0 if args.preset == "single_pass" else 101         # single_pass here: the format's plain rule
    dev_w, outs = [], []
    for i, spec in enumerate(wl.tensors):
        dev_w.append(torch.from_numpy(wl.generate(i).view(np.int16)).view(torch.bfloat16).cuda())
        outs.append(None)
    elements = wl.elements
    stream = torch.cuda.current_stream()

    def step():
        for i, W in enumerate(dev_w):
            outs[i] = api.soar_mx_quantize(W, 2, n_beta, 1, outs[i], stream)

    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    res = [o.read_result() for o in outs]
    byts = elements * (2.0 + 0.5 + 1.0 / 32)                    # read W; write codes and one scale byte per 32
    gbs = byts / (ms * 1e-3) / 1e9
    cpu = None
    if not args.no_cpu:
        from oracle import soar_ref as R
        spec = wl.tensors[0]
        rows = max(1, min(spec.rows, args.cpu_rows) // WL._chunk_rows(spec.cols)) * WL._chunk_rows(spec.cols)
        w = wl.generate(0, 0, rows)
        t0 = time.perf_counter()
        R.mx_quantize(w, n_beta=n_beta)
        dt = time.perf_counter() - t0
        cpu = dict(value=2.0 * w.size / dt / 1e9, unit="GB/s", cores=R.num_threads(), kind="oracle",
                   sample=f"first {rows} rows x {spec.cols} cols of tensor '{spec.name}', {dt:.1f} s")
    print(json.dumps(dict(
        metric="soar_quantize_bf16_input_throughput", value=2.0 * elements / (ms * 1e-3) / 1e9, unit="GB/s", n_gpus=1,
        steps=args.steps, warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="f32", data="synthetic",
        config=dict(workload=wl.name, format="mxfp4", search=("2 x 101 pairs" if n_beta else "plain rule"),
                    tensors=len(wl.tensors), elements=elements,
                    l2="inputs (%.2f GB per step) exceed the 126 MB L2" % (2 * elements / 1e9)),
        elements_per_s=elements / (ms * 1e-3),
        roofline=dict(bound="hbm", kernel="mx_kernel", achieved=gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                      frac=gbs / peaks["hbm_gbs"], traffic=None, peak_source=peaks["source"]),
        rel_error=[r.sse / r.sumsq for r in res], cpu_baseline=cpu, e2e=None,
        gpu_launches=2 * len(wl.tensors) * args.steps, clocks=clocks)), flush=True)


def run_row_sharded(args):
    """One tensor (the workload's largest) split by rows over the ranks: strong scaling.  Each rank runs the
    stages on its rows and the ranks all-reduce the workspace-header fields between stages."""
    import torch
    import torch.distributed as dist

    from paper_2605_12245_b200 import api
    from paper_2605_12245_b200 import row_sharded as RS
    from paper_2605_12245_b200 import sharding as SH

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    api.lib()
    peaks = load_peaks()
    wl = pick_workload(args.workload)
    ti = max(range(len(wl.tensors)), key=lambda i: wl.tensors[i].rows * wl.tensors[i].cols)
    spec = wl.tensors[ti]
    cr = WL._chunk_rows(spec.cols)                       # parts start on the generator's chunk boundaries
    per = ((spec.rows + world - 1) // world + cr - 1) // cr * cr
    r0, r1 = min(spec.rows, rank * per), min(spec.rows, (rank + 1) * per)
    cfg = preset_cfg(api, args.preset, args)
    W = torch.from_numpy(wl.generate(ti, r0, r1).view(np.int16)).view(torch.bfloat16).cuda()
    out = api.alloc_buffers(r1 - r0, spec.cols, cfg)
    stream = torch.cuda.current_stream()
    elements = spec.rows * spec.cols

    if world == 1:      # no process group: the combine step still runs, over one part
        def reduce(buf, how):
            return None
    else:
        reduce = RS.dist_all_reduce()
    header = out.workspace[:api.WORKSPACE_HEADER_BYTES]

    def step():
        for stage in RS.stages(cfg.max_iters):
            api.soar_quantize_stage([W], cfg, [out], out.workspace, stage)
            RS.combine_header(header, stage, cfg.max_iters, reduce)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    api.soar_trace_begin()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    trace = api.soar_trace_end()
    barrier()
    clocks = sampler.stop()
    ms = SH.max_over_ranks(e0.elapsed_time(e1) / args.steps, "cuda")
    res = out.read_result()
    dom = max(trace, key=lambda k: trace[k][1])
    n_launch, tot_ms = trace[dom]
    local_elems = (r1 - r0) * spec.cols
    byts = local_elems * sum(kernel_bytes_per_elem(dom, cfg, t) for t in range(res.iters_run if dom == "iterate_kernel" else 1)) * args.steps
    achieved = byts / (tot_ms * 1e-3) / 1e9
    if rank == 0:
        line = dict(
            metric="soar_quantize_bf16_input_throughput", value=2.0 * elements / (ms * 1e-3) / 1e9, unit="GB/s",
            n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=ms, higher_is_better=True,
            scaling="strong", vs_baseline=None, dtype="f32", data="synthetic",
            config=dict(workload=wl.name, tensor=spec.name, rows=spec.rows, cols=spec.cols, preset=args.preset,
                        max_iters=cfg.max_iters, n_beta=cfg.n_beta, n_dq=cfg.n_dq, early_stop_rel=cfg.early_stop_rel,
                        iters_run=res.iters_run, elements=elements,
                        l2="inputs (%.2f GB per rank) exceed the 126 MB L2" % (2 * (r1 - r0) * spec.cols / 1e9),
                        parallelism=f"{world} rank(s), rows split evenly, two small all-reduces per stage"),
            elements_per_s=elements / (ms * 1e-3),
            roofline=dict(bound="hbm", kernel=dom, achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                          frac=achieved / peaks["hbm_gbs"], traffic=None, launches=n_launch,
                          kernel_ms_per_step=tot_ms / args.steps,
                          peak_source=peaks["source"] + " (rank 0's kernels and rows)"),
            kernels={k: dict(launches=v[0], ms_per_step=v[1] / args.steps) for k, v in trace.items()},
            cpu_baseline=None, e2e=None, gpu_launches=sum(v[0] for v in trace.values()), clocks=clocks)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def launcher_command(n_ranks: int, argv, port: int):
    """The command that starts ``n_ranks`` ranks of this script on one node, one per GPU."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def self_launch(args, argv) -> int:
    """``bench.py --gpus N`` started as a plain process: start the N ranks here and pass their output on."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return subprocess.call(launcher_command(args.gpus, argv, port))


def run_dry(args):
    """The multi-rank plumbing alone, on CPU ranks over gloo (no GPU, no quantizer): rendezvous, barrier and
    the maximum over ranks that every timed number goes through.  Rank 0 prints the rank count."""
    import torch.distributed as dist

    from paper_2605_12245_b200 import sharding as SH
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms = SH.max_over_ranks(1.0 + rank, "cpu")
    units = SH.sum_over_ranks(1.0, "cpu")
    if rank == 0:
        print(json.dumps(dict(dry_run=True, n_gpus=world, ranks_seen=int(units), ms_per_step=ms)), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config4")
    ap.add_argument("--preset", default="paper", choices=["paper", "single_pass", "coupled_pair"])
    ap.add_argument("--cpu-rows", type=int, default=4096, help="rows of tensor 0 the CPU baseline quantizes")
    ap.add_argument("--ref-rows", type=int, default=1024, help="rows per step of the reference arm")
    ap.add_argument("--pairs", type=int, default=0, help="candidate pairs per block (overrides the preset's grid)")
    ap.add_argument("--iters", type=int, default=None, help="iterations T, early stop off (overrides the preset)")
    ap.add_argument("--sweep", default="", help="comma-separated candidate-pair counts to time, one iteration each")
    ap.add_argument("--objective", default="plain", choices=["plain", "weighted"],
                    help="weighted: the column-weighted objective through soar_quantize_weighted")
    ap.add_argument("--format", default="nvfp4", choices=["nvfp4", "mxfp4"],
                    help="mxfp4: the MXFP4 entry point (preset single_pass = the format's plain rule)")
    ap.add_argument("--row-sharded", action="store_true",
                    help="split the workload's largest tensor by rows over the ranks (strong scaling)")
    ap.add_argument("--sweep-dq", default="", help="comma-separated counts of E4M3 codes per block to time with beta = 1")
    ap.add_argument("--no-batch", action="store_true", help="one soar_quantize call per tensor instead of soar_quantize_batch")
    ap.add_argument("--graph", action="store_true", help="replay each step from a CUDA graph (no per-kernel trace)")
    ap.add_argument("--deterministic", action="store_true", help="SOAR_FLAG_DETERMINISTIC: sums added in a fixed order")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-single-pass", action="store_true")
    ap.add_argument("--dry-run", action="store_true",
                    help="CPU ranks over gloo: only the launch and the rank bookkeeping (for tests)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        raise SystemExit(self_launch(args, sys.argv[1:]))      # one rank per GPU, started from here
    if args.dry_run:
        run_dry(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.format == "mxfp4":
        run_mxfp4(args)
    elif args.row_sharded:
        run_row_sharded(args)
    elif args.objective == "weighted":
        run_weighted(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
