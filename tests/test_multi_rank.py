"""Two gloo ranks on CPU: the host-side logic a multi-GPU run uses (tensor assignment, per-rank
workloads, max-over-ranks timing, whole-job throughput).  No data-path collective exists to
test: tensors are independent problems."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_12245_b200 import sharding as S
from paper_2605_12245_b200 import workloads as WL


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = S.assign_tensors(7, rank, world)
        t = S.max_over_ranks(1.0 + rank)                       # the slower rank defines the time
        thr = S.whole_job_throughput(100.0 * (rank + 1), 2.0 + rank)
        wl = S.rank_workload(WL.Workload("tiny", 5, "student_t4", (WL.TensorSpec("w", 4, 64),)), rank)
        bits = WL.generate(wl, 0, workers=1)
        dist.barrier()
        np.save(os.path.join(out_dir, f"r{rank}.npy"), bits)
        with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
            f.write(f"{mine}|{t}|{thr}")
    finally:
        dist.destroy_process_group()


def test_two_ranks_share_bookkeeping_only(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    seen = []
    for r in range(world):
        mine, t, thr = open(tmp_path / f"r{r}.txt").read().split("|")
        seen += eval(mine)
        assert float(t) == 2.0                                  # max(1, 2)
        assert float(thr) == pytest.approx((100.0 + 200.0) / 3.0)   # all units / slowest time
    assert sorted(seen) == list(range(7))                       # every tensor exactly once
    a, b = np.load(tmp_path / "r0.npy"), np.load(tmp_path / "r1.npy")
    assert a.shape == b.shape and not np.array_equal(a, b)      # same shapes, different draws


def test_single_process_helpers_need_no_process_group():
    assert S.assign_tensors(5, 1, 2) == [1, 3]
    assert S.max_over_ranks(3.5) == 3.5
    assert S.whole_job_throughput(10.0, 2.0) == 5.0
    with pytest.raises(ValueError):
        S.assign_tensors(5, 2, 2)


# ---- one tensor split by rows: the header plumbing between stages (no kernels run here)

def _header_worker(rank, world, port, out_dir):
    import ctypes as C

    from paper_2605_12245_b200 import api
    from paper_2605_12245_b200 import row_sharded as RS
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        T = 3
        h = api.SoarWorkspaceHeader()
        h.amax_bits = 0x3C00 + 7 * rank                 # the larger one must win
        h.error = rank                                  # an error on any part stops all
        h.zero_blocks = 10 + rank
        h.wide = 100 * (rank + 1)
        h.sumsq = 1.5 + rank
        for i in range(T + 1):
            h.num[i], h.den[i], h.gsum[i] = 1.0 + i + 10 * rank, 2.0 + i + 20 * rank, -(3.0 + i) - rank
        raw = bytearray(api.WORKSPACE_HEADER_BYTES)
        raw[:C.sizeof(h)] = bytes(h)
        header = torch.frombuffer(raw, dtype=torch.uint8)
        snaps = []
        for stage in RS.stages(T):
            RS.combine_header(header, stage, T, RS.dist_all_reduce())
            snaps.append(bytes(raw[:C.sizeof(h)]))
        np.save(os.path.join(out_dir, f"h{rank}.npy"), np.frombuffer(b"".join(snaps), dtype=np.uint8))
    finally:
        dist.destroy_process_group()


def test_row_sharded_header_fields_are_combined_stage_by_stage(tmp_path):
    import ctypes as C

    from paper_2605_12245_b200 import api
    from paper_2605_12245_b200 import row_sharded as RS
    world, port, T = 2, _free_port(), 3
    mp.spawn(_header_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    size = C.sizeof(api.SoarWorkspaceHeader)
    per_rank = [np.load(tmp_path / f"h{r}.npy").reshape(-1, size) for r in range(world)]
    stage_list = RS.stages(T)
    assert stage_list == [api.STAGE_AMAX, api.STAGE_INIT, 0, 1, 2, api.STAGE_FINALIZE]
    for r in range(world):
        snaps = [api.SoarWorkspaceHeader.from_buffer_copy(per_rank[r][i].tobytes()) for i in range(len(stage_list))]
        a = snaps[0]                                   # after the amax stage
        assert a.amax_bits == 0x3C07 and a.error == 1 and a.sumsq == 1.5 + 2.5
        assert a.num[0] == 1.0 + 10 * r and a.zero_blocks == 10 + r          # not yet combined
        b = snaps[1]                                   # after init: stage-0 sums and the zero-block count
        assert (b.num[0], b.den[0], b.gsum[0]) == (1.0 + 11.0, 2.0 + 22.0, -3.0 - 4.0)
        assert b.zero_blocks == 21 and b.sumsq == 4.0                        # sumsq is not added twice
        assert b.num[1] == 2.0 + 10 * r and b.wide == 100 * (r + 1)
        for t in range(T):                             # after iteration t: entries t+1
            c = snaps[2 + t]
            assert (c.num[t + 1], c.den[t + 1], c.gsum[t + 1]) == (2 * (2.0 + t) + 10, 2 * (3.0 + t) + 20, -2 * (4.0 + t) - 1)
            if t + 2 <= T:
                assert c.num[t + 2] == 3.0 + t + 10 * r                      # later entries untouched
        # the counter that grows in every stage is combined once, after the last iteration
        assert snaps[2].wide == snaps[3].wide == 100 * (r + 1) and snaps[4].wide == 300
        assert bytes(snaps[-1]) == bytes(snaps[-2])    # nothing is combined after the report stage


def test_row_sharded_schedule_combines_every_written_entry_exactly_once():
    from paper_2605_12245_b200 import api
    from paper_2605_12245_b200 import row_sharded as RS
    for T in (0, 1, 4):
        seen = []
        for stage in RS.stages(T):
            seen += [(n, i) for n, i, how in RS.fields_written(stage, T) if how == RS.SUM]
        want = [("sumsq", 0), ("zero_blocks", 0), ("wide", 0)] + [(f, i) for f in ("num", "den", "gsum") for i in range(T + 1)]
        assert sorted(seen) == sorted(want)                     # sums: once each, none missing
        assert RS.fields_written(api.STAGE_FINALIZE, T) == []
        # the counter that grows until the report is combined after the last stage before it
        last = T - 1 if T > 0 else api.STAGE_INIT
        assert ("wide", 0, RS.SUM) in RS.fields_written(last, T)
    with pytest.raises(ValueError):
        RS.fields_written(4, 4)
    # views address the published layout
    import ctypes as C
    raw = bytearray(api.WORKSPACE_HEADER_BYTES)
    header = torch.frombuffer(raw, dtype=torch.uint8)
    RS.header_view(header, "den", 3).fill_(2.5)
    RS.header_view(header, "amax_bits").fill_(0x3F80)
    h = api.SoarWorkspaceHeader.from_buffer_copy(bytes(raw[:C.sizeof(api.SoarWorkspaceHeader)]))
    assert h.den[3] == 2.5 and h.amax_bits == 0x3F80 and h.num[3] == 0.0


def test_bench_starts_its_own_ranks_when_given_a_rank_count():
    """``bench.py --gpus 2`` as a plain process starts two ranks itself; the dry run keeps them on CPU
    (gloo) and reports how many ranks met."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--dry-run"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["ranks_seen"] == 2 and line["ms_per_step"] == 2.0


def test_launcher_command_is_one_rank_per_gpu_on_the_loopback_address():
    import importlib.util
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    cmd = bench.launcher_command(4, ["--gpus", "4", "--steps", "2"], 29517)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29517"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"]
