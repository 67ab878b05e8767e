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
