"""The multi-GPU plumbing (no data-path collective: shard the independent units, reduce only the
timing) exercised with two gloo ranks on CPU."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_20334_b200 import multi


def test_shard_units_partitions_every_unit_once():
    for n in (0, 1, 7, 1024, 1025):
        for w in (1, 2, 3, 8):
            ranges = [multi.shard_units(n, w, r) for r in range(w)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            for (a, b), (c, d) in zip(ranges, ranges[1:]):
                assert b == c and a <= b
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        multi.shard_units(10, 2, 2)


def test_whole_job_throughput_counts_all_ranks():
    assert multi.whole_job_tokens_per_s(131072, 4, 2.0) == pytest.approx(4 * 131072 / 2e-3)
    assert multi.whole_job_tokens_per_s([100, 300], 2, 1000.0) == pytest.approx(400.0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        begin, end = multi.shard_units(1025, world, rank)
        my_ms = 3.0 + rank  # rank 1 is the slow one
        slowest = multi.max_over_ranks(my_ms)
        counts = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(counts, torch.tensor([end - begin]))
        out[rank] = (slowest, [int(c) for c in counts])
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timing_and_cover_all_units():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 4.0
    assert sum(res[0][1]) == 1025 and res[0][1] == res[1][1]


def test_max_over_ranks_without_process_group_is_identity():
    assert multi.max_over_ranks(2.5) == 2.5


def test_bench_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` with no launcher around it must start two ranks itself and report
    n_gpus 2 with the slowest rank's time (stubbed step on CPU: gloo, no GPU work)."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items()
           if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--stub-step",
                          "--steps", "3", "--scaling", "strong"], capture_output=True, text=True,
                         env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1  # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["scaling"] == "strong"
    assert line["ms_per_step"] >= 3.9  # rank 1 sleeps 4 ms per step: the maximum over ranks
    assert line["layers_of_rank0"] == [0, 16]
    assert line["config"]["workload"].startswith("config 3")
