"""The N > 1 path of the benchmark on CPU: two gloo ranks.

The backward path is data parallel over tokens with no exchange inside it, so bench.py --gpus N runs N replicas on
their own tokens and combines only timings: whole-job FLOPs over the slowest rank's time.  This test drives that
host-side logic (seeding per rank, max-over-ranks reduction, aggregate value) with world_size 2 on the gloo backend.
The last test starts `python bench.py --gpus 2` the way a user would (no torchrun, no WORLD_SIZE): the script must
launch the two ranks itself and report n_gpus = 2; a CPU stub of the step stands in for the GPU work.
"""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local = [3.0, 5.0][rank]                      # rank 1 is the slow one
        ms_e2e_local = [40.0, 30.0][rank]
        ms, ms_e2e = bench.max_over_ranks(ms_local, ms_e2e_local, world, torch.device("cpu"))
        value = bench.aggregate_value(flops_per_rank=6e12, world=world, ms=ms)
        out[rank] = (ms, ms_e2e, value, bench.rank_seed(0, rank))
    finally:
        dist.destroy_process_group()


def test_two_rank_aggregation_over_gloo():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        ms, ms_e2e, value, seed = res[rank]
        assert ms == 5.0 and ms_e2e == 40.0                   # max over ranks, on every rank
        assert value == pytest.approx(2 * 6e12 / 5e-3 / 1e12)  # all ranks' FLOPs over the slowest time
    assert res[0][3] != res[1][3]                              # ranks draw different tokens


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(1.5, None, 1, torch.device("cpu")) == (1.5, None)
    assert bench.aggregate_value(4e12, 1, 2.0) == pytest.approx(2000.0)


def test_bench_gpus_flag_starts_the_ranks_itself():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "2", "--warmup", "1", "--stub-cpu"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                     # rank 0 alone prints
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2
    assert rec["ms_per_step"] == 5.0                           # the slower rank's time
    assert rec["value"] == pytest.approx(2 * 6e12 / 5e-3 / 1e12)
    assert rec["seeds"][0] != rec["seeds"][1]
