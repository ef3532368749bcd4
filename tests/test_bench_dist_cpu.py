"""The multi-process side of bench.py on CPU (gloo, world size 2): replicas with no collective
on the data path, max-over-ranks timing, whole-job value, and the reference arm's rank rule."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 10.0 + 5.0 * rank  # rank 1 is the slow one
    got = bench.max_over_ranks(ms)
    dist.barrier()
    value = bench.whole_job_value(128, 4, got, world)
    # per-block times: the element-wise max over ranks, and the record built from them
    blocks = bench.max_over_ranks_vec([10.0 + rank, 12.0 - rank, 11.0])
    rec = bench.timing_record(blocks, 4, {"sm_mhz": 1500.0})
    out[rank] = (got, value, bench.dist_env()[:2], blocks, rec)
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_gloo():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0
    # two replicas of 128 tokens x 4 steps over the slower rank's 15 ms
    assert abs(res[0][1] - 2 * 128 * 4 / 15e-3) < 1e-6 and res[0][1] == res[1][1]
    assert res[0][2] == (0, 2) and res[1][2] == (1, 2)
    assert res[0][3] == res[1][3] == [11.0, 12.0, 11.0]
    rec = res[0][4]
    assert rec["repeats"] == 3 and rec["ms_per_step_median"] == 11.0 / 4 and rec["ms_per_step_best"] == 11.0 / 4
    assert abs(rec["sm_cycles_per_step_median"] - 11.0 / 4 * 1e-3 * 1500e6) < 1e-3


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(10, 2, 1000.0, 1) == 20.0
    assert bench.max_over_ranks_vec([1.0, 2.5]) == [1.0, 2.5]


def test_reference_arm_non_zero_rank_exits_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
