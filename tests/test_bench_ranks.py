"""The N > 1 path of bench.py on CPU: two gloo ranks, no data-path collective, the job's time is the
slowest rank's and the value is the aggregate over ranks; the reference arm runs on rank 0 only."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench

    # rank r took (10 + 5 r) ms in total and (4 + 2 r) ms in its sparse launches
    total, sparse = bench.max_over_ranks([10.0 + 5 * rank, 4.0 + 2 * rank], dist, torch.device("cpu"))
    value = bench.aggregate_tflops(1e12, 3, sparse, world)
    # heads of one layer split across the ranks: the job's flops are the sum of the shares
    job_flops = bench.sum_over_ranks(1e12 * (rank + 1), dist, torch.device("cpu"))
    out[rank] = (total, sparse, value, job_flops)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_aggregate_with_the_slowest_ranks_time():
    world = 2
    port = _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]  # every rank ends with the same aggregate
    total, sparse, value, job_flops = res[0]
    assert total == 15.0 and sparse == 6.0 and job_flops == 3e12
    # 2 ranks x 3 calls x 1 TFLOP in 6 ms
    assert abs(value - 2 * 3 * 1.0 / 6e-3) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks([1.5, 2.5], None, torch.device("cpu")) == [1.5, 2.5]
    assert abs(bench.aggregate_tflops(2e12, 5, 10.0, 1) - 1000.0) < 1e-9
    assert bench.sum_over_ranks(2.5, None, torch.device("cpu")) == 2.5


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
           "--steps", "1", "--warmup", "1", "--gpus", "2"]
    r1 = subprocess.run(cmd, env=dict(env, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["value"] > 0 and line["unit"] == "TFLOP/s" and line["vs_baseline"] is None
