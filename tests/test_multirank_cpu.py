"""The N > 1 path of bench.py on CPU: two gloo ranks.  The layer has no exchange step between ranks (each
rank runs an independent batch), so what is multi-rank is only the bookkeeping: per-rank seeds, the
max-over-ranks of the device time, the whole-job throughput, and the reference arm running on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 5.0 + 2.0 * rank                       # rank 1 is the slow one
    ms = bench.slowest_rank_ms(ms_local)
    out[rank] = (ms, bench.whole_job_tokens_per_s(1000, world, ms), bench.rank_seed(1237, rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_rank_time():
    world, port = 2, 29500 + os.getpid() % 1000
    manager = mp.Manager()
    out = manager.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 7.0
    assert out[0][1] == out[1][1] == 2 * 1000 / 7e-3
    assert out[0][2] != out[1][2]


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.slowest_rank_ms(3.5) == 3.5
    assert bench.whole_job_tokens_per_s(32768, 1, 10.0) == 32768 / 10e-3


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                        "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                        "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
