"""The path does not shard (batch 1, strictly sequential draft steps): N GPUs run N independent replicas.
What the N > 1 launch adds on the host is checked here with two gloo ranks on the CPU: per-rank seeds differ,
the job's step time is the slowest rank's, the throughput counts every rank's round, and the reference arm
prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]
    got = bench.slowest_rank(mine, world, "cpu")
    dist.barrier()
    out[rank] = (got, bench.replica_seed(rank), bench.rounds_per_second(world, got[0]))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_count_both_rounds():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29671, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == [15.0, 3.0, 7.0]
    assert res[0][1] != res[1][1]
    assert res[0][2] == 2 * 1e3 / 15.0


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--config", "t_bf16",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--config", "t_bf16",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["higher_is_better"] is False
