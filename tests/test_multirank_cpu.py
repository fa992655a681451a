"""The N > 1 path of bench.py is 'replicas only': ranks share no data, only the barrier and the
reductions of time (max) and tokens (sum).  Covered here with two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, ms_e2e, tok = bench.reduce_over_ranks(dist, "cpu", 10.0 + rank, 20.0 - rank, 100.0 * (rank + 1))
    wl = bench.replica_workload(bench.synth.workload("c1"), rank)
    out[rank] = (ms, ms_e2e, tok, wl.seed)
    dist.barrier()
    dist.destroy_process_group()


def test_rank_reduction_and_replica_seeds_with_gloo():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29631, out), nprocs=world, join=True)
    for r in range(world):
        ms, ms_e2e, tok, seed = out[r]
        assert ms == 11.0 and ms_e2e == 20.0 and tok == 300.0      # max, max, sum over ranks
    assert out[0][3] != out[1][3]                                   # every replica draws its own batch


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["unit"] == "tokens/s"
