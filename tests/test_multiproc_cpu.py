"""The multi-rank side of bench.py on CPU (gloo, world size 2): ranks take disjoint sample ranges of the
seeded stream, the reported time is the slowest rank's, the throughput counts every rank's tokens, and the
reference arm only runs on rank 0.  No GPU."""
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
    sys.path.insert(0, ROOT)
    import bench
    from paper_2502_11494_b200 import workloads as W

    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = W.LLAVA15_B64.with_(B=2, d=64)
    rng = bench.rank_samples(rank, w.B)
    keys, _ = W.make_batch(w, device="cpu", samples=rng)
    ms = bench.max_over_ranks(10.0 * (rank + 1), torch.device("cpu"), True)     # rank 1 is the slow one
    dist.barrier()
    out[rank] = (list(rng), float(keys.float().abs().sum()), ms, bench.job_tokens_per_s(world, w.B, w.n_vis, 5, ms))
    dist.destroy_process_group()


def test_two_ranks_shard_samples_and_report_the_slowest_time():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
    (r0, s0, ms0, v0), (r1, s1, ms1, v1) = out[0], out[1]
    assert r0 == [0, 1] and r1 == [2, 3]                     # disjoint, contiguous sample ranges
    assert s0 != s1                                          # hence different data
    assert ms0 == ms1 == 20.0                                # max over ranks, same on both
    assert v0 == v1 == 2 * 2 * 576 * 5 / 20e-3               # whole-job tokens / slowest time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""      # other ranks exit 0 without work
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                        "llava15_b1", "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0
