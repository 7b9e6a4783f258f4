"""Host logic of the multi-GPU benchmark path, on CPU with two gloo ranks.

The decoding path shards by series with no exchange step: every rank decodes its own batch.
What the ranks share is bookkeeping only -- distinct series per rank, the max-over-ranks time,
the whole-job throughput, and the rule that the CPU-reference arm runs on rank 0 alone."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from tsfm_inputs import make_series, workload
    wl = bench.rank_workload(workload("C0", batch=3, series_recipe="c1"), rank)
    s = make_series(wl)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")       # rank 1 is the slow one
    value = bench.whole_job_value(world, wl.batch, wl.n_patches, 4, ms)
    json.dump({"ms": ms, "value": value, "checksum": float(np.abs(s).sum()), "first": s[0, :4].tolist()},
              open(os.path.join(out_dir, f"r{rank}.json"), "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_decode_different_series_and_agree_on_the_job_time(tmp_path):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"r{i}.json")) for i in range(world)]
    assert r[0]["ms"] == r[1]["ms"] == 15.0                       # max over ranks, seen by both
    assert r[0]["value"] == r[1]["value"] == 2 * 3 * 4 * 4 / 15e-3    # all ranks' patches / slowest time
    assert r[0]["first"] != r[1]["first"]                          # each rank has its own series


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C0",
                          "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True,
                         timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env["RANK"] = "0"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C0",
                          "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True,
                         timeout=300)
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
