"""The N > 1 path of bench.py on CPU: two gloo ranks.  The hot path shards by independent
microbatches with no data-path collective, so what there is to check is the host logic: every
rank draws its own microbatch, the reported time is the max over ranks and the token count the
sum, and the reference arm prints on rank 0 only."""

import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2512_23353_b200 import workloads as wl

    w = bench.rank_workload(wl.WORKLOADS["small_llm"], rank, world)
    off, A = wl.microbatch(w)
    elapsed, tokens = bench.reduce_over_ranks(10.0 + 5.0 * rank, float(off[-1]))
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"off": off.tolist(), "elapsed": elapsed, "tokens": tokens, "T": int(off[-1])}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_microbatch(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0["off"] != r1["off"]                       # independent microbatches
    assert r0["elapsed"] == r1["elapsed"] == 15.0       # max over ranks
    assert r0["tokens"] == r1["tokens"] == r0["T"] + r1["T"]


def test_single_process_reduce_is_identity():
    import bench
    assert bench.reduce_over_ranks(3.0, 7.0) == (3.0, 7.0)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_line_has_the_contract_keys():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--cpu-seqs", "2", "--cpu-len-div", "64", "--workload", "small_llm"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
