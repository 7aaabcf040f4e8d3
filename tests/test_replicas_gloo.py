"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent replicas, reduced report."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from synth_inputs import get_config
    # every rank draws its own batch (weak scaling): different seeds, same law
    lens = bench.lengths_for(get_config("4b"), seed=3 + rank)
    maxima, sums = bench.reduce_over_ranks([10.0 + rank, 20.0 - rank], [100 * (rank + 1), 7, len(lens)],
                                           torch.device("cpu"), world)
    out[rank] = (maxima, sums, int(lens.sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_max_time_and_sum_tokens():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29611, out), nprocs=world, join=True)
    for rank in range(world):
        maxima, sums, _ = out[rank]
        assert maxima == [11.0, 20.0]              # max over ranks of each timing
        assert sums == [300.0, 14.0, 128.0]        # whole-job totals
    assert out[0][2] != out[1][2]                  # the replicas hold different batches


def test_single_process_reduce_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks([1.5], [2.0, 3.0], torch.device("cpu"), 1) == ([1.5], [2.0, 3.0])


def test_reference_arm_prints_one_line_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "1", "--gpus", "2"], capture_output=True, text=True, env=env, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher around it re-executes under torch.distributed.run with two ranks
    (gloo here: no GPU); the line counts both replicas."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], capture_output=True,
                       text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2 and lines[0]["sequences_all_ranks"] == 128
    # a rank count that contradicts the launcher is refused instead of silently measuring fewer GPUs
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "3", "--dry-run"], capture_output=True,
                       text=True, env=dict(env, RANK="0", WORLD_SIZE="1"), timeout=120)
    assert r.returncode != 0


def test_workload_recipes():
    sys.path.insert(0, ROOT)
    from synth_inputs import get_config, kv_lengths_lognormal, kv_lengths_uniform, make_page_tables
    l = kv_lengths_uniform(64, 1024, 8192, 3)
    assert l.min() >= 1024 and l.max() <= 8192 and len(l) == 64
    ln = kv_lengths_lognormal(4096, 4096, 0.7, 256, 32768, 3)
    assert 3500 < np.median(ln) < 4700 and ln.max() <= 32768 and ln.min() >= 256
    pt, n = make_page_tables(l + 100, 16, 7)
    used = pt[pt >= 0]
    assert len(np.unique(used)) == len(used) == n          # no page shared, pool fully used
    assert sorted(used.tolist()) == list(range(n))
    import bench
    cfg = get_config("4b")
    gb = bench.algorithmic_bytes_per_step(cfg, 3, 64 * 4608) / 1e9
    assert 57 < gb < 60                                     # 8.04 weights + 43.5 KV + draft + logits
