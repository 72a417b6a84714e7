"""The multi-GPU path is N independent replicas (no data-path collective).  What the ranks do
together - agree on the slowest time and add up their tokens - is exercised here with two gloo
ranks on the CPU; the reference arm must print on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dev_ms, e2e_ms, toks = bench.aggregate_over_ranks(dist, world, 10.0 + rank, 20.0 - rank, 100 + rank, "cpu")
    plan = bench.replica_plan(rank, None)
    out.put((rank, dev_ms, e2e_ms, toks, plan["prompt_seed"]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_aggregate_max_time_and_sum_of_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, dev_ms, e2e_ms, toks, seed in res:
        assert dev_ms == 11.0 and e2e_ms == 20.0 and toks == 201.0
    assert res[0][4] != res[1][4]                              # each replica decodes its own prompt


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "3", "--gpus", "2"], capture_output=True, text=True, env=env,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "3", "--gpus", "2"], capture_output=True, text=True, env=env,
                       timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
