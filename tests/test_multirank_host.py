"""Host logic of the multi-GPU benchmark path (replicas only: no data-path collective exists), on two gloo ranks.

Each rank is an independent replica; what the ranks share is the timing protocol: a barrier, the maximum of the
per-rank times, and a whole-job value computed from it on rank 0.  The reference arm runs on rank 0 alone.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2508_12594_b200 import workloads
    w = workloads.CONFIGS["tiny"]
    wr = bench.rank_workload(w, rank)
    inp = workloads.make_inputs(wr)
    dist.barrier()
    ms = bench.max_over_ranks(10.0 * (rank + 1), dist, "cpu")          # rank 1 is the slower replica
    out.put((rank, wr.seed, float(inp.K.double().sum()), ms, bench.whole_job_value(w, world, ms)))
    dist.destroy_process_group()


def test_two_replicas_time_as_the_slowest_and_draw_different_batches():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, 29512, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, sum0, ms0, v0), (r1, seed1, sum1, ms1, v1) = res
    assert (r0, r1) == (0, 1) and seed1 == seed0 + 1000 and sum0 != sum1
    assert ms0 == ms1 == 20.0                                            # the maximum over ranks, on every rank
    assert v0 == v1 == 2 * 1024 / 20e-3                                  # both replicas' tokens over the slowest time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0


def test_gpus_flag_starts_its_own_replicas():
    """`bench.py --gpus 2` outside a launcher starts two ranks itself (here the reference arm, which needs no GPU):
    rank 0 prints the one line, the other rank exits quietly, and the line says two ranks."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
