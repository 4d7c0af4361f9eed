"""World-size-2 run of the benchmark's multi-rank host logic on CPU (gloo): disjoint micro-batch
shards, no data-path collective, slowest-rank timing, whole-job throughput; and the reference
arm's rule that only rank 0 prints."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    import bench
    from oracle import feplb_oracle as O
    from paper_2604_19654_b200 import workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = W.get_workload("cfg1")
    mbs = bench.rank_microbatches(rank, 2)
    loads = []
    for mb in mbs:                                   # each rank plans its own micro-batches, independently
        ids, _ = W.gen_routing(w, mb)
        counts, load = O.route_hist(ids, w.E, w.R)
        p = O.plan(counts, O.select_dynamic(counts, w.E, w.R, w.dyn), w.R, w.tau, w.max_num_dyn)
        loads.append(p["load_after"].tolist())
    ms = 10.0 + 5.0 * rank                           # rank 1 is the slow one
    slowest = bench.max_over_ranks(ms, world, "cpu")
    gathered = [None] * world
    dist.all_gather_object(gathered, (mbs, loads))
    dist.barrier()
    q.put((rank, slowest, gathered))
    dist.destroy_process_group()


def test_two_ranks_shard_microbatches_and_time_by_the_slowest():
    import bench
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, slow0, g0), (r1, slow1, g1) = res
    assert slow0 == slow1 == 15.0                    # max over ranks, seen by every rank
    assert g0 == g1
    mbs0, mbs1 = g0[0][0], g0[1][0]
    assert set(mbs0).isdisjoint(mbs1) and len(mbs0) == len(mbs1) == 2
    assert g0[0][1] != g0[1][1]                      # different micro-batches, different plans
    assert bench.whole_job_throughput(2, 10, 256, 15.0) == 2 * 10 * 256 / 0.015


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "cfg1"], env=env, capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "cfg1"], env=env, capture_output=True, text=True)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "cfg1"


def test_dyn_sensitivity_is_monotone_and_reactive_mask_beats_fixed():
    """The dyn sweep of the paper's Section 3.5 on synthetic routing: more dynamic experts never
    hurt on average, and choosing the busiest experts beats a fixed set (host plan only)."""
    import bench
    from paper_2604_19654_b200 import workloads as W
    w = W.get_workload("cfg3")
    r2, _ = bench.plan_sensitivity(w, 2, n_mb=4)
    r4, a4 = bench.plan_sensitivity(w, 4, n_mb=4)
    r8, _ = bench.plan_sensitivity(w, 8, n_mb=4)
    assert 0 < r2 <= r4 <= r8 <= 100
    fixed, _ = bench.plan_sensitivity(w, 4, mask="fixed", n_mb=4)
    literal, _ = bench.plan_sensitivity(w, 4, policy=0, n_mb=4)
    assert fixed < r4 and literal <= r4 and a4 < 1.2
