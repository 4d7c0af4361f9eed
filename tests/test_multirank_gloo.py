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


# ----------------------------------------------------------------------------- expert parallelism over real ranks

def _ep_worker(rank, world, port, q):
    """One rank of a real expert-parallel group on CPU.  Control plane: the library's (all-gather of
    the counts + feplb_ep_schedule).  Data plane: replayed on numpy arrays through object
    collectives, with the oracle's FFN on the rows each rank executes."""
    from oracle import feplb_oracle as O
    from paper_2604_19654_b200 import ep, feplb as F, workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    R = world
    w = W.get_workload("cfg1").with_(name="ep", T=48 * R, E=4 * R, R=R, K=3, dyn=2, max_num_dyn=2, tau=1, alpha=1.4)
    x, ids, gates = W.gen_microbatch(w, 7)                       # the whole micro-batch, seeded: every rank draws the same
    w1, w3, w2 = W.gen_weights(w)
    T_loc, L = w.T // R, w.E // R
    t0 = rank * T_loc                                            # this rank's tokens: [t0, t0 + T_loc)
    my_ids, my_x, my_g = ids[t0:t0 + T_loc], x[t0:t0 + T_loc], gates[t0:t0 + T_loc]
    cfg = F.config_from_workload(w)
    # ---- control plane
    local_counts = np.bincount(my_ids.ravel(), minlength=w.E).astype(np.int32)
    cbs = ep.exchange_counts(local_counts)
    sch = ep.schedule(cfg, cbs, rank)
    plan = sch["plan"]
    # ---- Phase 1: every slot's row to the home of its expert, in (source rank, slot) order
    out_p1 = [[] for _ in range(R)]
    for s_loc in range(T_loc * w.K):
        e = int(my_ids.ravel()[s_loc])
        out_p1[e // L].append((e, rank, s_loc, my_x[s_loc // w.K]))
    assert [len(v) for v in out_p1] == sch["p1_send"].tolist()
    everything = [None] * R
    dist.all_gather_object(everything, out_p1)
    seg = {e: [] for e in range(rank * L, (rank + 1) * L)}      # expert -> rows in segment order
    for src in range(R):
        assert len(everything[src][rank]) == sch["p1_recv"][src]
        for (e, s, s_loc, row) in everything[src][rank]:
            seg[e].append((s, s_loc, row))
    # ---- Phase 2: migrated pieces (rows + the expert's weights) from the home to the receiving rank
    out_p2 = [[] for _ in range(R)]
    taken = {e: 0 for e in seg}
    for (e, src, dst, slot, rows, nbytes) in sch["copies"]:
        if src == rank:
            piece = seg[e][taken[e]:taken[e] + rows]
            taken[e] += rows
            out_p2[dst].append((e, slot, piece, (w1[e], w3[e], w2[e])))
    assert [sum(len(m[2]) for m in v) for v in out_p2] == sch["p2_send"].tolist()
    dist.all_gather_object(everything, out_p2)
    work = [(e, rows[taken[e]:], (w1[e], w3[e], w2[e])) for e, rows in seg.items()]      # home remainders, home weights
    slots_seen = []
    for src in range(R):
        got = everything[src][rank]
        assert sum(len(m[2]) for m in got) == sch["p2_recv"][src]
        for (e, slot, piece, wts) in got:
            assert nbytes == 3 * w.d * w.f * 2 and slot // cfg.max_num_dyn == rank
            slots_seen.append(slot)
            work.append((e, piece, wts))                        # weights as they arrived in the receive slot
    assert len(set(slots_seen)) == len(slots_seen)
    assert sum(len(rows) for _, rows, _ in work) == int(plan.load_after[rank])
    # ---- expert FFN on the rows this rank executes, then the combine: results straight back to the sources
    out_c = [[] for _ in range(R)]
    for (e, rows, (a1, a3, a2)) in work:
        if not rows:
            continue
        xb = np.stack([r[2] for r in rows])
        y = O.expert_ffn(xb, np.zeros(len(rows), np.int64), a1[None], a3[None], a2[None])
        for (s, s_loc, _), yr in zip(rows, y):
            out_c[s].append((s_loc, yr))
    assert [len(v) for v in out_c] == sch["comb_send"].tolist()
    dist.all_gather_object(everything, out_c)
    y_slots = np.zeros((T_loc * w.K, w.d))
    for src in range(R):
        assert len(everything[src][rank]) == sch["comb_recv"][src]
        for (s_loc, yr) in everything[src][rank]:
            y_slots[s_loc] = yr
    out = O.combine(y_slots, np.arange(T_loc * w.K).reshape(T_loc, w.K), my_g)
    ref = O.moe_layer(x, ids, gates, w1, w3, w2, w.E, tokens=np.arange(t0, t0 + T_loc))
    err = float(np.abs(out - ref).max() / np.abs(ref).max())
    summary = (plan.moves, plan.groups, plan.load_before.tolist(), plan.load_after.tolist(), sch["copies"])
    gathered = [None] * R
    dist.all_gather_object(gathered, (summary, sch["p1_send"].tolist(), sch["p1_recv"].tolist(), sch["p2_send"].tolist(),
                                      sch["p2_recv"].tolist(), sch["comb_send"].tolist(), sch["comb_recv"].tolist(), err))
    dist.barrier()
    q.put((rank, gathered))
    dist.destroy_process_group()


def _run_ep(world):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_ep_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return res[0][1]


def _check_ep(world):
    g = _run_ep(world)
    summaries = [r[0] for r in g]
    assert all(s == summaries[0] for s in summaries)            # every rank derived the same plan and copy list
    moves, _, before, after, copies = summaries[0]
    assert len(moves) >= 1 and max(after) < max(before)
    for name, (snd, rcv) in {"phase 1": (1, 2), "phase 2": (3, 4), "combine": (5, 6)}.items():
        send = np.array([r[snd] for r in g])                    # send[s][r]
        recv = np.array([r[rcv] for r in g])                    # recv[r][s]
        assert np.array_equal(send, recv.T), name               # what s sends to r is what r expects from s
    assert np.array([r[3] for r in g]).sum() == sum(m[3] for m in moves)
    assert max(r[7] for r in g) < 1e-12                         # the replayed layer equals the oracle's


def test_expert_parallel_protocol_world_2():
    _check_ep(2)


def test_expert_parallel_protocol_world_4():
    _check_ep(4)
