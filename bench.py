#!/usr/bin/env python
"""Benchmark of the FEPLB MoE-layer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

A step is one pass of the whole path (route_hist -> plan || dispatch + static FFN -> dynamic FFN
-> combine) over one seeded synthetic micro-batch.  Rank 0 prints ONE JSON line.  With N > 1
(torchrun) every rank runs its own micro-batches, there is no data-path collective, and the value
is all ranks' tokens over the slowest rank's device time (weak scaling).

``--impl reference`` times the CPU oracle (oracle/), as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_19654_b200 import workloads as W  # noqa: E402

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"
# DRAM bytes (read + write) of one k_grouped_gemm launch at the benchmarked workload, from the ncu
# capture summarised under profiles/; none (null in the line) where no capture exists.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {     # keyed by (workload, GEMM launches per forward)
    ("cfg2", 2): {"bytes": 380.3e6, "source": "profiles/k_grouped_gemm_cfg2.md: 760.6 MB over the 2 launches of one forward "
                                              "(capture of the merged two-CTA launches)"},
    ("cfg2", 4): {"bytes": 190.0e6, "source": "capture of the four-launch form: 760 MB over the 4 launches of one forward"},
}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm_gbs=j["hbm_gbs"], bf16_tflops=j["bf16_tflops"],
                    bf16_tflops_sustained=j.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(self.gpu)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def mark(self):
        """Index of the next sample: ``summary(a, b)`` then covers what was sampled between two marks."""
        time.sleep(0.06)                       # let the sample that covers "now" arrive
        return len(self.lines)

    def stop(self):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        return self.summary(0, None)

    def summary(self, a=0, b=None):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        sm, mx, reasons = [], [], set()
        for ln in self.lines[a:b]:
            f = [s.strip() for s in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------- oracle arm

def _oracle_step(O, w, x, ids, gates, weights, tokens):
    """The oracle's whole path on the micro-batch restricted to ``tokens``."""
    sub_ids, sub_x, sub_g = ids[tokens], x[tokens], gates[tokens]
    counts, load = O.route_hist(sub_ids, w.E, w.R)
    mask = O.select_dynamic(counts, w.E, w.R, w.dyn)
    plan = O.plan(counts, mask, w.R, tau=w.tau, max_num_dyn=w.max_num_dyn)
    s2r, r2t, _, S_pad = O.permute(sub_ids, w.E, 1)
    xp = O.gather_rows(sub_x, r2t)
    y = O.expert_ffn(xp, O.row_experts(sub_ids, s2r, S_pad), *weights)
    out = O.combine(y, s2r, sub_g)
    return out, plan


def _oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads") for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(w, steps, warmup, sample_tokens, weights=None):
    from oracle import feplb_oracle as O
    weights = weights if weights is not None else W.gen_weights(w)
    times = []
    for i in range(warmup + steps):
        x, ids, gates = W.gen_microbatch(w, i % w.n_microbatches)
        tokens = np.arange(min(sample_tokens, w.T))
        t0 = time.perf_counter()
        _oracle_step(O, w, x, ids, gates, weights, tokens)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    n_tok = min(sample_tokens, w.T)
    return n_tok * len(times) / sum(times), 1e3 * sum(times) / len(times), n_tok


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = min(w.T, args.ref_sample_tokens)
    val, ms, n_tok = time_oracle(w, args.steps, args.warmup, sample)
    cores = _oracle_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": _config_dict(w, args, extra={"sample_tokens_per_step": n_tok}),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {n_tok} tokens of each micro-batch, whole path (numpy fp64 oracle)"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _config_dict(w, args, extra=None):
    c = {"workload": w.name, "T": w.T, "d": w.d, "f": w.f, "E": w.E, "top_k": w.K, "virtual_ranks": w.R,
         "dyn": w.dyn, "max_num_dyn": w.max_num_dyn, "tau": w.tau, "micro_batches": w.n_microbatches,
         "routing": f"{w.routing}(alpha={w.alpha})", "parallelism": f"dp{args.gpus} (independent micro-batches per rank)",
         "cache": "inputs rotate over the micro-batches; weights (%.2f GiB) exceed the 126 MB L2"
                  % (3 * w.E * w.d * w.f * 2 / 2 ** 30)}
    if getattr(args, "split", False):
        c["plan"] = "split extension on (not in the paper)"
    if extra:
        c.update(extra)
    return c


# --------------------------------------------------------------------------------------------- sharding

def rank_microbatches(rank, n_mb):
    """Micro-batch seeds of one rank: every rank owns its own, disjoint, block (weak scaling)."""
    return [rank * n_mb + i for i in range(n_mb)]


def max_over_ranks(ms, world, device):
    """Slowest rank's time; an all-reduce(MAX) when there is more than one rank."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(world, steps, tokens_per_step, ms):
    """Tokens all ranks processed over the slowest rank's time."""
    return world * steps * tokens_per_step / (ms * 1e-3)


# --------------------------------------------------------------------------------------------- CUDA arm

def gemm_flops(w):
    """Algorithmic flops of the expert FFN per micro-batch: three GEMMs, 2*d*f each, per slot."""
    return 6.0 * w.d * w.f * w.S


def run_cuda(args, w):
    import torch
    import torch.distributed as dist
    from paper_2604_19654_b200 import build as B
    from paper_2604_19654_b200 import feplb as F

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torch.distributed.run")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.build()
    cfg = F.config_from_workload(w, phase2_copy=1 if args.phase2 else 0, split=1 if args.split else 0)
    ctx = F.Context(cfg)
    ctx.set_gemm_form({"auto": F.FORM_AUTO, "single": F.FORM_SINGLE, "pair": F.FORM_PAIR, "weight_m": F.FORM_WEIGHT_M}[args.form])
    ctx.set_launch_merging(args.merge)
    buf = F.Buffers(cfg)

    weights = W.gen_weights(w)
    d_w1, d_w3, d_w2 = (F.bf16_tensor(a) for a in weights)
    n_mb = w.n_microbatches
    host = [W.gen_microbatch(w, mb) for mb in rank_microbatches(rank, n_mb)]
    dev = [(F.bf16_tensor(x), torch.from_numpy(i).cuda(), torch.from_numpy(g).cuda()) for x, i, g in host]
    stream = torch.cuda.current_stream()

    def step(i):
        x, ids, g = dev[i % n_mb]
        ctx.moe_forward(x, ids, g, d_w1, d_w3, d_w2, buf, want_plan=False, stream=stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ---------------------------------------------------------------
    for i in range(max(args.warmup, 3)):
        step(i)
    ctx.check_status()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()

    def timed(n):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        for i in range(n):
            step(i)
        ev1.record(stream)
        barrier()
        return max_over_ranks(ev0.elapsed_time(ev1), world, "cuda")

    def timed_blocks(min_total_ms):
        """Blocks of exactly K steps, each bracketed by barrier + synchronize and timed by CUDA events
        on the launching stream (slowest rank), repeated until the timed region is long enough for
        the clock samples to mean something; the median block is reported."""
        blocks = []
        while len(blocks) < args.max_repeats and (not blocks or sum(blocks) < min_total_ms):
            blocks.append(timed(args.steps))
        return blocks

    # (1) the headline: K steps between two events, nothing else on the stream
    m0 = sampler.mark() if rank == 0 else 0
    launches0 = ctx.launch_count()
    blocks = timed_blocks(args.min_timed_ms)
    launches = (ctx.launch_count() - launches0) // len(blocks)
    m1 = sampler.mark() if rank == 0 else 0
    ctx.check_status()
    ms_total = float(np.median(blocks))
    args.repeats, args.block_ms_min, args.block_ms_max = len(blocks), float(min(blocks)), float(max(blocks))
    # (2) the same blocks again with the library's per-stage events on (they end each stage's
    # chain of programmatic launches, so this pass is slower): stage times and the kernel roofline
    ctx.set_timeline(True)
    ctx.timeline_totals(reset=True)
    blocks2 = timed_blocks(args.min_timed_ms)
    totals, n_fw = ctx.timeline_totals(reset=True)
    ctx.set_timeline(False)
    m2 = sampler.mark() if rank == 0 else 0
    ctx.check_status()
    clocks = sampler.summary(m0, m1) if rank == 0 else None
    args.clocks_stage_pass = sampler.summary(m1, m2) if rank == 0 else None
    args.ms_instrumented = float(np.median(blocks2)) / args.steps
    value = whole_job_throughput(world, args.steps, w.T, ms_total)
    # (3) dispatch and combine alone over rotating buffer sets larger than the L2 (cold figures)
    args.cold = measure_cold_io(F, ctx, cfg, w, dev, stream) if rank == 0 and not args.quick else None
    if rank == 0:
        sampler.stop()

    # ---- end to end through the host-buffer entry point -----------------------------------------
    e2e_value, h2d, d2h = None, w.T * w.d * 2 + 2 * w.T * w.K * 4, w.T * w.d * 2
    if not args.quick:
        e2e_value = _time_e2e(args, w, ctx, buf, host, d_w1, d_w3, d_w2, stream, barrier, world, n_mb)

    # ---- stragglers: token loads from the plan; GEMM time of every virtual rank run alone ---------
    strag = None
    if rank == 0 and not args.no_straggler and not args.quick:
        strag = measure_stragglers(F, ctx, w, cfg, buf, dev, d_w1, d_w3, d_w2, stream, n_mb)
    args.backward_result = None
    if rank == 0 and args.backward:
        args.backward_result = measure_backward(F, w, dev, d_w1, d_w3, d_w2, stream, n_mb, min(args.steps, 100), args.bwd_pair)
    _report(args, w, ctx, rank, world, value, ms_total, launches, clocks, totals, n_fw, e2e_value, h2d, d2h, strag, weights, n_mb)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def measure_cold_io(F, ctx, cfg, w, dev, stream, reps=24):
    """feplb_dispatch and feplb_combine timed alone, each call on the next of several buffer sets
    whose combined footprint exceeds the 126 MB L2, so that neither the rows read nor the rows
    written are still cached from the previous call.  Median of CUDA-event times per call."""
    import torch
    per_set = 2.0 * (w.T * w.d + 2 * w.S * w.d)                  # x, x_perm, y_perm of one set
    n_sets = int(min(8, max(3, np.ceil(3 * 126e6 / per_set) + 1)))
    sets = [F.Buffers(cfg) for _ in range(n_sets)]
    n_mb = len(dev)
    for i, b in enumerate(sets):                                  # fill every set once (valid indices, y_perm defined)
        x, ids, g = dev[i % n_mb]
        ctx.route_hist(ids, b.counts, b.rank_load, stream=stream)
        ctx.dispatch(x, ids, b.counts, b.x_perm, b.slot_to_row, b.row_to_token, stream=stream)
        b.y_perm.copy_(b.x_perm)
    torch.cuda.synchronize()
    ctx.check_status()
    t_disp, t_comb = [], []
    for r in range(reps):
        b = sets[r % n_sets]
        x, ids, g = dev[(r % n_sets) % n_mb]
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        ctx.dispatch(x, ids, b.counts, b.x_perm, b.slot_to_row, b.row_to_token, stream=stream)
        e1.record(stream)
        ctx.combine(b.y_perm, b.slot_to_row, g, b.out, stream=stream)
        e2.record(stream)
        torch.cuda.synchronize()
        if r >= n_sets:                                           # the first round warms instruction caches only
            t_disp.append(e0.elapsed_time(e1))
            t_comb.append(e1.elapsed_time(e2))
    ctx.check_status()
    io_bytes = 2.0 * (w.T * w.d + w.S * w.d) + 12.0 * w.S
    del sets
    torch.cuda.empty_cache()
    return {"buffer_sets": n_sets, "footprint_mb": n_sets * per_set / 1e6,
            "dispatch_us": float(np.median(t_disp)) * 1e3, "combine_us": float(np.median(t_comb)) * 1e3,
            "dispatch_gbs_cold": io_bytes / (float(np.median(t_disp)) * 1e-3) / 1e9,
            "combine_gbs_cold": io_bytes / (float(np.median(t_comb)) * 1e-3) / 1e9,
            "note": "stand-alone feplb_dispatch (histogram + ranks, scan, gather) and feplb_combine, one call per "
                    "buffer set in rotation; the in-pipeline (warm) figures are roofline.dispatch_gbs / combine_gbs"}


def pick_bf16_peak(peaks, clocks):
    """The bf16 denominator that matches the clock regime of the run it divides: the burst figure
    when the SM clock sat within 5 % of its maximum and no power cap was active, else the sustained one."""
    sus = peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]
    if clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
        burst = clocks["sm_mhz"] >= 0.95 * clocks["sm_max_mhz"] and "sw_power_cap" not in clocks.get("reasons", [])
        return (peaks["bf16_tflops"], "burst") if burst else (sus, "sustained")
    return sus, "sustained (no clock samples)"


def merged_timeline(st):
    """One forward on one time axis, [name, start_us, end_us], origin = the forward's first kernel.
    Device intervals come from CUDA events; the host marks of the planner thread are placed
    relative to the instant the counts left the device (the thread polls pinned memory, so it sees
    them within a PCIe write of the scan kernel's end)."""
    if not st or not st.get("dev_total_us"):
        return None
    counts_at = st["dev_hist_us"]
    h0 = st["host_counts_ready_us"]
    s0 = counts_at + st["dev_counts_to_static_start_us"]
    s1 = counts_at + st["dev_counts_to_static_end_us"]
    d1 = st["dev_total_us"] - st["dev_combine_us"]
    host = [["host: counts seen by planner", counts_at, counts_at],
            ["host: greedy plan", counts_at + st["host_plan_done_us"] - h0 - st["plan_us"], counts_at + st["host_plan_done_us"] - h0],
            ["host: dynamic table published / upload enqueued", counts_at + st["host_upload_enqueued_us"] - h0,
             counts_at + st["host_upload_enqueued_us"] - h0]]
    if st.get("ffn_launches", 4) < 3:
        # weights-on-M form: one launch per pass; the marks inside the launches come from the GPU's timer
        p1e = s0 + st["dev_ffn_pass1_us"]
        tl = [["hist+scan (counts to host)", 0.0, counts_at],
              ["rank+gather (dispatch)", counts_at, counts_at + st["dev_dispatch_us"]],
              ["FFN pass 1: static groups (until the first CTA runs out of them)", s0, s1]] + host + [
              ["FFN pass 1: remaining static and dynamic groups", s1, p1e],
              ["FFN pass 2: static, then dynamic groups", d1 - st["dev_ffn_pass2_us"], d1],
              ["longest device-side wait for the dynamic table", s1, s1 + st["dev_plan_wait_us"]],
              ["combine", d1, st["dev_total_us"]]]
        return [[n, round(a, 2), round(b, 2)] for n, a, b in tl]
    tl = [["hist+scan (counts to host)", 0.0, counts_at],
          ["rank+gather (dispatch)", counts_at, counts_at + st["dev_dispatch_us"]],
          ["static FFN (pass 1 + pass 2)", s0, s1]] + host + [
          ["dynamic FFN (pass 1 + pass 2)", d1 - st["dev_dynamic_ffn_us"], d1],
          ["combine", d1, st["dev_total_us"]]]
    if st.get("phase2_copy_bytes"):
        tl.insert(6, ["phase-2 weight copies", counts_at + st["host_upload_enqueued_us"] - h0,
                      counts_at + st["dev_counts_to_copies_done_us"]])
    return [[n, round(a, 2), round(b, 2)] for n, a, b in tl]


def run_sweep(args):
    """The scaling sweep (not the default bench line): cfg3's layer at T x R points, one JSON line
    per point with tokens/s, GEMM TFLOP/s and fraction of peak, and the straggler ratios before and
    after rebalancing.  Weights are generated once; two micro-batches per point."""
    import torch
    from paper_2604_19654_b200 import build as B
    from paper_2604_19654_b200 import feplb as F
    torch.cuda.set_device(0)
    B.build()
    points = W.sweep_points()
    if args.sweep != "all":
        keep = set(args.sweep.split(","))
        points = [p for p in points if p.name in keep]
    weights = W.gen_weights(points[0])
    d_w1, d_w3, d_w2 = (F.bf16_tensor(a) for a in weights)
    peaks = _peaks()
    stream = torch.cuda.current_stream()
    for w in points:
        cfg = F.config_from_workload(w)
        ctx, buf = F.Context(cfg), F.Buffers(cfg)
        n_mb = 2
        host = [W.gen_microbatch(w, mb) for mb in range(n_mb)]
        dev = [(F.bf16_tensor(x), torch.from_numpy(i).cuda(), torch.from_numpy(g).cuda()) for x, i, g in host]
        for i in range(3):
            ctx.moe_forward(*dev[i % n_mb], d_w1, d_w3, d_w2, buf, want_plan=False, stream=stream)
        ctx.check_status()
        ctx.set_timeline(True)
        ctx.timeline_totals(reset=True)
        steps = max(4, min(40, int(2.0e5 / w.T)))
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record(stream)
        for i in range(steps):
            ctx.moe_forward(*dev[i % n_mb], d_w1, d_w3, d_w2, buf, want_plan=False, stream=stream)
        ev1.record(stream)
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1) / steps
        totals, n_fw = ctx.timeline_totals(reset=True)
        ctx.set_timeline(False)
        ffn_us = (totals["dev_static_ffn_us"] + totals["dev_dynamic_ffn_us"]) / n_fw
        tflops = gemm_flops(w) / (ffn_us * 1e-6) / 1e12
        strag = measure_stragglers(F, ctx, w, cfg, buf, dev, d_w1, d_w3, d_w2, stream, n_mb, reps=2) if w.R > 1 else None
        io_bytes = 2.0 * (w.T * w.d + w.S * w.d) + 12.0 * w.S
        print(json.dumps({
            "sweep_point": w.name, "T": w.T, "R": w.R, "tokens_per_s": w.T / (ms * 1e-3), "ms_per_step": ms,
            "gemm_tflops": tflops, "gemm_frac_of_sustained_peak": tflops / peaks["bf16_tflops_sustained"],
            "gemm_frac_of_burst_peak": tflops / peaks["bf16_tflops"],
            "dispatch_gbs": io_bytes / (totals["dev_dispatch_us"] / n_fw * 1e-6) / 1e9,
            "combine_gbs": io_bytes / (totals["dev_combine_us"] / n_fw * 1e-6) / 1e9,
            "straggler": strag}), flush=True)
        ctx.close()
        del buf, dev
        torch.cuda.empty_cache()


def measure_backward(F, w, dev, d_w1, d_w3, d_w2, stream, n_mb, steps, bwd_pair=-1):
    """Forward + backward of the layer (weight gradients included, so expert segments are padded
    to 128 rows), timed per phase with CUDA events on the launching stream."""
    import torch
    cfg = F.config_from_workload(w, row_align=128)
    ctx, buf, bwd = F.Context(cfg), F.Buffers(cfg), F.BackwardBuffers(cfg)
    ctx.set_gemm_form(F.FORM_AUTO, bwd_pair)
    ctx.set_preact_buffer(bwd.ab)
    w1t = torch.empty(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda")
    w3t = torch.empty_like(w1t)
    w2t = torch.empty(w.E, w.f, w.d, dtype=torch.bfloat16, device="cuda")
    ctx.transpose_weights(d_w1, d_w3, d_w2, w1t, w3t, w2t, stream=stream)
    dw1 = torch.zeros(w.E, w.f, w.d, dtype=torch.float32, device="cuda")
    dw3 = torch.zeros_like(dw1)
    dw2 = torch.zeros(w.E, w.d, w.f, dtype=torch.float32, device="cuda")
    d_out = [torch.randn(w.T, w.d, device="cuda", dtype=torch.float32).mul_(0.02).to(torch.bfloat16) for _ in range(2)]

    def fwd(i):
        x, ids, g = dev[i % n_mb]
        ctx.moe_forward(x, ids, g, d_w1, d_w3, d_w2, buf, want_plan=False, stream=stream)

    def back(i):
        ctx.moe_backward(d_out[i & 1], dev[i % n_mb][2], w1t, w3t, w2t, buf, bwd, dw1, dw3, dw2, accumulate=True, stream=stream)

    for i in range(3):
        fwd(i)
        back(i)
    ctx.check_status()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    torch.cuda.synchronize()
    for i in range(steps):
        ev[i][0].record(stream)
        fwd(i)
        ev[i][1].record(stream)
        back(i)
        ev[i][2].record(stream)
    torch.cuda.synchronize()
    ctx.check_status()
    f_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    b_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    ctx.close()
    peaks = _peaks()
    bwd_tflops = 2.0 * gemm_flops(w) / (b_ms * 1e-3) / 1e12
    return {"fwd_ms": f_ms, "bwd_ms": b_ms, "bwd_over_fwd": b_ms / f_ms, "steps": steps,
            "bwd_layer_tflops": bwd_tflops, "bwd_frac_of_sustained_peak": bwd_tflops / peaks["bf16_tflops_sustained"],
            "note": "backward = combine bwd + dgrad GEMMs (fused SwiGLU derivative) + 3 weight-gradient "
                    "GEMMs (fp32 accumulate into dW) + dispatch bwd; TFLOP/s counts 12*d*f per slot over the whole "
                    "backward time; row_align = 128"}


def plan_sensitivity(w, dyn, policy=1, mask="reactive", split=0, n_mb=8):
    """Mean reduction of the token straggler (max - mean rows per rank, the paper's Section 3.1
    metric) and mean max/mean after the plan, over ``n_mb`` micro-batches.  Host code only."""
    from paper_2604_19654_b200 import feplb as F
    red, after = [], []
    for mb in range(n_mb):
        ids, _ = W.gen_routing(w, mb)
        counts = np.bincount(ids.ravel(), minlength=w.E).astype(np.int32)
        if mask == "reactive":                       # the dyn busiest experts of every rank
            m = F.select_dynamic(counts, w.E, w.R, dyn)
        else:                                        # a fixed set: the first dyn experts of every rank
            m = np.zeros(w.E, np.uint8)
            for r in range(w.R):
                m[r * w.L: r * w.L + dyn] = 1
        p = F.plan(F.config_from_workload(w, dyn=dyn, policy=policy, split=split), counts, m)
        b, a = p.load_before.astype(float), p.load_after.astype(float)
        sb, sa = b.max() - b.mean(), a.max() - a.mean()
        red.append(1.0 - sa / sb if sb > 0 else 0.0)
        after.append(a.max() / a.mean())
    return 100.0 * float(np.mean(red)), float(np.mean(after))


def run_sensitivity(args):
    """The paper's dyn sweep (Section 3.5, dyn = 2, 4, 8) plus policy / mask / split variants on
    cfg3's routing at EP degrees 2..16; prints a markdown table.  No GPU needed."""
    from paper_2604_19654_b200 import build as B
    B.build()
    base = W.get_workload("cfg3")
    print("| R | experts/rank | dyn=2 | dyn=4 | dyn=8 | dyn=4, LITERAL | dyn=4, fixed mask | dyn=4, split |")
    print("|---|---|---|---|---|---|---|---|")
    for R in (2, 4, 8, 16):
        w = base.with_(R=R)
        cells = ["-%.0f %% (%.2f)" % plan_sensitivity(w, min(dyn, w.L)) for dyn in (2, 4, 8)]
        cells.append("-%.0f %% (%.2f)" % plan_sensitivity(w, 4, policy=0))
        cells.append("-%.0f %% (%.2f)" % plan_sensitivity(w, 4, mask="fixed"))
        cells.append("-%.0f %% (%.2f)" % plan_sensitivity(w, 4, split=1))
        print(f"| {R} | {w.L} | " + " | ".join(cells) + " |")


def _time_e2e(args, w, ctx, buf, host, d_w1, d_w3, d_w2, stream, barrier, world, n_mb):
    import torch
    import torch.distributed as dist
    from paper_2604_19654_b200 import feplb as F
    pinned = []
    for x, i, g in host:
        pinned.append((torch.from_numpy(x.view(np.int16)).pin_memory(), torch.from_numpy(i).pin_memory(),
                       torch.from_numpy(g).pin_memory()))
    # staging slots: the copies of micro-batch i+1 overlap the kernels of micro-batch i, and the host
    # reuses a slot only several steps later, when its result copy has long finished
    ns = F.HOST_SLOTS
    out_host = [torch.empty(w.T, w.d, dtype=torch.int16).pin_memory() for _ in range(ns)]
    x_dev = [torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda") for _ in range(ns)]
    i_dev = [torch.empty(w.T, w.K, dtype=torch.int32, device="cuda") for _ in range(ns)]
    g_dev = [torch.empty(w.T, w.K, dtype=torch.float32, device="cuda") for _ in range(ns)]
    o_dev = [torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda") for _ in range(ns)]

    def stage(i):
        s = i % ns
        xh, ih, gh = pinned[i % n_mb]
        ctx.host_stage_inputs(s, xh, ih, gh, x_dev[s], i_dev[s], g_dev[s])

    def step_host(i, last):
        s = i % ns
        xh, ih, gh = pinned[i % n_mb]
        if not last:
            stage(i + 1)                     # the next micro-batch's input copies run under this forward
        ctx.host_wait(s)                     # the slot's previous result has reached its host buffer
        ctx.moe_forward_host_async(s, xh, ih, gh, x_dev[s], i_dev[s], g_dev[s], d_w1, d_w3, d_w2, buf,
                                   o_dev[s], out_host[s], stream=stream)

    stage(0)
    for i in range(2 * ns):
        step_host(i, i == 2 * ns - 1)
    for s in range(ns):
        ctx.host_wait(s)
    barrier()
    t0 = time.perf_counter()
    stage(0)                                 # every timed step's input copies start inside the timed region
    for i in range(args.steps):
        step_host(i, i == args.steps - 1)
    for s in range(ns):
        ctx.host_wait(s)                     # every result is in host memory
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    barrier()
    return whole_job_throughput(world, args.steps, w.T, max_over_ranks(e2e_ms, world, "cuda"))


def time_oracle_single_thread(w, sample_tokens, weights):
    """The oracle with its BLAS limited to one thread (the plain loops are single-threaded anyway)."""
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        return None
    with threadpool_limits(limits=1):
        val, _, n_tok = time_oracle(w, 1, 0, sample_tokens, weights)
    return {"value": val, "sample_tokens": n_tok}


def _report(args, w, ctx, rank, world, value, ms_total, launches, clocks, totals, n_fw, e2e_value, h2d, d2h, strag, weights, n_mb):
    if rank == 0:
        peaks = _peaks()
        ffn_us = totals["dev_static_ffn_us"] + totals["dev_dynamic_ffn_us"]
        per_fw = int(round(totals.get("ffn_launches", 0) / n_fw)) if n_fw and totals.get("ffn_launches") else 4
        gemm_launches = per_fw * n_fw
        flops_launch = gemm_flops(w) / per_fw
        achieved = (flops_launch / (ffn_us * 1e-6 / gemm_launches)) / 1e12 if ffn_us > 0 else None
        # the denominator follows the clock regime of the pass the kernel times were taken in
        clk2 = getattr(args, "clocks_stage_pass", None)
        peak, regime = pick_bf16_peak(peaks, clk2)
        sus = peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]
        io_bytes = 2.0 * (w.T * w.d + w.S * w.d) + 12.0 * w.S
        cold = getattr(args, "cold", None) or {}
        traffic = NCU_TRAFFIC_BYTES_PER_LAUNCH.get((w.name, per_fw)) if args.form in ("auto", "pair") else None
        roof = {"bound": "tensor", "kernel": ("k_grouped_gemm, static + dynamic groups per launch" if per_fw == 2 else "k_grouped_gemm") if args.form != "weight_m" else "k_ffn_wm",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak if achieved else None,
                "peak_source": f"{peaks['source']} ({regime}: chosen from the SM clock and power-cap state sampled during this pass)",
                "clocks": clk2,
                "frac_of_burst": achieved / peaks["bf16_tflops"] if achieved else None,
                "frac_of_sustained": achieved / sus if achieved else None,
                "frac_of_nominal_2250": achieved / 2250.0 if achieved else None,
                "traffic": traffic["bytes"] if traffic else None, "traffic_source": traffic["source"] if traffic else None,
                "launches_timed": gemm_launches, "avg_launch_us": ffn_us / gemm_launches if gemm_launches else None,
                # the same launches by the GPU's own timer (first CTA's start to last CTA's end, taken inside
                # the kernels; merged launches only): without the launch gap the CUDA events include
                "avg_launch_us_kernel_timer": ((totals["dev_ffn_pass1_us"] + totals["dev_ffn_pass2_us"]) / gemm_launches
                                               if gemm_launches and totals.get("dev_ffn_pass1_us") else None),
                "dispatch_gbs": io_bytes / (totals["dev_dispatch_us"] / n_fw * 1e-6) / 1e9 if n_fw and totals["dev_dispatch_us"] else None,
                "combine_gbs": io_bytes / (totals["dev_combine_us"] / n_fw * 1e-6) / 1e9 if n_fw and totals["dev_combine_us"] else None,
                "dispatch_gbs_cold": cold.get("dispatch_gbs_cold"), "combine_gbs_cold": cold.get("combine_gbs_cold"),
                "hbm_peak_gbs": peaks["hbm_gbs"], "hbm_nominal_gbs": 7700.0}
        stage_us = {k: (v / n_fw if n_fw else None) for k, v in totals.items()}
        # the targets the benchmark spec sets for config 2, as this run meets them or not
        targets = None
        if achieved:
            hbm = peaks["hbm_gbs"]
            targets = {"gemm_ge_0.60_of_bf16_peak_of_this_clock_regime": bool(achieved / peak >= 0.60),
                       "gemm_ge_0.60_of_burst_bf16_peak": bool(achieved / peaks["bf16_tflops"] >= 0.60),
                       "dispatch_ge_0.60_of_hbm_peak": bool(roof["dispatch_gbs"] and roof["dispatch_gbs"] / hbm >= 0.60),
                       "combine_ge_0.60_of_hbm_peak": bool(roof["combine_gbs"] and roof["combine_gbs"] / hbm >= 0.60),
                       "dispatch_cold_ge_0.60_of_hbm_peak": bool(cold.get("dispatch_gbs_cold", 0) / hbm >= 0.60) if cold else None,
                       "combine_cold_ge_0.60_of_hbm_peak": bool(cold.get("combine_gbs_cold", 0) / hbm >= 0.60) if cold else None}
        # CPU oracle on the host cores: a bounded sample of the same workload
        cpu = None
        if not args.quick:
            cpu_val, cpu_ms, n_tok = time_oracle(w, 2, 1, min(w.T, 4096), weights)
            cpu = {"value": cpu_val, "unit": UNIT, "cores": _oracle_threads(), "kind": "oracle",
                   "sample": f"first {n_tok} tokens of 2 micro-batches, whole path (numpy fp64 oracle)",
                   "single_thread": time_oracle_single_thread(w, min(w.T, 512), weights)}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": _config_dict(w, args),
            "repeats": getattr(args, "repeats", 1),
            "block_ms": {"median": ms_total, "min": getattr(args, "block_ms_min", None), "max": getattr(args, "block_ms_max", None),
                         "note": "each block is exactly `steps` steps between barrier + synchronize; blocks repeat until "
                                 f"{args.min_timed_ms:.0f} ms are timed; value and ms_per_step are the median block's"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roof, "targets_cfg2": targets if w.name == "cfg2" else None,
            "cpu_baseline": cpu, "stage_us": stage_us, "timeline": merged_timeline(stage_us), "cold_io": cold or None,
            "straggler": strag,
            # stage_us, timeline and roofline come from a second pass of the same blocks with per-stage
            # events on; those events cost time, so that pass is slower than ms_per_step
            "ms_per_step_with_stage_events": getattr(args, "ms_instrumented", None),
        }
        if getattr(args, "backward_result", None):
            line["backward"] = args.backward_result
        if args.phase2:   # Phase-2 weight copies on the copy engines, overlapped with the static GEMM
            line["phase2"] = {
                "copy_bytes_per_step": stage_us["phase2_copy_bytes"],
                "copies_done_us_after_counts": stage_us["dev_counts_to_copies_done_us"],
                "static_gemm_end_us_after_counts": stage_us["dev_counts_to_static_end_us"],
                "copy_gbs": (stage_us["phase2_copy_bytes"] / max(stage_us["dev_counts_to_copies_done_us"], 1e-9) / 1e3
                             if stage_us["phase2_copy_bytes"] else None)}
        print(json.dumps(line), flush=True)


def measure_stragglers(F, ctx, w, cfg, buf, dev, d_w1, d_w3, d_w2, stream, n_mb, reps=3):
    """Token straggler from the plans and GEMM straggler from per-virtual-rank launches, before
    (every group on its home rank) and after rebalancing, averaged over the micro-batches."""
    import torch
    tok_b, tok_a, gem_b, gem_a, gem_bm, gem_am, tok_bm, tok_am = [], [], [], [], [], [], [], []
    L = w.E // w.R
    for i in range(min(n_mb, 4)):
        x, ids, g = dev[i]
        p = ctx.moe_forward(x, ids, g, d_w1, d_w3, d_w2, buf, want_plan=True, stream=stream)
        torch.cuda.synchronize()
        lb, la = p.load_before.astype(np.float64), p.load_after.astype(np.float64)
        tok_b.append(lb.max() / lb.mean())
        tok_a.append(la.max() / la.mean())
        tok_bm.append(lb.max() - lb.mean())
        tok_am.append(la.max() - la.mean())
        groups = p.groups
        per_rank = {"before": [], "after": []}
        for label, key in (("before", lambda gr: gr[0] // L), ("after", lambda gr: gr[3])):
            for r in range(w.R):
                sel = [gr for gr in groups if key(gr) == r]
                if not sel:
                    per_rank[label].append(0.0)
                    continue
                d_groups = torch.from_numpy(F.groups_to_numpy(sel)).cuda()
                ts = []
                for _ in range(reps):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    ctx.expert_ffn(buf.x_perm, d_w1, d_w3, d_w2, d_groups, len(sel), buf.h_scratch, buf.y_perm, stream=stream)
                    e1.record(stream)
                    torch.cuda.synchronize()
                    ts.append(e0.elapsed_time(e1))
                per_rank[label].append(float(np.median(ts)))
        b, a = np.array(per_rank["before"]), np.array(per_rank["after"])
        gem_b.append(b.max() / b.mean())
        gem_a.append(a.max() / a.mean())
        gem_bm.append(b.max() - b.mean())
        gem_am.append(a.max() - a.mean())
    def min_gain(before, after):      # smallest per-micro-batch reduction of max - mean (1 = all of it removed)
        return float(min(1.0 - a / b if b > 0 else 0.0 for b, a in zip(before, after)))
    return {"token_ratio_before": float(np.mean(tok_b)), "token_ratio_after": float(np.mean(tok_a)),
            "token_max_minus_mean_rows_before": float(np.mean(tok_bm)), "token_max_minus_mean_rows_after": float(np.mean(tok_am)),
            "token_min_gain_over_micro_batches": min_gain(tok_bm, tok_am),
            "gemm_min_gain_over_micro_batches": min_gain(gem_bm, gem_am),
            "gemm_ratio_before": float(np.mean(gem_b)), "gemm_ratio_after": float(np.mean(gem_a)),
            "gemm_max_minus_mean_ms_before": float(np.mean(gem_bm)), "gemm_max_minus_mean_ms_after": float(np.mean(gem_am)),
            "micro_batches": len(tok_b), "definition": "max over virtual ranks / mean; GEMM time = expert FFN of one rank's groups run alone"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--ref-sample-tokens", type=int, default=1024)
    ap.add_argument("--no-straggler", action="store_true")
    ap.add_argument("--split", action="store_true",
                    help="plan with the splitting extension (a hot expert is cut in multiples of the granule; not in the paper)")
    ap.add_argument("--backward", action="store_true", help="also time forward + backward (weight gradients included)")
    ap.add_argument("--phase2", action="store_true",
                    help="really copy migrated experts' weights into the receive buffer (copy engines) during the static GEMM")
    ap.add_argument("--min-timed-ms", type=float, default=1000.0,
                    help="repeat the block of --steps steps until this much device time has been timed (median block reported)")
    ap.add_argument("--max-repeats", type=int, default=400)
    ap.add_argument("--form", default="auto", choices=["auto", "single", "pair", "weight_m"],
                    help="grouped-GEMM form of the forward launches (feplb_set_gemm_form); auto is the library's choice")
    ap.add_argument("--merge", type=int, default=-1, choices=[-1, 0, 1],
                    help="feplb_set_launch_merging: 1 = one GEMM launch per pass over static then dynamic groups, 0 = four launches, -1 = library's choice")
    ap.add_argument("--bwd-pair", type=int, default=-1, choices=[-1, 0, 1, 2, 3],
                    help="with --backward: pair mask of the backward GEMMs (feplb_set_gemm_form), -1 = library's choice")
    ap.add_argument("--quick", action="store_true",
                    help="device-resident timing only: no end-to-end loop, stragglers or CPU baseline (for profiling)")
    ap.add_argument("--sweep", default=None,
                    help='"all" or comma-separated sweep-point names (cfg5-T8192-R8, ...): prints one line per point')
    ap.add_argument("--sensitivity", action="store_true",
                    help="host-only table: straggler reduction vs dyn, policy, mask, split (no GPU)")
    args = ap.parse_args()
    if args.quick and args.min_timed_ms == 1000.0:
        args.min_timed_ms = 0.0                     # profiling runs: one block per pass, few launches
    if args.sensitivity:
        run_sensitivity(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    w = W.get_workload(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_cuda(args, w)


if __name__ == "__main__":
    main()
