"""The seeded generators: determinism, shapes, and the load skew the workloads are meant to have."""
import numpy as np

from paper_2604_19654_b200 import workloads as W


def test_bf16_roundtrip_and_rne():
    a = np.array([1.0, -2.5, 0.02, 1.00390625, 1.01171875], np.float32)   # last two: ties
    b = W.f32_to_bf16_bits(a)
    back = W.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[1] == -2.5
    assert back[3] == 1.0            # 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0)
    assert back[4] == 1.015625       # 1 + 3*2^-8 is halfway -> even mantissa (1 + 2^-6)
    assert np.array_equal(W.f32_to_bf16_bits(back), b)
    assert np.array_equal(W.bf16_bits_to_f64(b), back.astype(np.float64))


def test_routing_is_seeded_and_well_formed():
    for name in ("cfg1", "cfg2", "cfg4"):
        w = W.get_workload(name)
        ids, gates = W.gen_routing(w, 1)
        ids2, gates2 = W.gen_routing(w, 1)
        assert np.array_equal(ids, ids2) and np.array_equal(gates, gates2)
        assert ids.shape == (w.T, w.K) and ids.dtype == np.int32 and gates.dtype == np.float32
        assert ids.min() >= 0 and ids.max() < w.E
        srt = np.sort(ids, axis=1)
        assert np.all(srt[:, 1:] != srt[:, :-1])               # K distinct experts per token
        assert np.allclose(gates.sum(1), 1.0, atol=1e-5)
        assert np.all(np.diff(gates, axis=1) <= 1e-7)          # slots ordered by descending logit
        other, _ = W.gen_routing(w, 2)
        assert not np.array_equal(ids, other)


def test_cfg4_hot_experts_take_35_percent():
    w = W.get_workload("cfg4")
    ids, _ = W.gen_routing(w, 0)
    counts = np.bincount(ids.ravel(), minlength=w.E)
    top3 = np.sort(np.argsort(-counts)[:3])
    assert len({int(e) // w.L for e in top3}) == 1             # all on one virtual rank
    assert abs(counts[top3].sum() / w.S - 0.35) < 0.002
    ids1, _ = W.gen_routing(w, 1)
    c1 = np.bincount(ids1.ravel(), minlength=w.E)
    assert np.array_equal(np.sort(np.argsort(-c1)[:3]), top3)  # hot set fixed across micro-batches


def test_skew_of_dirichlet_workloads():
    for name, lo, hi in (("cfg2", 1.1, 2.2), ("cfg3", 1.1, 2.6)):
        w = W.get_workload(name)
        ratios = []
        for mb in range(4):
            ids, _ = W.gen_routing(w, mb)
            load = np.bincount(ids.ravel() // w.L, minlength=w.R)
            ratios.append(load.max() / load.mean())
        assert lo < np.mean(ratios) < hi


def test_activations_and_weights():
    w = W.get_workload("cfg1")
    x = W.gen_activations(w, 0)
    w1, w3, w2 = W.gen_weights(w)
    assert x.shape == (w.T, w.d) and w1.shape == (w.E, w.f, w.d) and w2.shape == (w.E, w.d, w.f)
    assert abs(W.bf16_bits_to_f64(w1).std() - 0.02) < 2e-3
    assert not np.array_equal(w1, w3)
    assert np.array_equal(W.gen_weights(w)[2], w2)
    assert len(W.sweep_points()) == 20


# ----------------------------------------------------------------------------- bench.py host arithmetic

def test_bench_peak_selection_and_roofline_arithmetic():
    """The bf16 denominator follows the clock regime of the run; flops per micro-batch are 6 d f per slot; the
    timeline of a forward is ordered on one axis."""
    import bench
    peaks = {"bf16_tflops": 1634.5, "bf16_tflops_sustained": 1377.1}
    burst = {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": []}
    capped = {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"]}
    slow = {"sm_mhz": 1500.0, "sm_max_mhz": 1965.0, "reasons": []}
    assert bench.pick_bf16_peak(peaks, burst) == (1634.5, "burst")
    assert bench.pick_bf16_peak(peaks, capped)[0] == 1377.1
    assert bench.pick_bf16_peak(peaks, slow)[0] == 1377.1
    assert bench.pick_bf16_peak(peaks, None)[0] == 1377.1
    w = W.get_workload("cfg2")
    assert bench.gemm_flops(w) == 6.0 * 2048 * 768 * 4096 * 6
    assert bench.whole_job_throughput(2, 10, 4096, 5.0) == 2 * 10 * 4096 / 5e-3
    assert bench.rank_microbatches(1, 4) == [4, 5, 6, 7]
    st = {"dev_hist_us": 16.0, "host_counts_ready_us": 300.0, "host_plan_done_us": 302.5, "plan_us": 1.0,
          "host_upload_enqueued_us": 302.7, "dev_counts_to_static_start_us": 45.0, "dev_counts_to_static_end_us": 110.0,
          "dev_total_us": 360.0, "dev_combine_us": 28.0, "dev_dispatch_us": 30.0, "dev_static_ffn_us": 280.0,
          "dev_dynamic_ffn_us": 0.0, "ffn_launches": 2.0, "dev_ffn_pass1_us": 175.0, "dev_ffn_pass2_us": 96.0,
          "dev_plan_wait_us": 9.0}
    tl = bench.merged_timeline(st)
    assert tl and all(len(e) == 3 and e[1] <= e[2] for e in tl)
    names = [e[0] for e in tl]
    assert any("plan" in n for n in names) and any("combine" in n for n in names)
    plan = [e for e in tl if e[0] == "host: greedy plan"][0]
    static_end = 16.0 + 110.0
    assert plan[2] < static_end                       # the plan lands inside the static window of this example
    assert bench.merged_timeline({}) is None
