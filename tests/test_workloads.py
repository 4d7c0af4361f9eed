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
