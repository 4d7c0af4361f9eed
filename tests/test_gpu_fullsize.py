"""Full-size GPU parity: the GLM-5-like layer (T=16384, d=6144, f=2048, E=128, top-8, R=8) in the
launch configuration the benchmark times, and two points of the scaling sweep.  Integer stages
are compared in full; the fp64 oracle cannot run 9.9 TFLOP in a test, so floating point is checked
on sampled outputs it can compute one by one: rows of y_perm around tile and group boundaries of
seeded experts, whole-layer outputs of seeded tokens, and the combine on the GPU's own y_perm."""
import numpy as np
import pytest

from oracle import feplb_oracle as O
from paper_2604_19654_b200 import build as B
from paper_2604_19654_b200 import feplb as F
from paper_2604_19654_b200 import workloads as W

from gpu_utils import DeviceCase, assert_close, oracle_mask

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cfg3_weights():
    B.build()
    return W.gen_weights(W.get_workload("cfg3"))


def _sample_rows(counts, pad_off, experts, rng):
    """Rows to check per expert: first, last, both sides of every 128-row tile boundary (up to 6
    boundaries), and a few random ones."""
    rows = []
    for e in experts:
        c, p = int(counts[e]), int(pad_off[e])
        if c == 0:
            continue
        local = {0, c - 1}
        for b in range(128, c, 128)[:6]:
            local.update((b - 1, b))
        local.update(rng.integers(0, c, size=4).tolist())
        rows += [p + r for r in sorted(local) if 0 <= r < c]
    return np.array(rows, np.int64)


def _check_full_size(case, n_experts=10, n_tokens=12):
    w = case.w
    p = case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    case.ctx.check_status()
    # ---- integers, in full
    counts, load = O.route_hist(case.ids, w.E, w.R)
    mask = oracle_mask(counts, w)
    op = O.plan(counts, mask, w.R, tau=w.tau, max_num_dyn=w.max_num_dyn)
    assert np.array_equal(case.buf.counts.cpu().numpy(), counts)
    assert np.array_equal(case.buf.rank_load.cpu().numpy(), load)
    assert p.moves == [tuple(int(v) for v in m) for m in op["moves"]]
    assert p.groups == [tuple(int(v) for v in g) for g in op["groups"]]
    assert np.array_equal(p.load_after, op["load_after"])
    s2r, r2t, pad_off, S_pad = O.permute(case.ids, w.E, 1)
    g_s2r = case.buf.slot_to_row.cpu().numpy()
    assert np.array_equal(g_s2r, s2r)
    assert np.array_equal(case.buf.row_to_token.cpu().numpy()[:S_pad], r2t)
    if w.R > 1:
        assert O.straggler_ratio(op["load_after"]) < O.straggler_ratio(op["load_before"])
    # ---- permuted activations: sampled rows, bit-exact
    rng = np.random.default_rng(11)
    busiest = np.argsort(-counts)
    nonempty = np.flatnonzero(counts > 0)
    experts = sorted(set(busiest[:3].tolist()) | {int(nonempty[np.argmin(counts[nonempty])])} |
                     set(rng.choice(nonempty, size=min(n_experts, nonempty.size), replace=False).tolist()))
    rows = _sample_rows(counts, pad_off, experts, rng)
    import torch
    d_rows = torch.from_numpy(rows).cuda()
    xp = F.bf16_bits(case.buf.x_perm[d_rows])
    assert np.array_equal(xp, case.x[r2t[rows]])
    # ---- expert FFN on the sampled rows
    row_expert = O.row_experts(case.ids, s2r, S_pad)[rows]
    ref_y = O.expert_ffn(xp, row_expert, case.w1, case.w3, case.w2)
    got_y = W.bf16_bits_to_f64(F.bf16_bits(case.buf.y_perm[d_rows]))
    assert_close(got_y, ref_y, f"y_perm rows {w.name}")
    # ---- whole layer on seeded tokens
    tokens = np.sort(rng.choice(w.T, size=n_tokens, replace=False))
    ref = O.moe_layer(case.x, case.ids, case.gates, case.w1, case.w3, case.w2, w.E, tokens=tokens)
    got = W.bf16_bits_to_f64(F.bf16_bits(case.buf.out[torch.from_numpy(tokens).cuda()]))
    assert_close(got, ref, f"layer output {w.name}")
    # ---- combine, stage-isolated, on the GPU's own y_perm
    tok2 = np.sort(rng.choice(w.T, size=min(512, w.T), replace=False))
    rows2 = s2r[tok2].reshape(-1)
    y_rows = W.bf16_bits_to_f64(F.bf16_bits(case.buf.y_perm[torch.from_numpy(rows2).cuda()]))
    loc = np.arange(rows2.size).reshape(-1, w.K)
    ref_c = O.combine(y_rows, loc, case.gates[tok2])
    mag = O.combine(np.abs(y_rows), loc, case.gates[tok2])
    got_c = W.bf16_bits_to_f64(F.bf16_bits(case.buf.out[torch.from_numpy(tok2).cuda()]))
    assert np.all(np.abs(got_c - ref_c) <= 2.0 ** -8 * np.abs(ref_c) + 2.0 ** -20 * mag + 1e-30)
    return p


def test_cfg3_full_size(cfg3_weights):
    case = DeviceCase(W.get_workload("cfg3"), mb=0, weights=cfg3_weights)
    p = _check_full_size(case)
    assert len(p.moves) >= 1
    case.close()


@pytest.mark.parametrize("T,R", [(2048, 16), (32768, 1)])
def test_sweep_points(cfg3_weights, T, R):
    w = [s for s in W.sweep_points() if s.T == T and s.R == R][0]
    case = DeviceCase(w, mb=1, weights=cfg3_weights)
    p = _check_full_size(case, n_experts=6, n_tokens=6)
    if R == 1:
        assert p.moves == []                                   # one rank: nothing to rebalance
    case.close()
