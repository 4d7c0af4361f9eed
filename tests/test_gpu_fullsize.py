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
    p_groups_cmp = p.groups           # (with phase2_copy the receive-slot labels live in the device table only)
    assert np.array_equal(case.buf.counts.cpu().numpy(), counts)
    assert np.array_equal(case.buf.rank_load.cpu().numpy(), load)
    assert p.moves == [tuple(int(v) for v in m) for m in op["moves"]]
    assert p_groups_cmp == [tuple(int(v) for v in g) for g in op["groups"]]
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


def test_cfg3_smooth_full_size(cfg3_weights):
    """The GLM-5-like layer with the popularity mixed half and half with the uniform distribution
    (unbalanced max/mean 1.1-1.7): a benchmarked workload, same weights as cfg3."""
    case = DeviceCase(W.get_workload("cfg3-smooth"), mb=2, weights=cfg3_weights)
    p = _check_full_size(case, n_experts=6, n_tokens=8)
    assert len(p.moves) >= 1
    case.close()


def test_cfg3_full_size_with_phase2_weight_copies(cfg3_weights):
    """cfg3 with the migrated experts' weights really copied into receive slots during the static
    GEMM (72 MiB per expert) and the dynamic GEMM reading them there."""
    case = DeviceCase(W.get_workload("cfg3"), mb=1, weights=cfg3_weights, phase2_copy=1)
    case.ctx.set_timeline(True)
    p = _check_full_size(case, n_experts=6, n_tokens=8)
    tl = case.ctx.get_timeline()
    assert tl["phase2_copy_bytes"] == 3 * 6144 * 2048 * 2 * len(p.moves) + sum(m[3] for m in p.moves) * 6144 * 2   # weights and rows
    case.close()


# (T, R): T = 65536 is the one size at which element offsets into x_perm / y_perm pass 2^31
# (524,288 rows x 6144 columns); the others cover every virtual EP degree of the sweep.
@pytest.mark.parametrize("T,R", [(2048, 16), (32768, 1), (8192, 2), (8192, 4), (65536, 8)])
def test_sweep_points(cfg3_weights, T, R):
    w = [s for s in W.sweep_points() if s.T == T and s.R == R][0]
    case = DeviceCase(w, mb=1, weights=cfg3_weights)
    p = _check_full_size(case, n_experts=6, n_tokens=6)
    if R == 1:
        assert p.moves == []                                   # one rank: nothing to rebalance
    if T == 65536:
        import torch
        # rows whose element offset exceeds 2^31: the last rows of the last non-empty expert were sampled
        # by _check_full_size only if that expert was drawn; check the very last live row explicitly
        s2r, r2t, pad_off, S_pad = O.permute(case.ids, w.E, 1)
        last = S_pad - 1
        assert last * w.d > 2 ** 31
        assert np.array_equal(F.bf16_bits(case.buf.x_perm[last]), case.x[r2t[last]])
        e_last = int(O.row_experts(case.ids, s2r, S_pad)[last])
        ref = O.expert_ffn(case.x[r2t[last]][None, :], np.array([e_last]), case.w1, case.w3, case.w2)
        got = W.bf16_bits_to_f64(F.bf16_bits(case.buf.y_perm[last]))[None, :]
        assert_close(got, ref, "last row of y_perm beyond 2^31 elements")
    case.close()


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_plan_upload_lands_inside_the_static_window(name, cfg3_weights):
    """Section 2.3's overlap condition, asserted: the planner thread has enqueued the upload of the
    dynamic group table before the static-expert GEMM ends.  Both intervals start when the counts
    leave the device: the host one is (upload enqueued - counts seen by the planner thread), the
    device one (counts written -> static tiles done).  Median over 20 forwards after warm-up."""
    w = W.get_workload(name)
    case = DeviceCase(w, mb=0, weights=cfg3_weights if name == "cfg3" else None)
    for _ in range(3):
        case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf, want_plan=False)
    case.ctx.check_status()
    case.ctx.set_timeline(True)
    host, dev, plan_us = [], [], []
    for _ in range(20):
        case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf, want_plan=False)
        tl = case.ctx.get_timeline()
        host.append(tl["host_upload_enqueued_us"] - tl["host_counts_ready_us"])
        dev.append(tl["dev_counts_to_static_end_us"])
        plan_us.append(tl["plan_us"])
    case.ctx.check_status()
    assert min(host) >= 0 and min(dev) > 0
    assert np.median(host) < np.median(dev), (np.median(host), np.median(dev))
    # the greedy itself is tens of microseconds at most (the paper quotes ~50 us on one core)
    assert np.median(plan_us) < 200
    case.close()


def test_cfg3_backward_full_size_sampled(cfg3_weights):
    """Backward pass at the GLM-5-like size, in the forms the context picks by itself (pair form for
    activation and weight gradients), accumulating into zeroed fp32 gradients.  The fp64 oracle
    cannot run the whole backward (3 x 9.9 TFLOP); it runs sub-problems whose gradients equal entries
    of the full problem's:
      * single (token, k) slots of a handful of tokens -> d_gates of those slots and, summed over k, d_x of those tokens;
      * one expert restricted to a few hidden units -> rows of dW1[e], dW3[e] and columns of dW2[e]
        for those units (every row of the expert's segment enters each entry), for the busiest and
        the smallest non-empty expert and two seeded ones;
    and d_gates in full, stage-isolated: <d_out[t], y_perm[row]> in fp64 over the GPU's own y_perm."""
    import torch
    w = W.get_workload("cfg3")
    case = DeviceCase(w, mb=0, weights=cfg3_weights, row_align=128)
    ctx, cfg = case.ctx, case.cfg
    bwd = F.BackwardBuffers(cfg)
    ctx.set_preact_buffer(bwd.ab)
    ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf, want_plan=False)
    w1t = torch.empty(w.E, w.d, w.f, dtype=torch.bfloat16, device="cuda")
    w3t = torch.empty_like(w1t)
    w2t = torch.empty(w.E, w.f, w.d, dtype=torch.bfloat16, device="cuda")
    ctx.transpose_weights(case.d_w1, case.d_w3, case.d_w2, w1t, w3t, w2t)
    rng = np.random.default_rng(21)
    d_out = W.f32_to_bf16_bits(rng.standard_normal((w.T, w.d)).astype(np.float32))
    dw1 = torch.zeros(w.E, w.f, w.d, dtype=torch.float32, device="cuda")
    dw3 = torch.zeros_like(dw1)
    dw2 = torch.zeros(w.E, w.d, w.f, dtype=torch.float32, device="cuda")
    ctx.moe_backward(F.bf16_tensor(d_out), case.d_gates, w1t, w3t, w2t, case.buf, bwd, dw1, dw3, dw2, accumulate=True)
    ctx.check_status()
    dO = W.bf16_bits_to_f64(d_out)

    def close(got, ref, what, tol=2e-2):
        bound = tol * np.abs(ref).max() + tol * np.abs(ref)
        err = np.abs(got - ref)
        assert np.all(err <= bound), (what, float(err.max()), float(np.abs(ref).max()))

    # ---- tokens: d_x and d_gates from the sub-problem made of these tokens alone
    tokens = np.sort(rng.choice(w.T, size=6, replace=False))
    rdx, rdg = np.zeros((tokens.size, w.d)), np.zeros((tokens.size, w.K))
    for i, t in enumerate(tokens):                              # one (token, k) slot at a time: d_x is their sum
        for k in range(w.K):
            e = int(case.ids[t, k])
            dx1, dg1, _, _, _ = O.moe_layer_backward(case.x[t][None], np.zeros((1, 1), np.int64), case.gates[t, k].reshape(1, 1),
                                                     case.w1[e][None], case.w3[e][None], case.w2[e][None], dO[t][None], 1)
            rdx[i] += dx1[0]
            rdg[i, k] = dg1[0, 0]
    d_tok = torch.from_numpy(tokens).cuda()
    close(W.bf16_bits_to_f64(F.bf16_bits(bwd.d_x[d_tok])), rdx, "d_x of sampled tokens")
    close(bwd.d_gates[d_tok].cpu().numpy().astype(np.float64), rdg, "d_gates of sampled tokens")
    # ---- d_gates in full against the GPU's own y_perm
    s2r = case.buf.slot_to_row.cpu().numpy()
    got_dg = bwd.d_gates.cpu().numpy().astype(np.float64)
    for t0 in range(0, w.T, 2048):
        rows = torch.from_numpy(s2r[t0:t0 + 2048].reshape(-1).astype(np.int64)).cuda()
        y = W.bf16_bits_to_f64(F.bf16_bits(case.buf.y_perm[rows])).reshape(-1, w.K, w.d)
        ref = np.einsum("td,tkd->tk", dO[t0:t0 + 2048], y)
        mag = np.einsum("td,tkd->tk", np.abs(dO[t0:t0 + 2048]), np.abs(y))
        assert np.all(np.abs(got_dg[t0:t0 + 2048] - ref) <= 2.0 ** -18 * mag + 1e-30), t0   # fp32 sum of 6144 products
    # ---- weight gradients of sampled experts on sampled hidden units
    counts = np.bincount(case.ids.ravel(), minlength=w.E)
    nonempty = np.flatnonzero(counts > 0)
    experts = sorted({int(np.argmax(counts)), int(nonempty[np.argmin(counts[nonempty])])} |
                     set(rng.choice(nonempty, size=2, replace=False).tolist()))
    units = np.array(sorted({0, 1, 127, 128, 255, 256, w.f - 1} | set(rng.integers(0, w.f, size=3).tolist())))
    d_units = torch.from_numpy(units).cuda()
    for e in experts:
        tt, kk = np.nonzero(case.ids == e)                      # slots of expert e, in segment order
        sub_ids = np.zeros((tt.size, 1), np.int64)
        _, _, r1, r3, r2 = O.moe_layer_backward(case.x[tt], sub_ids, case.gates[tt, kk][:, None],
                                                case.w1[e][units][None], case.w3[e][units][None],
                                                case.w2[e][:, units][None], dO[tt], 1)
        close(dw1[e][d_units].cpu().numpy().astype(np.float64), r1[0], f"dW1[{e}] ({tt.size} rows)")
        close(dw3[e][d_units].cpu().numpy().astype(np.float64), r3[0], f"dW3[{e}] ({tt.size} rows)")
        close(dw2[e][:, d_units].cpu().numpy().astype(np.float64), r2[0], f"dW2[{e}] ({tt.size} rows)")
    for e in np.flatnonzero(counts == 0)[:4]:
        assert not dw1[e].any() and not dw2[e].any()           # experts without rows: untouched zeros
    case.close()
