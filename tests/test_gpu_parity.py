"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer results bit-exact; floating point within
|gpu - ref| <= 1e-2 * max|ref| + 1e-2 * |ref| (bf16 inputs, fp32 accumulation)."""
import numpy as np
import pytest

from oracle import feplb_oracle as O
from paper_2604_19654_b200 import build as B
from paper_2604_19654_b200 import feplb as F
from paper_2604_19654_b200 import workloads as W

from gpu_utils import DeviceCase, assert_close, oracle_mask, upload_groups

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    B.build()


def _torch():
    import torch
    return torch


def _tiny(T, K, E, R, d=128, f=64, **kw):
    base = W.get_workload("cfg1")
    return base.with_(name="tiny", T=T, K=K, E=E, R=R, d=d, f=f, **kw)


# ----------------------------------------------------------------------------- integer stages

HIST_CASES = [W.get_workload("cfg1"), W.get_workload("cfg2"), W.get_workload("cfg4"),
              _tiny(1, 1, 4, 2), _tiny(37, 3, 6, 3), _tiny(1025, 5, 16, 4), _tiny(3000, 8, 128, 8),
              _tiny(64, 2, 1, 1),
              _tiny(77, 8, 16, 4, d=6144),       # six 2 KiB slices per row: a token's slices are copied by several warps and CTAs
              _tiny(50, 32, 64, 4, d=256)]       # the largest top-k


@pytest.mark.parametrize("w", HIST_CASES, ids=lambda w: f"{w.name}-T{w.T}K{w.K}E{w.E}")
@pytest.mark.parametrize("A", [1, 128])
def test_hist_and_dispatch_bit_exact(w, A):
    torch = _torch()
    ids, _ = W.gen_routing(w, 0) if w.E >= w.K and w.E > 1 else (np.zeros((w.T, w.K), np.int32), None)
    if w.name == "tiny" and w.E >= 4:
        rng = np.random.default_rng(w.T)
        ids = rng.integers(0, w.E, size=(w.T, w.K)).astype(np.int32)      # duplicates inside a token are legal
        ids[ids == 1] = 0                                                  # expert 1 stays empty
    x = W.gen_activations(w, 0)
    cfg = F.config_from_workload(w, row_align=A)
    ctx, buf = F.Context(cfg), F.Buffers(cfg)
    d_ids, d_x = torch.from_numpy(ids).cuda(), F.bf16_tensor(x)
    buf.x_perm.fill_(7.0)
    ctx.route_hist(d_ids, buf.counts, buf.rank_load)
    ctx.dispatch(d_x, d_ids, buf.counts, buf.x_perm, buf.slot_to_row, buf.row_to_token)
    ctx.check_status()
    counts, load = O.route_hist(ids, w.E, w.R)
    s2r, r2t, pad_off, S_pad = O.permute(ids, w.E, A)
    assert np.array_equal(buf.counts.cpu().numpy(), counts)
    assert np.array_equal(buf.rank_load.cpu().numpy(), load)
    assert np.array_equal(buf.slot_to_row.cpu().numpy()[: w.T], s2r)
    g_r2t = buf.row_to_token.cpu().numpy()
    assert np.array_equal(g_r2t[:S_pad], r2t)
    assert np.all(g_r2t[S_pad:] == -1)
    xp = O.gather_rows(x, r2t)
    assert np.array_equal(F.bf16_bits(buf.x_perm)[:S_pad], xp)            # row copies and zero padding
    ctx.close()


def test_out_of_range_expert_id_is_reported_not_trapped():
    torch = _torch()
    w = _tiny(64, 2, 8, 2)
    cfg = F.config_from_workload(w)
    ctx, buf = F.Context(cfg), F.Buffers(cfg)
    ids = np.zeros((w.T, w.K), np.int32)
    ids[5, 1] = 8
    ids[9, 0] = -3
    ctx.route_hist(torch.from_numpy(ids).cuda(), buf.counts, buf.rank_load)
    with pytest.raises(F.FeplbError) as ei:
        ctx.check_status()
    assert ei.value.code == F.E_RANGE
    assert int(buf.counts.sum()) == w.T * w.K - 2
    ctx.check_status()                                                    # the status word was cleared
    ctx.close()


def test_dispatch_skips_slots_with_an_id_out_of_range():
    """Slots whose id lies outside [0, E) get slot_to_row = -1 and no row; every other slot is ranked as the
    stable counting sort over the valid slots alone ranks it, and the error is reported."""
    torch = _torch()
    w = _tiny(300, 4, 8, 2, d=2304)                                       # 2304 / 8 = 288 chunks: a ragged third slice
    cfg = F.config_from_workload(w)
    ctx, buf = F.Context(cfg), F.Buffers(cfg)
    rng = np.random.default_rng(5)
    ids = rng.integers(0, w.E, size=(w.T, w.K)).astype(np.int32)
    bad = rng.random(ids.shape) < 0.05
    ids[bad] = np.where(rng.random(bad.sum()) < 0.5, w.E + 3, -1)
    x = W.gen_activations(w, 0)
    d_ids = torch.from_numpy(ids).cuda()
    ctx.route_hist(d_ids, buf.counts, buf.rank_load)
    with pytest.raises(F.FeplbError):
        ctx.check_status()
    buf.x_perm.fill_(7.0)
    ctx.dispatch(F.bf16_tensor(x), d_ids, buf.counts, buf.x_perm, buf.slot_to_row, buf.row_to_token)
    with pytest.raises(F.FeplbError) as ei:
        ctx.check_status()
    assert ei.value.code == F.E_RANGE
    flat = ids.reshape(-1)
    valid = np.flatnonzero(~bad.reshape(-1))
    order = valid[np.argsort(flat[valid], kind="stable")]                 # valid slots in expert order, ties by slot
    want = np.full(flat.size, -1, np.int32)
    want[order] = np.arange(order.size, dtype=np.int32)
    assert np.array_equal(buf.slot_to_row.cpu().numpy().reshape(-1), want)
    r2t = buf.row_to_token.cpu().numpy()
    assert np.array_equal(r2t[: order.size], (order // w.K).astype(np.int32))
    assert np.all(r2t[order.size:] == -1)
    got = F.bf16_bits(buf.x_perm)
    assert np.array_equal(got[: order.size], x[order // w.K])
    assert np.all(got[order.size:] == 0x40E0)                             # bf16 7.0: rows without a slot stay untouched
    ctx.close()


def test_dispatch_with_wrong_counts_is_reported():
    torch = _torch()
    w = _tiny(64, 2, 8, 2)
    cfg = F.config_from_workload(w)
    ctx, buf = F.Context(cfg), F.Buffers(cfg)
    ids = np.random.default_rng(0).integers(0, 8, size=(w.T, w.K)).astype(np.int32)
    d_ids = torch.from_numpy(ids).cuda()
    ctx.route_hist(d_ids, buf.counts, buf.rank_load)
    buf.counts[3] += 1
    ctx.dispatch(F.bf16_tensor(W.gen_activations(w, 0)), d_ids, buf.counts, buf.x_perm, buf.slot_to_row, buf.row_to_token)
    with pytest.raises(F.FeplbError) as ei:
        ctx.check_status()
    assert ei.value.code == F.E_DEVICE
    ctx.close()


@pytest.mark.parametrize("A", [1, 128])
@pytest.mark.parametrize("noalloc", [False, True])
def test_dispatch_with_wrong_counts_stays_inside_the_buffers(A, noalloc):
    """Counts that disagree with the ids (too large, too small, negative, absurdly large) give a wrong
    permutation and FEPLB_E_DEVICE, but no access outside x_perm / row_to_token: both are
    allocated with guard rows behind them that must stay untouched, and every slot_to_row entry is
    -1 or a row inside the buffer."""
    torch = _torch()
    w = _tiny(64, 2, 8, 2)
    cfg = F.config_from_workload(w, row_align=A)
    ctx, buf = F.Context(cfg), F.Buffers(cfg)
    cap, guard = F.s_pad(cfg), 64
    ids = np.random.default_rng(0).integers(0, 8, size=(w.T, w.K)).astype(np.int32)
    d_ids = torch.from_numpy(ids).cuda()
    d_x = F.bf16_tensor(W.gen_activations(w, 0))
    true_counts = np.bincount(ids.ravel(), minlength=w.E).astype(np.int32)
    for delta in ({3: +1}, {7: +5}, {0: -2}, {2: -10 ** 6}, {1: 2 ** 30, 2: 2 ** 30, 3: 2 ** 30}, {5: +1000}):
        counts = true_counts.copy()
        for e, dv in delta.items():
            counts[e] = dv if abs(dv) >= 10 ** 6 else counts[e] + dv
        xp = torch.full((cap + guard, w.d), 9.0, dtype=torch.bfloat16, device="cuda")
        r2t = torch.full((cap + guard,), 12345, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        d_counts = torch.from_numpy(counts).cuda()
        if noalloc:
            F.dispatch_noalloc(cfg, d_x, d_ids, d_counts, xp, buf.slot_to_row, r2t, status)
            torch.cuda.synchronize()
            assert int(status.item()) & 2
        else:
            ctx.dispatch(d_x, d_ids, d_counts, xp, buf.slot_to_row, r2t)
            with pytest.raises(F.FeplbError) as ei:
                ctx.check_status()
            assert ei.value.code == F.E_DEVICE
        assert bool((xp[cap:] == 9.0).all()) and bool((r2t[cap:] == 12345).all()), delta
        s2r = buf.slot_to_row.cpu().numpy()
        assert ((s2r >= -1) & (s2r < cap)).all(), delta
    ctx.close()


def test_home_groups_match_the_no_move_plan():
    torch = _torch()
    for w, A in ((W.get_workload("cfg2"), 1), (W.get_workload("cfg1"), 128)):
        ids, _ = W.gen_routing(w, 1)
        cfg = F.config_from_workload(w, row_align=A)
        ctx, buf = F.Context(cfg), F.Buffers(cfg)
        ctx.route_hist(torch.from_numpy(ids).cuda(), buf.counts, buf.rank_load)
        groups = torch.zeros(w.E, 5, dtype=torch.int32, device="cuda")
        mask_out = torch.zeros(w.E, dtype=torch.uint8, device="cuda")
        ctx.home_groups(buf.counts, None, groups, mask_out)               # REACTIVE: mask from counts on the device
        counts, _ = O.route_hist(ids, w.E, w.R)
        mask = oracle_mask(counts, w)
        assert np.array_equal(mask_out.cpu().numpy(), mask)
        pad_off, _ = O.segment_offsets(counts, A)
        exp = [(e, int(pad_off[e]), int(counts[e]), e // w.L, int(mask[e])) for e in range(w.E)]
        assert [tuple(r) for r in groups.cpu().numpy().tolist()] == exp
        # the oracle's plan with an empty mask lists the same non-empty groups
        p = O.plan(counts, np.zeros(w.E, np.uint8), w.R, row_align=A)
        assert [g[:4] for g in p["groups"]] == [g[:4] for g in exp if g[2] > 0]
        ctx.close()


# ----------------------------------------------------------------------------- expert FFN

def _ffn_case(E, d, f, rows_per_expert, A=1, seed=0, order=None, form=None):
    """Builds x_perm / groups for the given per-expert row counts and checks H-free Y parity."""
    torch = _torch()
    rng = np.random.default_rng(seed)
    counts = np.asarray(rows_per_expert)
    pad_off, S_pad = O.segment_offsets(counts, A)
    w = _tiny(max(int(counts.sum()), 1), 1, E, 1, d=d, f=f)
    cfg = F.config_from_workload(w, row_align=A)
    ctx = F.Context(cfg)
    if form is not None:
        ctx.set_gemm_form(form)
    cap = F.s_pad(cfg)
    xb = W.f32_to_bf16_bits((rng.standard_normal((cap, d)) * 0.5).astype(np.float32))
    w1 = W.f32_to_bf16_bits((rng.standard_normal((E, f, d)) / np.sqrt(d)).astype(np.float32))
    w3 = W.f32_to_bf16_bits((rng.standard_normal((E, f, d)) / np.sqrt(d)).astype(np.float32))
    w2 = W.f32_to_bf16_bits((rng.standard_normal((E, d, f)) / np.sqrt(f)).astype(np.float32))
    row_expert = np.full(cap, -1, np.int64)
    groups = []
    for e in range(E):
        row_expert[pad_off[e]: pad_off[e] + counts[e]] = e
        groups.append((e, int(pad_off[e]), int(counts[e]), 0, e % 2))
    if order is not None:
        groups = [groups[i] for i in order]
    d_x, d_w1, d_w3, d_w2 = (F.bf16_tensor(a) for a in (xb, w1, w3, w2))
    h = torch.zeros(cap, f, dtype=torch.bfloat16, device="cuda")
    y = torch.full((cap, d), 3.0, dtype=torch.bfloat16, device="cuda")
    d_groups = upload_groups(groups)
    ctx.expert_ffn(d_x, d_w1, d_w3, d_w2, d_groups, len(groups), h, y, which=F.FFN_STATIC)
    ctx.expert_ffn(d_x, d_w1, d_w3, d_w2, d_groups, len(groups), h, y, which=F.FFN_DYNAMIC)
    ctx.check_status()
    ref = O.expert_ffn(xb, row_expert, w1, w3, w2)
    got = W.bf16_bits_to_f64(F.bf16_bits(y))
    live = row_expert >= 0
    worst = assert_close(got[live], ref[live], f"FFN E={E} d={d} f={f}")
    assert np.all(got[~live] == 3.0)                                      # rows outside the groups are untouched
    ctx.close()
    return worst


@pytest.mark.parametrize("E,d,f,rows", [
    (1, 128, 64, [128]),                       # one full tile, smallest shapes (bn = 64 in both passes)
    (1, 128, 64, [1]),                         # a single row
    (2, 128, 64, [5, 200]),                    # ragged last tiles
    (4, 256, 128, [0, 129, 0, 383]),           # empty experts; bn = 128 in both passes
    (3, 512, 192, [300, 17, 128]),             # f % 128 != 0 -> bn = 64 in pass 1, 128 in pass 2
    (8, 384, 256, [64, 1, 0, 257, 128, 127, 513, 2]),   # d % 256 != 0 -> bn = 64 in pass 2
    (2, 2048, 768, [700, 45]),                 # the mid layer's shapes: 32 K blocks wrap the 4-stage ring
])
def test_expert_ffn_parity(E, d, f, rows):
    _ffn_case(E, d, f, rows)


@pytest.mark.parametrize("form", [F.FORM_SINGLE, F.FORM_PAIR, F.FORM_WEIGHT_M])
@pytest.mark.parametrize("E,d,f,rows", [
    (1, 256, 128, [1]),                        # one row: a 16-row block, one chunk for half of the epilogue warps
    (4, 256, 128, [0, 129, 0, 383]),           # empty experts; blocks of 144, 192 + 191 rows
    (3, 512, 256, [16, 17, 33]),               # block sizes around the 16-row granule and the 32-row chunk
    (2, 256, 384, [128, 256]),                 # exactly one small and one big unit per weight-tile pair
    (5, 256, 128, [257, 31, 255, 513, 97]),    # alternating small / big units: both TMEM slot schemes in turn
    (2, 2048, 768, [700, 45]),                 # the mid layer's shapes: 32 K blocks wrap the 3-stage ring many times
    (2, 512, 128, [5000, 3]),                  # many blocks of one group, more units than CTAs in pass 2
])
def test_expert_ffn_parity_in_every_form(E, d, f, rows, form):
    """Shapes every form supports (f % 128 == 0, d % 256 == 0), each form forced in turn."""
    _ffn_case(E, d, f, rows, form=form)
    _ffn_case(E, d, f, rows, A=128, form=form, order=list(range(E))[::-1])


def test_expert_ffn_intermediates_within_rounding_of_the_oracle():
    """Stage-isolated and tight: the H buffer against the oracle's hidden activation rounded to bf16,
    and Y against the oracle fed with that rounded H.  One bf16 rounding is 2^-9 relative; allowed
    here: 2^-7 of the value (a near-tie of the fp32 vs fp64 sum may flip the rounding, and fp32
    accumulation order differs) plus, for values that are themselves the result of cancellation,
    2^-16 (H) and 2^-10 (Y, a sum over f products) of the largest value.  Measured: 99.95 % of H
    equal bit for bit, the rest one bf16 step apart; Y within 2^-11 of the largest value."""
    torch = _torch()
    w = W.get_workload("cfg2").with_(T=600, E=8, R=2, d=512, f=256)
    case = DeviceCase(w)
    case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    case.ctx.check_status()
    s2r, r2t, _, S_pad = O.permute(case.ids, w.E, 1)
    rexp = O.row_experts(case.ids, s2r, S_pad)
    x_rows = O.gather_rows(case.x, r2t)
    h_ref = O._round_f64_to_bf16(O.expert_hidden(x_rows, rexp, case.w1, case.w3))
    h_gpu = W.bf16_bits_to_f64(F.bf16_bits(case.buf.h_scratch))[:S_pad]
    assert np.all(np.abs(h_gpu - h_ref) <= 2.0 ** -7 * np.abs(h_ref) + 2.0 ** -16 * np.abs(h_ref).max())
    assert np.mean(h_gpu == h_ref) > 0.99                      # nearly all elements round the same way
    y_ref = O.expert_ffn(x_rows, rexp, case.w1, case.w3, case.w2, round_h_bf16=True)
    y_gpu = W.bf16_bits_to_f64(F.bf16_bits(case.buf.y_perm))[:S_pad]
    assert np.all(np.abs(y_gpu - y_ref) <= 2.0 ** -7 * np.abs(y_ref) + 2.0 ** -10 * np.abs(y_ref).max())
    case.close()


def test_expert_ffn_padded_segments_and_group_order():
    _ffn_case(5, 256, 128, [130, 0, 7, 256, 90], A=128)
    _ffn_case(5, 256, 128, [130, 0, 7, 256, 90], A=1, order=[4, 2, 0, 3, 1])


def test_expert_ffn_many_tiles_per_cta():
    # more tiles than CTAs: every CTA walks several tiles, both accumulator stages and phases flip
    _ffn_case(6, 256, 128, [4000, 3000, 2500, 1, 6000, 777])


def test_expert_ffn_rejects_bad_group_without_trapping():
    torch = _torch()
    w = _tiny(128, 1, 2, 1)
    cfg = F.config_from_workload(w)
    ctx = F.Context(cfg)
    cap = F.s_pad(cfg)
    z = torch.zeros(cap, 128, dtype=torch.bfloat16, device="cuda")
    wz = torch.zeros(2, 64, 128, dtype=torch.bfloat16, device="cuda")
    w2z = torch.zeros(2, 128, 64, dtype=torch.bfloat16, device="cuda")
    h = torch.zeros(cap, 64, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(cap, 128, dtype=torch.bfloat16, device="cuda")
    bad = upload_groups([(5, 0, 10, 0, 0), (0, 100, 100, 0, 0)])          # expert out of range; rows past the buffer
    ctx.expert_ffn(z, wz, wz, w2z, bad, 2, h, y)
    with pytest.raises(F.FeplbError) as ei:
        ctx.check_status()
    assert ei.value.code == F.E_DEVICE
    with pytest.raises(F.FeplbError):
        ctx.expert_ffn(z, wz, wz, w2z, bad, 5000, h, y)                   # more groups than the table holds
    ctx.close()


# ----------------------------------------------------------------------------- combine

@pytest.mark.parametrize("T,K,d", [(1, 1, 128), (33, 2, 128), (257, 6, 2048), (100, 8, 6144), (50, 32, 256)])
def test_combine_parity(T, K, d):
    torch = _torch()
    rng = np.random.default_rng(T * K)
    w = _tiny(T, K, 32, 1, d=d)
    cfg = F.config_from_workload(w)
    ctx = F.Context(cfg)
    rows = T * K
    y = W.f32_to_bf16_bits(rng.standard_normal((rows, d)).astype(np.float32))
    s2r = rng.permutation(rows).astype(np.int32).reshape(T, K)
    gates = rng.random((T, K)).astype(np.float32)
    out = torch.zeros(T, d, dtype=torch.bfloat16, device="cuda")
    ctx.combine(F.bf16_tensor(y), torch.from_numpy(s2r).cuda(), torch.from_numpy(gates).cuda(), out)
    ref = O.combine(W.bf16_bits_to_f64(y), s2r, gates)
    got = W.bf16_bits_to_f64(F.bf16_bits(out))
    # one bf16 rounding of the result (2^-9 relative) plus fp32 accumulation error on the sum of |terms|
    mag = O.combine(np.abs(W.bf16_bits_to_f64(y)), s2r, gates)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -20 * mag + 1e-30)
    ctx.close()


def test_dispatch_then_combine_is_the_identity_for_k1():
    torch = _torch()
    w = _tiny(777, 1, 16, 4, d=256)
    cfg = F.config_from_workload(w, row_align=128)
    ctx, buf = F.Context(cfg), F.Buffers(cfg)
    ids = np.random.default_rng(1).integers(0, 16, size=(w.T, 1)).astype(np.int32)
    x = W.gen_activations(w, 0)
    d_ids = torch.from_numpy(ids).cuda()
    ctx.route_hist(d_ids, buf.counts, buf.rank_load)
    ctx.dispatch(F.bf16_tensor(x), d_ids, buf.counts, buf.x_perm, buf.slot_to_row, buf.row_to_token)
    ctx.combine(buf.x_perm, buf.slot_to_row, torch.ones(w.T, 1, device="cuda"), buf.out)
    ctx.check_status()
    assert np.array_equal(F.bf16_bits(buf.out)[: w.T], x)
    ctx.close()


# ----------------------------------------------------------------------------- whole layer

def _check_forward(case, split=0, sample=None):
    w = case.w
    p = case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    case.ctx.check_status()
    counts, load = O.route_hist(case.ids, w.E, w.R)
    mask = oracle_mask(counts, w)
    A = case.cfg.row_align
    op = O.plan(counts, mask, w.R, tau=case.cfg.tau, max_num_dyn=case.cfg.max_num_dyn, policy=case.cfg.policy,
                split=case.cfg.split, split_granule=case.cfg.split_granule, row_align=A)
    # integer outputs bit-exact: counts, per-rank loads before/after, moves, groups, permutation
    assert np.array_equal(case.buf.counts.cpu().numpy(), counts)
    assert np.array_equal(case.buf.rank_load.cpu().numpy(), load)
    assert p.moves == [tuple(int(v) for v in m) for m in op["moves"]]
    assert p.groups == [tuple(int(v) for v in g) for g in op["groups"]]
    assert np.array_equal(p.load_before, op["load_before"]) and np.array_equal(p.load_after, op["load_after"])
    s2r, r2t, _, S_pad = O.permute(case.ids, w.E, A)
    assert np.array_equal(case.buf.slot_to_row.cpu().numpy()[: w.T], s2r)
    assert np.array_equal(case.buf.row_to_token.cpu().numpy()[:S_pad], r2t)
    assert O.straggler_ratio(op["load_after"]) <= O.straggler_ratio(op["load_before"])
    got = W.bf16_bits_to_f64(F.bf16_bits(case.buf.out))[: w.T]
    tokens = None if sample is None else np.sort(np.random.default_rng(5).choice(w.T, size=sample, replace=False))
    ref = O.moe_layer(case.x, case.ids, case.gates, case.w1, case.w3, case.w2, w.E, tokens=tokens)
    assert_close(got if tokens is None else got[tokens], ref, f"layer output {w.name}")
    return p, op


@pytest.mark.parametrize("A", [1, 128])
def test_forward_cfg1(A):
    case = DeviceCase(W.get_workload("cfg1"), row_align=A)
    p, _ = _check_forward(case)
    assert len(p.moves) >= 1
    # a second pass on the same context gives bit-identical results (determinism)
    out1 = F.bf16_bits(case.buf.out).copy()
    y1 = F.bf16_bits(case.buf.y_perm).copy()
    case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    _torch().cuda.synchronize()
    assert np.array_equal(F.bf16_bits(case.buf.out), out1)
    n_live = int(case.ids.size)
    assert np.array_equal(F.bf16_bits(case.buf.y_perm)[:n_live], y1[:n_live]) or A == 128
    case.close()


def _random_workload(seed):
    """A seeded random small layer: odd token counts, expert counts that are not powers of two,
    several ranks, widths that give two to six 64-wide K blocks and ragged N tiles."""
    rng = np.random.default_rng(4200 + seed)
    R = int(rng.choice([1, 2, 3, 4]))
    L = int(rng.choice([1, 2, 3, 5, 8]))
    E = R * L
    K = int(rng.integers(1, min(E, 8) + 1))
    w = W.get_workload("cfg2").with_(
        name=f"rand{seed}", T=int(rng.integers(1, 700)), E=E, R=R, K=K,
        d=int(rng.choice([128, 256, 384])), f=int(rng.choice([64, 128, 192, 256])),
        dyn=int(rng.integers(0, L + 1)), max_num_dyn=int(rng.integers(0, 4)), tau=int(rng.choice([0, 1, 8, 64])),
        routing=str(rng.choice(["dirichlet", "zipf"])), alpha=float(rng.choice([0.2, 0.5, 1.2])))
    return w, int(rng.choice([1, 128])), int(rng.integers(0, 2)), int(rng.integers(0, 2))


@pytest.mark.parametrize("seed", range(16))
def test_forward_random_shapes(seed):
    w, A, split, pair = _random_workload(seed)
    case = DeviceCase(w, mb=seed, row_align=A, split=split, split_granule=128 if A == 128 else 16)
    case.ctx.set_gemm_form(F.FORM_PAIR if pair else F.FORM_SINGLE)
    case.ctx.set_launch_merging((seed >> 1) & 1)      # both launch orders: four launches, or two that pick the plan up on the device
    case.ctx.set_timeline(True)
    _check_forward(case)
    assert case.ctx.get_timeline()["ffn_launches"] == (2 if (seed >> 1) & 1 else 4)
    case.close()


def test_forward_at_the_maximum_top_k():
    """K = 32 (the library's limit): every token goes to 32 of 64 experts."""
    w = W.get_workload("cfg2").with_(name="maxK", T=333, E=64, R=4, K=32, d=256, f=128, dyn=4, max_num_dyn=4, tau=1)
    case = DeviceCase(w)
    _check_forward(case)
    case.close()


@pytest.mark.parametrize("A", [1, 128])
def test_forward_at_the_maximum_expert_count(A):
    """E = 1024 (the library's limit) on 16 ranks: group tables of 1024 entries, most experts with a
    handful of rows or none."""
    w = W.get_workload("cfg2").with_(name="maxE", T=1500, E=1024, R=16, K=8, d=128, f=64, dyn=8, max_num_dyn=4, tau=1, alpha=0.3)
    case = DeviceCase(w, row_align=A)
    _check_forward(case, sample=200)
    case.close()


def _random_workload_wm(seed):
    """Seeded random small layers in shapes the weights-on-M form takes (f % 128 == 0, d % 256 == 0)."""
    rng = np.random.default_rng(5200 + seed)
    R = int(rng.choice([1, 2, 3, 4]))
    L = int(rng.choice([1, 2, 3, 5, 8]))
    E = R * L
    K = int(rng.integers(1, min(E, 8) + 1))
    w = W.get_workload("cfg2").with_(
        name=f"randwm{seed}", T=int(rng.integers(1, 1500)), E=E, R=R, K=K,
        d=int(rng.choice([256, 512])), f=int(rng.choice([128, 256, 384])),
        dyn=int(rng.integers(0, L + 1)), max_num_dyn=int(rng.integers(0, 4)), tau=int(rng.choice([0, 1, 8, 64])),
        routing=str(rng.choice(["dirichlet", "zipf"])), alpha=float(rng.choice([0.2, 0.5, 1.2])))
    return w, int(rng.choice([1, 128])), int(rng.integers(0, 2)), int(rng.integers(0, 2))


@pytest.mark.parametrize("seed", range(16))
def test_forward_random_shapes_weights_on_m(seed):
    """The whole layer with the weights-on-M form forced: one launch per pass runs the static groups
    and then picks the planner's dynamic table up on the device.  Odd seeds also copy the migrated
    experts' weights into receive slots (Phase 2)."""
    w, A, split, phase2 = _random_workload_wm(seed)
    case = DeviceCase(w, mb=seed, row_align=A, split=split, split_granule=128 if A == 128 else 16, phase2_copy=phase2)
    case.ctx.set_gemm_form(F.FORM_WEIGHT_M)
    case.ctx.set_launch_merging(1)
    case.ctx.set_timeline(bool(seed & 1))
    _check_forward(case)
    if seed & 1:
        tl = case.ctx.get_timeline()
        if phase2:                             # with weight copies the dynamic groups keep launches of their own
            assert tl["ffn_launches"] == 4
        else:
            assert tl["ffn_launches"] == 2 and tl["dev_ffn_pass1_us"] > 0 and tl["dev_ffn_pass2_us"] > 0
            assert tl["dev_counts_to_static_start_us"] > 0
    # the same layer in the four-launch single-CTA form gives the same integers and an output within tolerance
    out_wm = W.bf16_bits_to_f64(F.bf16_bits(case.buf.out))[: w.T].copy()
    case.ctx.set_gemm_form(F.FORM_SINGLE)
    _check_forward(case)
    out_s = W.bf16_bits_to_f64(F.bf16_bits(case.buf.out))[: w.T]
    assert np.abs(out_wm - out_s).max() <= 2e-2 * max(np.abs(out_s).max(), 1e-30)
    case.close()


def test_weights_on_m_form_is_refused_for_shapes_it_does_not_take():
    case = DeviceCase(W.get_workload("cfg1"))                 # d = 128, f = 64
    with pytest.raises(F.FeplbError) as ei:
        case.ctx.set_gemm_form(F.FORM_WEIGHT_M)
    assert ei.value.code == F.E_INVALID
    _check_forward(case)
    case.close()


@pytest.mark.parametrize("form", [F.FORM_SINGLE, F.FORM_PAIR, F.FORM_WEIGHT_M])
def test_dynamic_table_arriving_late_is_waited_for_on_the_device(form):
    """The planner is held back for 3 ms, far longer than the static groups take, so every CTA of the
    merged launch runs out of static work and really waits for the table (bounded); results are
    unchanged and the timeline shows the wait."""
    w = W.get_workload("cfg2").with_(T=1024)
    case = DeviceCase(w, mb=1)
    case.ctx.set_gemm_form(form)
    case.ctx.set_launch_merging(1)
    case.ctx.set_timeline(True)
    case.ctx.set_planner_timing(planner_delay_us=3000)
    p, _ = _check_forward(case)
    assert len(p.moves) >= 1
    tl = case.ctx.get_timeline()
    assert tl["dev_plan_wait_us"] > 500, tl
    case.ctx.set_planner_timing(0, 0)
    waits = []
    for _ in range(5):                       # the best of five: a busy host can hold the planner thread up by itself
        _check_forward(case)
        waits.append(case.ctx.get_timeline()["dev_plan_wait_us"])
    assert min(waits) < tl["dev_plan_wait_us"], (waits, tl)
    case.close()


@pytest.mark.parametrize("form", [F.FORM_SINGLE, F.FORM_PAIR, F.FORM_WEIGHT_M])
def test_device_wait_for_the_plan_expires_cleanly(form):
    """The planner is held back for 150 ms while the GEMM's wait for its table is limited to 2 ms: the
    kernels give up, skip the dynamic groups, raise the status bit and return; the forward call itself
    succeeds (the plan did arrive on the host), feplb_check_status reports FEPLB_E_TIMEOUT, nothing
    hangs and the next forward is correct."""
    w = W.get_workload("cfg2").with_(T=1024)
    case = DeviceCase(w, mb=1)
    case.ctx.set_gemm_form(form)
    case.ctx.set_launch_merging(1)
    case.ctx.set_planner_timing(planner_delay_us=150000, device_wait_limit_us=2000)
    case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    with pytest.raises(F.FeplbError) as ei:
        case.ctx.check_status()
    assert ei.value.code == F.E_TIMEOUT
    case.ctx.set_planner_timing(0, 0)
    case.ctx.check_status()
    _check_forward(case)
    case.close()


@pytest.mark.parametrize("seed", range(4))
def test_forward_cfg1_other_seeds(seed):
    w = W.get_workload("cfg1")
    case = DeviceCase(w, mb=10 + seed)
    _check_forward(case)
    case.close()


def test_forward_cfg2_full():
    w = W.get_workload("cfg2")
    weights = W.gen_weights(w)
    for mb in (0, 3):
        case = DeviceCase(w, mb=mb, weights=weights)
        _check_forward(case, sample=None if mb == 0 else 256)
        case.close()


@pytest.mark.parametrize("split", [0, 1])
def test_forward_cfg4_extreme_skew(split):
    w = W.get_workload("cfg4")
    case = DeviceCase(w, mb=0, split=split)
    p, op = _check_forward(case, sample=512)
    if split:
        assert any(rows < max(c, 1) for (e, _, _, rows) in p.moves
                   for c in [int(np.bincount(case.ids.ravel(), minlength=w.E)[e])])   # a hot expert was cut
    case.close()


def test_forward_given_mask_and_literal_policy():
    w = W.get_workload("cfg2").with_(T=512)
    mask = np.zeros(w.E, np.uint8)
    mask[::4] = 1
    case = DeviceCase(w, mb=2, mask_policy=F.MASK_GIVEN, policy=F.POLICY_LITERAL)
    p = case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf,
                             dyn_mask_host=mask)
    case.ctx.check_status()
    counts, _ = O.route_hist(case.ids, w.E, w.R)
    op = O.plan(counts, mask, w.R, tau=w.tau, max_num_dyn=w.max_num_dyn, policy=O.POLICY_LITERAL)
    assert p.moves == [tuple(int(v) for v in m) for m in op["moves"]]
    assert p.groups == [tuple(int(v) for v in g) for g in op["groups"]]
    got = W.bf16_bits_to_f64(F.bf16_bits(case.buf.out))[: w.T]
    ref = O.moe_layer(case.x, case.ids, case.gates, case.w1, case.w3, case.w2, w.E)
    assert_close(got, ref, "layer output, given mask")
    with pytest.raises(F.FeplbError):                                      # a mask is mandatory in this mode
        case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    case.close()


def test_forward_host_buffers_and_timeline():
    torch = _torch()
    w = W.get_workload("cfg1")
    case = DeviceCase(w)
    case.ctx.set_timeline(True)
    xh = torch.from_numpy(case.x.view(np.int16)).pin_memory()
    ih = torch.from_numpy(case.ids).pin_memory()
    gh = torch.from_numpy(case.gates).pin_memory()
    oh = torch.zeros(w.T, w.d, dtype=torch.int16).pin_memory()
    x_dev = torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda")
    i_dev = torch.empty(w.T, w.K, dtype=torch.int32, device="cuda")
    g_dev = torch.empty(w.T, w.K, dtype=torch.float32, device="cuda")
    case.ctx.moe_forward_host(xh, ih, gh, x_dev, i_dev, g_dev, case.d_w1, case.d_w3, case.d_w2, case.buf, oh)
    case.ctx.check_status()
    ref = O.moe_layer(case.x, case.ids, case.gates, case.w1, case.w3, case.w2, w.E)
    assert_close(W.bf16_bits_to_f64(oh.numpy().view(np.uint16)), ref, "host-buffer forward")
    tl = case.ctx.get_timeline()
    assert tl["dev_total_us"] > 0 and tl["host_plan_done_us"] >= tl["host_counts_ready_us"] > 0
    assert tl["dev_static_ffn_us"] > 0 and tl["plan_us"] >= 0
    assert case.ctx.launch_count() > 0
    case.close()


def test_plan_wait_without_request_and_timeout_paths():
    w = W.get_workload("cfg1")
    cfg = F.config_from_workload(w)
    ctx = F.Context(cfg)
    with pytest.raises(F.FeplbError) as ei:
        ctx.plan_wait(10)
    assert ei.value.code == F.E_STATE
    ctx.close()


def test_empty_batch():
    w = _tiny(0, 2, 8, 2)
    cfg = F.config_from_workload(w)
    ctx, buf = F.Context(cfg), F.Buffers(cfg)
    torch = _torch()
    z = torch.zeros(1, 128, dtype=torch.bfloat16, device="cuda")
    zi = torch.zeros(1, 2, dtype=torch.int32, device="cuda")
    wz = torch.zeros(8, 64, 128, dtype=torch.bfloat16, device="cuda")
    w2z = torch.zeros(8, 128, 64, dtype=torch.bfloat16, device="cuda")
    p = ctx.moe_forward(z, zi, torch.zeros(1, 2, device="cuda"), wz, wz, w2z, buf)
    ctx.check_status()
    assert p.moves == [] and p.groups == [] and int(buf.counts.sum()) == 0
    ctx.close()


def test_pipelined_host_forward_matches_the_synchronous_one():
    """Back-to-back micro-batches through the two-slot pipelined entry point give, bit for bit, what
    the synchronous host-buffer entry point gives for each of them."""
    torch = _torch()
    w = W.get_workload("cfg2").with_(T=1024)
    case = DeviceCase(w, mb=0)
    mbs = [W.gen_microbatch(w, mb) for mb in range(5)]
    pin = [(torch.from_numpy(x.view(np.int16)).pin_memory(), torch.from_numpy(i).pin_memory(),
            torch.from_numpy(g).pin_memory()) for x, i, g in mbs]
    x_dev = [torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    i_dev = [torch.empty(w.T, w.K, dtype=torch.int32, device="cuda") for _ in range(2)]
    g_dev = [torch.empty(w.T, w.K, dtype=torch.float32, device="cuda") for _ in range(2)]
    o_dev = [torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    ref = []
    for xh, ih, gh in pin:
        oh = torch.zeros(w.T, w.d, dtype=torch.int16).pin_memory()
        case.ctx.moe_forward_host(xh, ih, gh, x_dev[0], i_dev[0], g_dev[0], case.d_w1, case.d_w3, case.d_w2, case.buf, oh)
        ref.append(oh.numpy().copy())
    outs = [torch.zeros(w.T, w.d, dtype=torch.int16).pin_memory() for _ in pin]   # one host buffer per micro-batch
    for n, (xh, ih, gh) in enumerate(pin):
        s = n & 1
        case.ctx.host_wait(s)
        case.ctx.moe_forward_host_async(s, xh, ih, gh, x_dev[s], i_dev[s], g_dev[s], case.d_w1, case.d_w3, case.d_w2,
                                        case.buf, o_dev[s], outs[n])
    case.ctx.host_wait(0)
    case.ctx.host_wait(1)
    case.ctx.check_status()
    for n in range(len(pin)):
        assert np.array_equal(outs[n].numpy(), ref[n]), n
    # the same with the inputs of micro-batch n+1 staged ahead of the forward of micro-batch n;
    # the forward then ignores its host input pointers (a wrong micro-batch's are passed on purpose)
    outs2 = [torch.zeros(w.T, w.d, dtype=torch.int16).pin_memory() for _ in pin]
    case.ctx.host_stage_inputs(0, *pin[0], x_dev[0], i_dev[0], g_dev[0])
    with pytest.raises(F.FeplbError):
        case.ctx.host_stage_inputs(0, *pin[0], x_dev[0], i_dev[0], g_dev[0])      # slot already staged
    for n in range(len(pin)):
        s = n & 1
        if n + 1 < len(pin):
            case.ctx.host_stage_inputs(s ^ 1, *pin[n + 1], x_dev[s ^ 1], i_dev[s ^ 1], g_dev[s ^ 1])
        case.ctx.host_wait(s)
        xh, ih, gh = pin[(n + 1) % len(pin)]
        case.ctx.moe_forward_host_async(s, xh, ih, gh, x_dev[s], i_dev[s], g_dev[s], case.d_w1, case.d_w3, case.d_w2,
                                        case.buf, o_dev[s], outs2[n])
    case.ctx.host_wait(0)
    case.ctx.host_wait(1)
    case.ctx.check_status()
    for n in range(len(pin)):
        assert np.array_equal(outs2[n].numpy(), ref[n]), n
    with pytest.raises(F.FeplbError):
        case.ctx.host_wait(F.HOST_SLOTS)
    case.close()


# ----------------------------------------------------------------------------- Phase-2 weight copies

@pytest.mark.parametrize("name,kw", [("cfg1", {}), ("cfg2", {}), ("cfg4", {"split": 1})])
def test_phase2_weight_copies_leave_the_output_unchanged(name, kw):
    """With phase2_copy the weights of migrated experts really travel to a receive buffer and the
    dynamic GEMM reads them there; the layer output must be bit-identical to the relabel-only path
    (Section 2.2: same expert, identical weights)."""
    torch = _torch()
    w = W.get_workload(name)
    if name != "cfg1":
        w = w.with_(T=1024)
    weights = W.gen_weights(w)
    base = DeviceCase(w, mb=0, weights=weights, **kw)
    p0 = base.ctx.moe_forward(base.d_x, base.d_ids, base.d_gates, base.d_w1, base.d_w3, base.d_w2, base.buf)
    base.ctx.check_status()
    out0 = F.bf16_bits(base.buf.out).copy()
    case = DeviceCase(w, mb=0, weights=weights, phase2_copy=1, **kw)
    case.ctx.set_timeline(True)
    p1 = case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    case.ctx.check_status()
    assert p1.moves == p0.moves and p1.groups == p0.groups and len(p1.moves) >= 1
    assert np.array_equal(F.bf16_bits(case.buf.out), out0)
    tl = case.ctx.get_timeline()
    moved_rows = sum(m[3] for m in p1.moves)
    assert tl["phase2_copy_bytes"] == 3 * w.d * w.f * 2 * len(p1.moves) + moved_rows * w.d * 2     # weights and rows
    assert tl["dev_counts_to_copies_done_us"] > 0

    # the kernel reads a migrated piece's weights from its receive slot, not from the home arrays:
    # recompute one moved group with ZERO home weights and the slot label -> same rows of y_perm
    e, src, dst, rows = p1.moves[0]
    slot = dst * case.cfg.max_num_dyn + 0                          # first move into dst takes its first slot
    assert all(m[2] != dst for m in p1.moves[:0])
    grp = [g for g in p1.groups if g[0] == e and g[3] == dst][0]
    y_ref = case.buf.y_perm[grp[1]: grp[1] + grp[2]].clone()
    zero1 = torch.zeros_like(case.d_w1)
    zero2 = torch.zeros_like(case.d_w2)
    case.buf.y_perm[grp[1]: grp[1] + grp[2]] = 7.0
    d_groups = upload_groups([(e, grp[1], grp[2], dst, 2 + slot)])
    case.ctx.expert_ffn(case.buf.x_perm, zero1, zero1, zero2, d_groups, 1, case.buf.h_scratch, case.buf.y_perm)
    case.ctx.check_status()
    assert torch.equal(case.buf.y_perm[grp[1]: grp[1] + grp[2]].view(torch.int16), y_ref.view(torch.int16))
    d_groups = upload_groups([(e, grp[1], grp[2], dst, 1)])        # labelled "home weights": zeros in, zeros out
    case.ctx.expert_ffn(case.buf.x_perm, zero1, zero1, zero2, d_groups, 1, case.buf.h_scratch, case.buf.y_perm)
    torch.cuda.synchronize()
    assert not case.buf.y_perm[grp[1]: grp[1] + grp[2]].float().abs().max().item()
    # ... and the piece's ROWS from the receive region of the rows, not from the permuted buffer: with the
    # piece's rows of x_perm zeroed the slot label still gives the same y, the home label gives zeros
    case.buf.x_perm[grp[1]: grp[1] + grp[2]] = 0
    d_groups = upload_groups([(e, grp[1], grp[2], dst, 2 + slot)])
    case.ctx.expert_ffn(case.buf.x_perm, case.d_w1, case.d_w3, case.d_w2, d_groups, 1, case.buf.h_scratch, case.buf.y_perm)
    case.ctx.check_status()
    assert torch.equal(case.buf.y_perm[grp[1]: grp[1] + grp[2]].view(torch.int16), y_ref.view(torch.int16))
    d_groups = upload_groups([(e, grp[1], grp[2], dst, 1)])
    case.ctx.expert_ffn(case.buf.x_perm, case.d_w1, case.d_w3, case.d_w2, d_groups, 1, case.buf.h_scratch, case.buf.y_perm)
    torch.cuda.synchronize()
    assert not case.buf.y_perm[grp[1]: grp[1] + grp[2]].float().abs().max().item()
    # a slot beyond the receive buffer is reported, not dereferenced
    d_groups = upload_groups([(e, grp[1], grp[2], dst, 2 + 10 ** 6)])
    case.ctx.expert_ffn(case.buf.x_perm, zero1, zero1, zero2, d_groups, 1, case.buf.h_scratch, case.buf.y_perm)
    with pytest.raises(F.FeplbError):
        case.ctx.check_status()
    base.close()
    case.close()


# ----------------------------------------------------------------------------- bounded waits, no GPU hang

def test_device_wait_gives_up_and_reports():
    """A device-side wait on a barrier that nothing completes ends after its limit with a status
    bit and a normal kernel return; the context keeps working afterwards."""
    case = DeviceCase(W.get_workload("cfg1"))
    case.ctx.selftest_bounded_wait(limit_us=3000)
    case.ctx.check_status()                                            # clean again
    _check_forward(case)
    case.close()


def test_planner_times_out_when_the_counts_do_not_arrive_and_recovers():
    """The counts are withheld by keeping the stream busy with other work; the planner's bounded
    wait expires (FEPLB_E_TIMEOUT), nothing hangs, and the next forward succeeds."""
    torch = _torch()
    case = DeviceCase(W.get_workload("cfg1"))
    case.ctx.set_planner_timeout(5)                                    # 5 ms
    a = torch.randn(8192, 8192, device="cuda", dtype=torch.bfloat16)
    for _ in range(60):                                                # ~60 x 0.8 ms of matmuls ahead of the layer
        a @ a
    with pytest.raises(F.FeplbError) as ei:
        case.ctx.moe_forward(case.d_x, case.d_ids, case.d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    assert ei.value.code == F.E_TIMEOUT
    torch.cuda.synchronize()
    case.ctx.set_planner_timeout(2000)
    case.ctx.check_status()
    _check_forward(case)
    case.close()


# ----------------------------------------------------------------------------- router top-k

@pytest.mark.parametrize("T,E,K", [(1, 8, 2), (300, 8, 8), (1000, 64, 6), (513, 128, 8), (64, 1024, 32), (77, 48, 1)])
def test_route_topk_parity(T, E, K):
    """ids bit-exact (descending logit, ties to the lower id), gates within fp32 rounding of the
    fp64 softmax over the selected logits."""
    torch = _torch()
    rng = np.random.default_rng(T + E + K)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    if T > 2:
        logits[1, :] = 0.5                                             # all tied
        logits[2, E // 2] = logits[2, 0] = logits[2].max() + 1.0       # a tie at the top
    w = _tiny(T, K, E, 1)
    ctx = F.Context(F.config_from_workload(w))
    ids = torch.zeros(T, K, dtype=torch.int32, device="cuda")
    gates = torch.zeros(T, K, dtype=torch.float32, device="cuda")
    ctx.route_topk(torch.from_numpy(logits).cuda(), ids, gates)
    ctx.check_status()
    ref_ids, ref_gates = O.route_topk(logits, K)
    assert np.array_equal(ids.cpu().numpy(), ref_ids)
    assert np.allclose(gates.cpu().numpy(), ref_gates, rtol=2e-6, atol=1e-7)
    ctx.close()


def test_router_feeds_the_layer():
    """logits -> feplb_route_topk -> feplb_moe_forward equals the oracle run from the same logits."""
    torch = _torch()
    w = W.get_workload("cfg1")
    rng = np.random.default_rng(3)
    logits = (rng.standard_normal((w.T, w.E)) * 2).astype(np.float32)
    case = DeviceCase(w)
    d_ids = torch.zeros(w.T, w.K, dtype=torch.int32, device="cuda")
    d_gates = torch.zeros(w.T, w.K, dtype=torch.float32, device="cuda")
    case.ctx.route_topk(torch.from_numpy(logits).cuda(), d_ids, d_gates)
    case.ctx.moe_forward(case.d_x, d_ids, d_gates, case.d_w1, case.d_w3, case.d_w2, case.buf)
    case.ctx.check_status()
    ids, gates = O.route_topk(logits, w.K)
    ref = O.moe_layer(case.x, ids, gates, case.w1, case.w3, case.w2, w.E)
    assert_close(W.bf16_bits_to_f64(F.bf16_bits(case.buf.out)), ref, "router + layer")
    case.close()
