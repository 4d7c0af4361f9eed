"""Pins of the CPU oracle against things other than itself: library routines, closed forms,
brute force, invariants, hand-worked vectors and the numbers the paper prints."""
import itertools
import math
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import feplb_oracle as O
from paper_2604_19654_b200 import workloads as W

from golden_utils import load_plan_cases

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kv(path):
    out = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out


# ----------------------------------------------------------------------------- paper numbers

def test_paper_expert_size_and_buffer():
    g = _kv(os.path.join(GOLDEN, "paper_numbers.txt"))
    w = W.get_workload("cfg3")
    expert_bytes = 3 * w.d * w.f * 2                       # W1, W3, W2 in bf16
    assert expert_bytes == int(g["expert_mib"]) * 2 ** 20   # Section 2.3: 72 MiB per expert
    assert int(g["max_num_dyn"]) * int(g["expert_mib"]) == int(g["buffer_mib"])
    assert int(g["buffer_mib"]) * 2 ** 20 / (int(g["hbm_gb"]) * 2 ** 30) < float(g["buffer_frac_below"]) + 1e-4
    assert w.E == int(g["experts"]) and w.E // 8 == int(g["experts_per_device_ep8"])
    assert w.L - w.dyn == int(g["static_per_device_dyn4"])


def test_paper_straggler_tables_arithmetic():
    """token_straggler is max - mean; the reductions printed in Tables 3 and 4 follow from the
    printed before/after values."""
    g = _kv(os.path.join(GOLDEN, "paper_numbers.txt"))
    for key in ("table3", "table4"):
        for row in g[key].split(";"):
            _, before, after, pct = row.split()
            assert round(100 * (1 - float(after) / float(before))) == int(pct)
    # a load vector whose max - mean is the Table 3 value: mean 10000, max 10000 + 6666
    load = [10000 + 6666, 10000 - 6666 / 7.0] + [10000 - 6666 / 7.0] * 6
    assert O.token_straggler(load) == pytest.approx(6666)
    assert O.straggler_ratio(load) == pytest.approx(1.6666)


# ----------------------------------------------------------------------------- histogram

@settings(max_examples=50, deadline=None)
@given(st.integers(1, 6), st.integers(1, 64), st.integers(1, 4), st.integers(0, 2 ** 31))
def test_hist_matches_bincount(r, t, k, seed):
    E = r * 3
    rng = np.random.default_rng(seed)
    ids = rng.integers(0, E, size=(t, k)).astype(np.int32)
    counts, load = O.route_hist(ids, E, r)
    assert np.array_equal(counts, np.bincount(ids.ravel(), minlength=E))
    assert counts.sum() == t * k == load.sum()               # token conservation
    assert np.array_equal(load, counts.reshape(r, 3).sum(1))


def test_hist_rejects_out_of_range():
    with pytest.raises(ValueError):
        O.route_hist(np.array([[0, 8]]), 8, 2)
    with pytest.raises(ValueError):
        O.route_hist(np.array([[-1, 0]]), 8, 2)


# ----------------------------------------------------------------------------- permutation

@settings(max_examples=50, deadline=None)
@given(st.integers(1, 12), st.integers(0, 80), st.integers(1, 4), st.sampled_from([1, 8, 128]),
       st.integers(0, 2 ** 31))
def test_permute_invariants_and_argsort(E, t, k, A, seed):
    rng = np.random.default_rng(seed)
    ids = rng.integers(0, E, size=(t, k)).astype(np.int32)
    s2r, r2t, pad_off, S_pad = O.permute(ids, E, A)
    counts = np.bincount(ids.ravel(), minlength=E)
    # every (token, k) slot placed exactly once
    flat = s2r.ravel()
    assert len(set(flat.tolist())) == t * k
    assert np.array_equal(np.sort(flat), np.flatnonzero(r2t >= 0))
    assert S_pad == sum(O.round_up(int(c), A) for c in counts)
    for s, row in enumerate(flat.tolist()):
        e = ids.ravel()[s]
        assert pad_off[e] <= row < pad_off[e] + counts[e]   # lands in its expert's segment
        assert r2t[row] == s // k
    # stability: rows of one expert appear in increasing slot order
    for e in range(E):
        rows = flat[ids.ravel() == e]
        assert np.all(np.diff(rows) == 1) if rows.size > 1 else True
    if A == 1 and t * k:
        order = np.argsort(ids.ravel(), kind="stable")       # library stable sort
        inv = np.empty_like(order)
        inv[order] = np.arange(order.size)
        assert np.array_equal(flat, inv)


def test_permute_bruteforce_tiny():
    ids = np.array([[2, 0], [0, 2], [1, 0]], np.int32)       # slots: 2 0 0 2 1 0
    s2r, r2t, pad_off, S_pad = O.permute(ids, 3, 1)
    assert s2r.ravel().tolist() == [4, 0, 1, 5, 3, 2]
    assert r2t.tolist() == [0, 1, 2, 2, 0, 1]
    assert pad_off.tolist() == [0, 3, 4] and S_pad == 6
    s2r, r2t, pad_off, S_pad = O.permute(ids, 3, 4)
    assert pad_off.tolist() == [0, 4, 8] and S_pad == 12
    assert s2r.ravel().tolist() == [8, 0, 1, 9, 4, 2]
    assert r2t.tolist() == [0, 1, 2, -1, 2, -1, -1, -1, 0, 1, -1, -1]


def test_gather_rows_roundtrip():
    rng = np.random.default_rng(0)
    x = rng.integers(0, 2 ** 16, size=(5, 7)).astype(np.uint16)
    ids = rng.integers(0, 4, size=(5, 3)).astype(np.int32)
    s2r, r2t, _, S_pad = O.permute(ids, 4, 8)
    xp = O.gather_rows(x, r2t)
    assert xp.shape == (S_pad, 7)
    for t in range(5):
        for k in range(3):
            assert np.array_equal(xp[s2r[t, k]], x[t])
    assert not xp[r2t < 0].any()


# ----------------------------------------------------------------------------- plan

@pytest.mark.parametrize("c", load_plan_cases(), ids=lambda c: c["case"])
def test_plan_handworked(c):
    R, L = int(c["R"]), int(c["L"])
    p = O.plan(c["counts_i"], c["mask_i"], R, tau=int(c["tau"]), max_num_dyn=int(c["max_num_dyn"]),
               ranks_per_domain=int(c["domain"]),
               policy=O.POLICY_LITERAL if c["policy"] == "literal" else O.POLICY_FIRST_FIT,
               split=int(c["split"]), split_granule=int(c["g"]))
    assert p["moves"] == c["moves_t"]
    assert p["load_before"].tolist() == c["before_i"]
    assert p["load_after"].tolist() == c["after_i"]
    assert len(c["counts_i"]) == R * L


def _check_plan_invariants(counts, mask, R, p, tau, max_num_dyn, D, split, g, A=1):
    E = len(counts)
    L = E // R
    D = D or R
    counts = np.asarray(counts)
    before = counts.reshape(R, L).sum(1)
    assert np.array_equal(p["load_before"], before)
    assert p["load_after"].sum() == before.sum() == counts.sum()      # conservation
    for dom in range(R // D):
        sl = slice(dom * D, (dom + 1) * D)
        assert p["load_after"][sl].sum() == before[sl].sum()           # nothing crosses a domain
        assert p["load_after"][sl].max() <= before[sl].max()           # max load never rises
    recv = np.zeros(R, int)
    seen_pairs = set()
    moved_rows = np.zeros(E, int)
    for (e, src, dst, rows) in p["moves"]:
        assert mask[e] and src == e // L and dst != src
        assert src // D == dst // D
        assert rows >= max(tau, 1)
        recv[dst] += 1
        assert (e, dst) not in seen_pairs
        seen_pairs.add((e, dst))
        moved_rows[e] += rows
        if not split:
            assert rows == counts[e]
        elif moved_rows[e] < counts[e]:
            assert rows % g == 0
    assert np.all(moved_rows <= counts)
    assert np.all(recv <= max_num_dyn)
    if not split:
        assert len({m[0] for m in p["moves"]}) == len(p["moves"])     # an expert moves at most once
    # groups tile each expert's segment exactly once, in expert order
    pad_off, _ = O.segment_offsets(counts, A)
    per_e = np.zeros(E, int)
    last_e = -1
    nxt = {}
    for (e, row_start, rows, exec_rank, is_dyn) in p["groups"]:
        assert e >= last_e and rows > 0 and is_dyn == int(bool(mask[e]))
        last_e = e
        assert row_start == nxt.get(e, int(pad_off[e]))
        nxt[e] = row_start + rows
        per_e[e] += rows
        if not mask[e]:
            assert exec_rank == e // L
    assert np.array_equal(per_e, counts)
    assert np.array_equal(p["exec_rows"].sum(0), counts)
    assert np.array_equal(p["exec_rows"].sum(1), p["load_after"])
    # replaying the moves reproduces load_after, and in whole mode every accepted move had rows < gap
    load = before.astype(np.int64).copy()
    for (e, src, dst, rows) in p["moves"]:
        if not split:
            assert rows < load[src] - load[dst]
        load[src] -= rows
        load[dst] += rows
    assert np.array_equal(load, p["load_after"])


plan_inputs = st.tuples(
    st.sampled_from([1, 2, 3, 4, 8]), st.integers(1, 6), st.integers(0, 2 ** 31),
    st.sampled_from([0, 1, 5, 40]), st.integers(0, 4), st.sampled_from([0, 1]),
    st.sampled_from([0, 1]), st.sampled_from([1, 16, 128]), st.booleans())


@settings(max_examples=300, deadline=None)
@given(plan_inputs)
def test_plan_invariants(args):
    R, L, seed, tau, mnd, policy, split, g, use_dom = args
    rng = np.random.default_rng(seed)
    E = R * L
    scale = rng.choice([4, 60, 2000])
    counts = (rng.dirichlet(np.full(E, 0.3)) * scale * E).astype(np.int64)
    mask = (rng.random(E) < 0.6).astype(np.uint8)
    D = 0
    if use_dom and R % 2 == 0:
        D = 2
    kw = dict(tau=tau, max_num_dyn=mnd, ranks_per_domain=D, policy=policy, split=split, split_granule=g)
    p = O.plan(counts, mask, R, **kw)
    _check_plan_invariants(counts, mask, R, p, tau, mnd, D, split, g)
    q = O.plan(counts.copy(), mask.copy(), R, **kw)                  # pure function
    assert p["moves"] == q["moves"] and p["groups"] == q["groups"]
    if split:
        M = -(-int(counts.sum()) // R) if not D else None
        if M is not None:
            for r in range(R):      # no rank is pushed across the mean: receivers stay <= M, donors >= M
                if p["load_after"][r] > p["load_before"][r]:
                    assert p["load_after"][r] <= M
                if p["load_after"][r] < p["load_before"][r]:
                    assert p["load_after"][r] >= M


def test_plan_closed_form_special_cases():
    counts = np.array([50, 10, 3, 7, 100, 20, 1, 9])
    full = np.ones(8, np.uint8)
    # R = 1, empty mask, tau above every count, no receive slots: nothing can move
    for kw, R, mask in [({}, 1, full), ({}, 2, np.zeros(8, np.uint8)), ({"tau": 101}, 2, full),
                        ({"max_num_dyn": 0}, 2, full)]:
        p = O.plan(counts, mask, R, **kw)
        assert p["moves"] == [] and np.array_equal(p["load_after"], p["load_before"])
        assert [g_[0] for g_ in p["groups"]] == list(range(8))
    # all counts equal: loads equal, gap 0
    p = O.plan(np.full(8, 5), full, 4)
    assert p["moves"] == []


def test_plan_one_hot_expert_exact():
    # loads [100, 10, 10]; hot expert 0 has 60 rows < gap 90 -> one move to rank 1 (lowest id of the two minima)
    counts = np.array([60, 40, 10, 0, 10, 0])
    mask = np.array([1, 0, 0, 0, 0, 0], np.uint8)
    p = O.plan(counts, mask, 3, tau=1)
    assert p["moves"] == [(0, 0, 1, 60)]
    assert p["load_after"].tolist() == [40, 70, 10]
    # a hot expert at least as large as the gap stays (moving it cannot lower the maximum)
    counts = np.array([95, 5, 10, 0, 10, 0])
    p = O.plan(counts, mask, 3, tau=1)
    assert p["moves"] == []


def _brute_force_best_max(counts, mask, R, max_num_dyn):
    """Smallest achievable max load over all placements of whole dynamic experts."""
    E = len(counts)
    L = E // R
    dyn = [e for e in range(E) if mask[e]]
    base = [0] * R
    for e in range(E):
        if not mask[e]:
            base[e // L] += counts[e]
    best = None
    for assign in itertools.product(range(R), repeat=len(dyn)):
        recv = [0] * R
        load = list(base)
        for e, r in zip(dyn, assign):
            load[r] += counts[e]
            if r != e // L:
                recv[r] += 1
        if max(recv) > max_num_dyn:
            continue
        m = max(load)
        best = m if best is None else min(best, m)
    return best


@settings(max_examples=60, deadline=None)
@given(st.sampled_from([(2, 2), (2, 3), (3, 2), (2, 4)]), st.integers(0, 2 ** 31), st.sampled_from([0, 1]))
def test_plan_bruteforce_bound(shape, seed, policy):
    R, L = shape
    rng = np.random.default_rng(seed)
    E = R * L
    counts = rng.integers(0, 50, size=E)
    mask = (rng.random(E) < 0.7).astype(np.uint8)
    p = O.plan(counts, mask, R, tau=1, max_num_dyn=3, policy=policy)
    best = _brute_force_best_max(counts.tolist(), mask.tolist(), R, 3)
    assert best <= p["load_after"].max() <= p["load_before"].max()


def test_select_dynamic():
    score = [5, 9, 9, 1, 0, 0, 3, 2]
    m = O.select_dynamic(score, 8, 2, 2)
    assert m.tolist() == [0, 1, 1, 0, 0, 0, 1, 1]          # rank 0: e1, e2; rank 1: e6 (3), e7 (2)
    assert O.select_dynamic([1, 1, 1, 1], 4, 1, 2).tolist() == [1, 1, 0, 0]   # ties -> lower id
    assert O.select_dynamic(score, 8, 2, 0).sum() == 0
    assert O.select_dynamic(score, 8, 2, 9).sum() == 8


def test_plan_improves_every_workload():
    for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
        w = W.get_workload(name)
        ids, _ = W.gen_routing(w, 0)
        counts, load = O.route_hist(ids, w.E, w.R)
        mask = O.select_dynamic(counts, w.E, w.R, w.dyn)
        for split in (0, 1):
            g = 16 if name == "cfg1" else 128
            p = O.plan(counts, mask, w.R, w.tau, w.max_num_dyn, split=split, split_granule=g)
            assert O.straggler_ratio(p["load_after"]) < O.straggler_ratio(load)
            _check_plan_invariants(counts, mask, w.R, p, w.tau, w.max_num_dyn, 0, split, g)


# ----------------------------------------------------------------------------- expert FFN

def _bits(a):
    return W.f32_to_bf16_bits(np.asarray(a, np.float32))


def test_silu_closed_forms():
    z = np.array([-3.0, -1.0, 0.0, 0.5, 2.0, 30.0])
    s = O.silu(z)
    assert s[2] == 0.0
    assert np.allclose(s - O.silu(-z), z)                    # silu(z) - silu(-z) = z
    assert s[1] == pytest.approx(-1.0 / (1.0 + math.e))
    assert s[5] == pytest.approx(30.0, rel=1e-12)
    assert np.allclose(s, z * 0.5 * (1.0 + np.tanh(z / 2.0)))   # sigmoid written via tanh


def test_ffn_against_scalar_loops():
    rng = np.random.default_rng(3)
    E, d, f, n = 3, 5, 4, 7                                   # non-square on purpose
    x = _bits(rng.standard_normal((n, d)))
    w1 = _bits(rng.standard_normal((E, f, d)))
    w3 = _bits(rng.standard_normal((E, f, d)))
    w2 = _bits(rng.standard_normal((E, d, f)))
    re = np.array([2, 0, 1, 1, -1, 0, 2])
    y = O.expert_ffn(x, re, w1, w3, w2)
    X, W1, W3, W2 = (W.bf16_bits_to_f64(a) for a in (x, w1, w3, w2))
    for i in range(n):
        e = re[i]
        if e < 0:
            assert not y[i].any()
            continue
        h = []
        for c in range(f):
            a = sum(X[i, j] * W1[e, c, j] for j in range(d))
            b = sum(X[i, j] * W3[e, c, j] for j in range(d))
            h.append(a / (1.0 + math.exp(-a)) * b)
        for o in range(d):
            ref = sum(h[c] * W2[e, o, c] for c in range(f))
            assert y[i, o] == pytest.approx(ref, rel=1e-12, abs=1e-15)


def test_ffn_one_hot_rows_and_linearity():
    rng = np.random.default_rng(4)
    E, d, f = 2, 6, 3
    w1 = _bits(rng.standard_normal((E, f, d)))
    w3 = _bits(rng.standard_normal((E, f, d)))
    w2 = _bits(rng.standard_normal((E, d, f)))
    W1, W3, W2 = (W.bf16_bits_to_f64(a) for a in (w1, w3, w2))
    x = _bits(np.eye(d))                                       # row i = unit vector i
    for e in range(E):
        y = O.expert_ffn(x, np.full(d, e), w1, w3, w2)
        for i in range(d):
            h = O.silu(W1[e, :, i]) * W3[e, :, i]              # x W1 picks column i of the d x f matrix
            assert np.allclose(y[i], W2[e] @ h, rtol=1e-12)
    # doubling W2 doubles y; W3 = 0 gives 0
    xr = _bits(rng.standard_normal((4, d)))
    y1 = O.expert_ffn(xr, np.zeros(4, int), w1, w3, w2)
    y2 = O.expert_ffn(xr, np.zeros(4, int), w1, w3, _bits(2 * W.bf16_bits_to_f32(w2)))
    assert np.allclose(y2, 2 * y1, rtol=1e-12)
    assert not O.expert_ffn(xr, np.zeros(4, int), w1, np.zeros_like(w3), w2).any()


def _rne_bf16_scalar(v: float) -> float:
    """Round one double to bf16 the way the hidden activation is stored: first to float32 (the
    accumulator's type), then to the nearest bf16, ties to the even mantissa -- written with
    integer arithmetic on the float32 bit pattern, one value at a time."""
    import struct
    (u,) = struct.unpack("<I", struct.pack("<f", v))          # struct rounds the double to float32
    keep, drop = u >> 16, u & 0xFFFF
    if drop > 0x8000 or (drop == 0x8000 and (keep & 1)):
        keep += 1
    (out,) = struct.unpack("<f", struct.pack("<I", (keep << 16) & 0xFFFFFFFF))
    return float(out)


def test_bf16_rounding_of_the_hidden_activation_is_nearest_even():
    """Pins oracle._round_f64_to_bf16 (the round_h_bf16 mode of expert_ffn) on values whose bf16
    neighbours are known by hand: bf16 keeps 8 significant bits, so the spacing at 1.0 is 2^-7."""
    r = lambda v: float(O._round_f64_to_bf16(np.array([v], np.float64))[0])
    assert r(1.0) == 1.0
    assert r(1.0 + 2.0 ** -8) == 1.0                            # tie -> even mantissa (down)
    assert r(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6             # tie -> even mantissa (up)
    assert r(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7    # just above the tie
    assert r(1.0 + 2.0 ** -8 - 2.0 ** -20) == 1.0                # just below it (truncation would also
    assert r(1.0 + 2.0 ** -7 - 2.0 ** -20) == 1.0 + 2.0 ** -7    #  give 1.0 here, but not on this line)
    assert r(-(1.0 + 3 * 2.0 ** -8)) == -(1.0 + 2.0 ** -6)       # sign-symmetric
    assert r(-(1.0 + 2.0 ** -8)) == -1.0
    assert r(2.0 ** -100 * (1.0 + 2.0 ** -8 + 2.0 ** -9)) == 2.0 ** -100 * (1.0 + 2.0 ** -7)   # small normal value
    assert r(255.5) == 256.0 and r(254.5) == 254.0 and r(0.0) == 0.0   # carry into the exponent; 254.5 ties to even
    # the value passes through float32 first, as the kernel's fp32 accumulator does: 2^-30 is below
    # float32's resolution at 1.0, so this is the tie again, not "just above" it
    assert r(1.0 + 2.0 ** -8 + 2.0 ** -30) == 1.0
    # on values that are exact in float32 it is the input generator's rounding (a separate routine)
    rng = np.random.default_rng(12)
    v32 = (rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, size=4096)).astype(np.float32)
    v32[:8] = np.float32(1.0) + np.arange(8, dtype=np.float32) * np.float32(2.0 ** -8)     # ties of both parities
    got = O._round_f64_to_bf16(v32.astype(np.float64))
    assert np.array_equal(got, W.bf16_bits_to_f64(W.f32_to_bf16_bits(v32)))
    assert np.array_equal(got, np.array([_rne_bf16_scalar(float(v)) for v in v32]))


def test_ffn_with_rounded_hidden_activation_against_scalar_loops():
    """expert_ffn(round_h_bf16=True): the hidden activation is rounded to bf16 before the second
    contraction.  Checked against scalar loops with the rounding written out per element."""
    rng = np.random.default_rng(13)
    E, d, f, n = 2, 6, 5, 6
    x = _bits(rng.standard_normal((n, d)))
    w1 = _bits(rng.standard_normal((E, f, d)))
    w3 = _bits(rng.standard_normal((E, f, d)))
    w2 = _bits(rng.standard_normal((E, d, f)))
    re = np.array([1, 0, 0, -1, 1, 0])
    y = O.expert_ffn(x, re, w1, w3, w2, round_h_bf16=True)
    y_plain = O.expert_ffn(x, re, w1, w3, w2)
    X, W1, W3, W2 = (W.bf16_bits_to_f64(a) for a in (x, w1, w3, w2))
    changed = 0
    for i in range(n):
        e = re[i]
        if e < 0:
            assert not y[i].any()
            continue
        h = []
        for c in range(f):
            a = sum(X[i, j] * W1[e, c, j] for j in range(d))
            b = sum(X[i, j] * W3[e, c, j] for j in range(d))
            h.append(_rne_bf16_scalar(a / (1.0 + math.exp(-a)) * b))
        for o in range(d):
            ref = sum(h[c] * W2[e, o, c] for c in range(f))
            assert y[i, o] == pytest.approx(ref, rel=1e-12, abs=1e-15)
            changed += y[i, o] != y_plain[i, o]
    assert changed > 0                                          # the mode really rounds something


# ----------------------------------------------------------------------------- combine, whole layer

def test_combine_scalar_loops_and_identity_roundtrip():
    rng = np.random.default_rng(5)
    T, K, d, E = 6, 3, 4, 5
    ids = rng.integers(0, E, size=(T, K)).astype(np.int32)
    s2r, r2t, _, S_pad = O.permute(ids, E, 8)
    y = rng.standard_normal((S_pad, d))
    g = rng.random((T, K)).astype(np.float32)
    out = O.combine(y, s2r, g)
    for t in range(T):
        for j in range(d):
            assert out[t, j] == pytest.approx(sum(float(g[t, k]) * y[s2r[t, k], j] for k in range(K)), rel=1e-13)
    # K = 1, gate = 1, identity "FFN": dispatch then combine returns x exactly
    ids1 = rng.integers(0, E, size=(T, 1)).astype(np.int32)
    x = _bits(rng.standard_normal((T, d)))
    s2r1, r2t1, _, _ = O.permute(ids1, E, 1)
    xp = O.gather_rows(x, r2t1)
    out1 = O.combine(W.bf16_bits_to_f64(xp), s2r1, np.ones((T, 1), np.float32))
    assert np.array_equal(out1, W.bf16_bits_to_f64(x))


def test_staged_pipeline_equals_layer_definition():
    """permute -> gather -> FFN on permuted rows -> combine equals sum_k g * FFN_e(x_t), with or
    without padding, and whatever the plan says (the plan only relabels ranks)."""
    w = W.get_workload("cfg1")
    x, ids, gates = W.gen_microbatch(w, 0)
    w1, w3, w2 = W.gen_weights(w)
    ref = O.moe_layer(x, ids, gates, w1, w3, w2, w.E)
    for A in (1, 128):
        s2r, r2t, _, S_pad = O.permute(ids, w.E, A)
        xp = O.gather_rows(x, r2t)
        re = O.row_experts(ids, s2r, S_pad)
        y = O.expert_ffn(xp, re, w1, w3, w2)
        out = O.combine(y, s2r, gates)
        assert np.allclose(out, ref, rtol=1e-12, atol=1e-18)
    sub = np.array([0, 17, 255])
    assert np.allclose(O.moe_layer(x, ids, gates, w1, w3, w2, w.E, tokens=sub), ref[sub], rtol=1e-12, atol=1e-18)


# ----------------------------------------------------------------------------- router, placement

def test_route_topk_against_library_sort_and_closed_forms():
    rng = np.random.default_rng(9)
    z = rng.standard_normal((40, 12)).astype(np.float32)
    z[3, 5] = z[3, 2]                                          # a tie: the lower id wins
    z[7, :] = 0.25                                             # all equal: ids 0..K-1, uniform gates
    ids, gates = O.route_topk(z, 4)
    order = np.argsort(-z.astype(np.float64), axis=1, kind="stable")[:, :4]   # library stable sort
    assert np.array_equal(ids, order)
    assert ids[7].tolist() == [0, 1, 2, 3] and np.allclose(gates[7], 0.25)
    assert np.allclose(gates.sum(1), 1.0) and np.all(np.diff(gates, axis=1) <= 1e-15)
    # two selected logits a > b: gate = sigmoid(a - b)
    ids2, g2 = O.route_topk(np.array([[1.0, 3.0, -2.0]]), 2)
    assert ids2.tolist() == [[1, 0]] and g2[0, 0] == pytest.approx(1.0 / (1.0 + math.exp(-2.0)))
    # K = E: plain softmax in sorted order
    ids3, g3 = O.route_topk(z[:5], 12)
    sm = np.exp(z[:5].astype(np.float64))
    sm /= sm.sum(1, keepdims=True)
    assert np.allclose(g3, np.take_along_axis(sm, ids3, axis=1))
    # the workloads' generator is this router applied to its logits: same ids, same gates
    w = W.get_workload("cfg1")
    gen_ids, gen_gates = W.gen_routing(w, 0)
    assert gen_ids.shape == (w.T, w.K) and np.allclose(gen_gates.sum(1), 1.0, atol=1e-6)


def test_place_experts_invariants_and_bruteforce():
    rng = np.random.default_rng(2)
    for R, L in ((2, 2), (2, 3), (3, 2), (4, 4)):
        load = rng.integers(1, 100, size=R * L).astype(float)
        pos = O.place_experts(load, R)
        assert sorted(pos.tolist()) == list(range(R * L))      # a permutation: every rank gets L experts
        rl = np.zeros(R)
        for e, p in enumerate(pos):
            rl[p // L] += load[e]
        if R * L <= 6:                                         # brute force: optimum over all balanced assignments
            best = min(max(sum(load[e] for e in range(R * L) if a[e] == r) for r in range(R))
                       for a in itertools.product(range(R), repeat=R * L)
                       if all(a.count(r) == L for r in range(R)))
            assert best <= rl.max() <= best * 4.0 / 3.0 + 1e-9  # the classical LPT bound
    # equal loads -> round-robin placement; one heavy expert ends up with the lightest companions
    assert O.place_experts([5, 5, 5, 5], 2).tolist() == [0, 2, 1, 3]
    pos = O.place_experts([100, 1, 2, 3], 2)
    assert pos[0] // 2 != pos[3] // 2 and pos[0] // 2 == pos[1] // 2   # 100 shares a rank with the lightest
    assert np.allclose(O.ema_update([10.0, 0.0], [0.0, 10.0], 0.9), [9.0, 1.0])


# ----------------------------------------------------------------------------- backward pass

def test_backward_against_finite_differences():
    """The oracle's gradients against central differences of its own forward definition, in fp64
    on a tiny layer (inputs chosen exactly representable in bf16 so that perturbations can be
    applied to the widened values)."""
    rng = np.random.default_rng(12)
    T, K, E, d, f = 5, 2, 3, 4, 3
    ids = np.array([rng.choice(E, size=K, replace=False) for _ in range(T)]).astype(np.int32)
    gates = rng.random((T, K)).astype(np.float32)
    xb = _bits(rng.standard_normal((T, d)))
    w1b, w3b, w2b = _bits(rng.standard_normal((E, f, d))), _bits(rng.standard_normal((E, f, d))), _bits(rng.standard_normal((E, d, f)))
    d_out = rng.standard_normal((T, d))
    dx, dg, dw1, dw3, dw2 = O.moe_layer_backward(xb, ids, gates, w1b, w3b, w2b, d_out, E)

    X, W1, W3, W2 = (W.bf16_bits_to_f64(a) for a in (xb, w1b, w3b, w2b))
    G = gates.astype(np.float64)

    def loss(X, G, W1, W3, W2):                                # scalar: <d_out, layer output>, plain fp64 definition
        tot = 0.0
        for t in range(T):
            for k in range(K):
                e = ids[t, k]
                a, b = W1[e] @ X[t], W3[e] @ X[t]
                tot += G[t, k] * float(d_out[t] @ (W2[e] @ (a / (1 + np.exp(-a)) * b)))
        return tot

    eps = 1e-6
    def fd(arr, idx, pos):
        args = [X.copy(), G.copy(), W1.copy(), W3.copy(), W2.copy()]
        args[pos][idx] += eps
        up = loss(*args)
        args[pos][idx] -= 2 * eps
        return (up - loss(*args)) / (2 * eps)

    for arr, grad, pos in ((X, dx, 0), (G, dg, 1), (W1, dw1, 2), (W3, dw3, 3), (W2, dw2, 4)):
        for idx in [tuple(rng.integers(0, n) for n in arr.shape) for _ in range(6)]:
            assert grad[idx] == pytest.approx(fd(arr, idx, pos), rel=1e-5, abs=1e-7)
    assert O.dsilu(np.array([0.0]))[0] == 0.5 and O.dsilu(np.array([40.0]))[0] == pytest.approx(1.0)


# ----------------------------------------------------------------------------- expert parallelism over real ranks

def test_ep_exchange_conservation_and_handworked_case():
    """ep_exchange against what must hold whatever the plan is, and against a case small enough to
    follow by hand."""
    # hand-worked: R = 2, L = 2.  Rank 0's tokens send 3 rows to e0, 1 to e2; rank 1's send 2 to e0, 1 to e1, 2 to e3.
    cbs = np.array([[3, 0, 1, 0], [2, 1, 0, 2]])
    counts = cbs.sum(0)                                        # [5, 1, 1, 2] -> loads [6, 3]
    p = O.plan(counts, [1, 1, 1, 1], 2, tau=1, max_num_dyn=2)
    assert p["moves"] == [(1, 0, 1, 1)]                        # gap 3: e0 (5) does not fit, e1 (1 row) moves 0 -> 1
    p1, p2, comb, copies = O.ep_exchange(cbs, p, 2)
    assert p1.tolist() == [[3, 1], [3, 2]]                     # to home: e0/e1 live on rank 0, e2/e3 on rank 1
    assert p2.tolist() == [[0, 1], [0, 0]]                     # the one row of e1 goes on from rank 0 to rank 1
    assert comb.tolist() == [[3, 2], [1, 3]]                   # rank 0 ran e0 (3 rows of rank 0, 2 of rank 1); rank 1 ran e2, e3 and e1's row
    assert copies == [(1, 0, 1, 2, 1)]                         # slot = dst * max_num_dyn + 0
    # conservation on random inputs
    rng = np.random.default_rng(31)
    for _ in range(30):
        R = int(rng.choice([2, 3, 4]))
        L = int(rng.choice([1, 2, 4]))
        cbs = rng.integers(0, 40, size=(R, R * L))
        counts = cbs.sum(0)
        mask = (rng.random(R * L) < 0.7).astype(np.uint8)
        mnd = int(rng.integers(0, 3))
        p = O.plan(counts, mask, R, tau=int(rng.choice([0, 5])), max_num_dyn=mnd)
        p1, p2, comb, copies = O.ep_exchange(cbs, p, mnd)
        assert np.array_equal(p1.sum(1), cbs.sum(1))           # every slot leaves its source once
        assert np.array_equal(p1.sum(0), counts.reshape(R, L).sum(1))      # and arrives at its expert's home
        assert np.array_equal(comb.sum(0), cbs.sum(1))         # every slot comes back to its source
        assert np.array_equal(comb.sum(1), p["load_after"])    # from the rank that executed it
        assert p2.sum() == sum(m[3] for m in p["moves"]) and not np.diag(p2).any()
        assert np.array_equal(p1.sum(0) - p2.sum(1) + p2.sum(0), p["load_after"])
        assert [c[:3] + (c[4],) for c in copies] == [tuple(m) for m in p["moves"]]
        slots = [c[3] for c in copies]
        assert len(set(slots)) == len(slots) and all(c[2] * mnd <= c[3] < (c[2] + 1) * mnd for c in copies)
