"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, and
its host-only steps (plan, dynamic-expert selection, sizing, argument checks) agree bit-exactly
with the oracle.  No compute call touches a GPU here."""
import ctypes as C
import os
import re

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import feplb_oracle as O
from paper_2604_19654_b200 import build as B
from paper_2604_19654_b200 import feplb as F
from paper_2604_19654_b200 import workloads as W

from golden_utils import load_plan_cases

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    B.build()


def _declared_symbols():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names += re.findall(r"\b(feplb_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert len(names) >= 20 and "feplb_expert_ffn" in names
    L = C.CDLL(F.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert F.lib().feplb_version() >= 100
    assert F.lib().feplb_strerror(F.E_TIMEOUT) == b"timed out"


def test_config_validation_and_s_pad():
    cfg = F.make_config(T=256, K=2, E=8, R=2, d=128, f=64)
    assert F.s_pad(cfg) == 512
    cfg128 = F.make_config(T=256, K=2, E=8, R=2, d=128, f=64, row_align=128)
    assert F.s_pad(cfg128) == 512 + 8 * 127
    for bad in (dict(E=7), dict(d=100), dict(f=32), dict(K=0), dict(K=33), dict(row_align=64), dict(R=3),
                dict(ranks_per_domain=3), dict(policy=7), dict(split_granule=0)):
        kw = dict(T=256, K=2, E=8, R=2, d=128, f=64)
        kw.update(bad)
        c = F.make_config(**kw)
        assert F.s_pad(c) == 0
        with pytest.raises(F.FeplbError):
            F.plan(c, np.zeros(c.E, np.int32), np.zeros(c.E, np.uint8))


def test_create_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(F.FeplbError):
        F.Context(F.make_config(T=256, K=2, E=8, R=2, d=128, f=64))


def _same_plan(cfg, counts, mask, A=1):
    p = F.plan(cfg, counts, mask)
    o = O.plan(counts, mask, cfg.R, tau=cfg.tau, max_num_dyn=cfg.max_num_dyn,
               ranks_per_domain=cfg.ranks_per_domain, policy=cfg.policy, split=cfg.split,
               split_granule=cfg.split_granule, row_align=A)
    assert p.moves == [tuple(int(v) for v in m) for m in o["moves"]]
    assert p.groups == [tuple(int(v) for v in g) for g in o["groups"]]
    assert np.array_equal(p.load_before, o["load_before"])
    assert np.array_equal(p.load_after, o["load_after"])
    return p


@settings(max_examples=400, deadline=None)
@given(st.sampled_from([1, 2, 3, 4, 8, 16]), st.integers(1, 8), st.integers(0, 2 ** 31),
       st.sampled_from([0, 1, 5, 64]), st.integers(0, 8), st.sampled_from([0, 1]), st.sampled_from([0, 1]),
       st.sampled_from([1, 16, 128]), st.booleans(), st.sampled_from([1, 128]))
def test_plan_matches_oracle_bit_exact(R, L, seed, tau, mnd, policy, split, g, dom, A):
    rng = np.random.default_rng(seed)
    E = R * L
    scale = int(rng.choice([3, 50, 1500]))
    counts = (rng.dirichlet(np.full(E, 0.3)) * scale * E).astype(np.int32)
    mask = (rng.random(E) < 0.6).astype(np.uint8)
    D = 2 if (dom and R % 2 == 0) else 0
    cfg = F.make_config(T=1, K=1, E=E, R=R, d=128, f=64, max_num_dyn=mnd, tau=tau, ranks_per_domain=D,
                        policy=policy, split=split, split_granule=g, row_align=A)
    _same_plan(cfg, counts, mask, A)


@pytest.mark.parametrize("c", load_plan_cases(), ids=lambda c: c["case"])
def test_c_planner_against_the_handworked_plans(c):
    """feplb_plan (the library's C++ planner) against the hand-worked file itself, not through the
    oracle: the two planners follow the same reading, so agreement between them proves nothing
    about branches both could misread."""
    R, L = int(c["R"]), int(c["L"])
    cfg = F.make_config(T=1, K=1, E=R * L, R=R, d=128, f=64, max_num_dyn=int(c["max_num_dyn"]), tau=int(c["tau"]),
                        ranks_per_domain=int(c["domain"]),
                        policy=F.POLICY_LITERAL if c["policy"] == "literal" else F.POLICY_FIRST_FIT,
                        split=int(c["split"]), split_granule=int(c["g"]))
    p = F.plan(cfg, np.array(c["counts_i"], np.int32), np.array(c["mask_i"], np.uint8))
    assert p.moves == c["moves_t"]
    assert p.load_before.tolist() == c["before_i"] and p.load_after.tolist() == c["after_i"]
    # the group table follows from the moves: pieces from the front of the segment, then the rest
    off, exp = 0, []
    for e, cnt in enumerate(c["counts_i"]):
        pos, left = off, cnt
        for (me, _s, dst, rows) in c["moves_t"]:
            if me == e:
                exp.append((e, pos, rows, dst, c["mask_i"][e]))
                pos, left = pos + rows, left - rows
        if left > 0:
            exp.append((e, pos, left, e // L, c["mask_i"][e]))
        off += cnt
    assert p.groups == exp


def test_plan_matches_oracle_on_workloads():
    for name in ("cfg1", "cfg2", "cfg3", "cfg3-smooth", "cfg4"):
        w = W.get_workload(name)
        for mb in range(min(3, w.n_microbatches)):
            ids, _ = W.gen_routing(w, mb)
            counts, _ = O.route_hist(ids, w.E, w.R)
            mask = O.select_dynamic(counts, w.E, w.R, w.dyn)
            assert np.array_equal(F.select_dynamic(counts, w.E, w.R, w.dyn), mask)
            for split in (0, 1):
                for policy in (0, 1):
                    cfg = F.config_from_workload(w, split=split, policy=policy)
                    _same_plan(cfg, counts.astype(np.int32), mask)


@settings(max_examples=100, deadline=None)
@given(st.sampled_from([1, 2, 4]), st.integers(1, 9), st.integers(0, 10), st.integers(0, 2 ** 31))
def test_select_dynamic_matches_oracle(R, L, dyn, seed):
    rng = np.random.default_rng(seed)
    score = rng.integers(0, 6, size=R * L)                     # many ties
    assert np.array_equal(F.select_dynamic(score, R * L, R, dyn), O.select_dynamic(score, R * L, R, dyn))


@settings(max_examples=150, deadline=None)
@given(st.sampled_from([1, 2, 3, 4, 8]), st.integers(1, 6), st.integers(0, 2 ** 31), st.integers(0, 4), st.sampled_from([0, 1]))
def test_ep_schedule_matches_the_oracle_row_by_row_count(R, L, seed, mnd, split):
    """feplb_ep_schedule (interval arithmetic on the plan's pieces) against the oracle's ep_exchange,
    which follows every row: all six send/receive vectors of every rank, the plan and the weight copies."""
    rng = np.random.default_rng(seed)
    E = R * L
    cbs = (rng.dirichlet(np.full(E, 0.4), size=R) * rng.integers(0, 600, size=(R, 1))).astype(np.int32)
    mask = (rng.random(E) < 0.7).astype(np.uint8)
    cfg = F.make_config(T=1, K=1, E=E, R=R, d=128, f=64, max_num_dyn=mnd, tau=int(rng.choice([0, 8])), split=split, split_granule=16)
    counts = cbs.sum(0)
    op = O.plan(counts, mask, R, tau=cfg.tau, max_num_dyn=mnd, split=split, split_granule=16)
    p1, p2, comb, copies = O.ep_exchange(cbs, op, mnd)
    for rank in range(R):
        s = F.ep_schedule(cfg, cbs, mask, rank)
        assert s["plan"].moves == [tuple(int(v) for v in m) for m in op["moves"]]
        assert s["plan"].groups == [tuple(int(v) for v in g) for g in op["groups"]]
        assert np.array_equal(s["p1_send"], p1[rank]) and np.array_equal(s["p1_recv"], p1[:, rank])
        assert np.array_equal(s["p2_send"], p2[rank]) and np.array_equal(s["p2_recv"], p2[:, rank])
        assert np.array_equal(s["comb_send"], comb[rank]) and np.array_equal(s["comb_recv"], comb[:, rank])
        assert [c[:5] for c in s["copies"]] == copies
        assert all(c[5] == 3 * 128 * 64 * 2 for c in s["copies"])


def test_plan_capacity_error():
    cfg = F.make_config(T=1, K=1, E=4, R=2, d=128, f=64, max_num_dyn=2, tau=1)
    p = F.Plan(cfg)
    p.c.cap_groups = 1
    cnt = np.array([50, 5, 1, 1], np.int32)
    msk = np.ones(4, np.uint8)
    rc = F.lib().feplb_plan(C.byref(cfg), cnt.ctypes.data_as(C.POINTER(C.c_int32)),
                            msk.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(p.c))
    assert rc == F.E_NOMEM


@settings(max_examples=100, deadline=None)
@given(st.sampled_from([(1, 4), (2, 2), (2, 8), (4, 4), (8, 16)]), st.integers(0, 2 ** 31), st.booleans())
def test_place_experts_and_ema_match_oracle(shape, seed, ties):
    R, L = shape
    rng = np.random.default_rng(seed)
    load = rng.integers(0, 5 if ties else 10 ** 6, size=R * L).astype(np.float64)
    assert np.array_equal(F.place_experts(load, R), O.place_experts(load, R))
    ema = rng.random(R * L)
    counts = rng.integers(0, 1000, size=R * L)
    ref = O.ema_update(ema, counts, 0.9)
    assert np.array_equal(F.ema_update(ema.copy(), counts, 0.9), ref)


def test_placement_lowers_the_straggler_of_drifting_routing():
    """Macro level + micro level together on a synthetic drift: popularity = persistent part +
    per-micro-batch noise.  Placing experts from the EMA of past counts lowers the unbalanced
    straggler, and the per-micro-batch plan lowers it further."""
    w = W.get_workload("cfg3")
    rng = np.random.default_rng(4)
    persistent = rng.dirichlet(np.full(w.E, 0.3))
    ema = np.zeros(w.E)
    def counts_of(mb):
        p = 0.7 * persistent + 0.3 * np.random.default_rng(100 + mb).dirichlet(np.full(w.E, 0.3))
        return np.random.default_rng(200 + mb).multinomial(w.S, p).astype(np.int32)
    for mb in range(20):
        F.ema_update(ema, counts_of(mb), 0.9)
    pos = F.place_experts(ema, w.R)
    inv = np.argsort(pos)                                       # expert sitting at each new position
    before, placed, planned = [], [], []
    for mb in range(20, 28):
        c = counts_of(mb)
        cp = c[inv]                                             # counts in the new expert order
        before.append(O.straggler_ratio(c.reshape(w.R, w.L).sum(1)))
        placed.append(O.straggler_ratio(cp.reshape(w.R, w.L).sum(1)))
        p = F.plan(F.config_from_workload(w), cp, F.select_dynamic(cp, w.E, w.R, w.dyn))
        planned.append(O.straggler_ratio(p.load_after))
    assert np.mean(placed) < np.mean(before) and np.mean(planned) < np.mean(placed)
    assert np.mean(planned) < 1.1
