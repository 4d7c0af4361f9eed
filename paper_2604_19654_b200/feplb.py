"""Thin ctypes binding over the C ABI of ``libfeplb.so`` (see ``include/feplb.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels (or, for
the plan, in its C++ host code).  PyTorch supplies device memory and streams.  If the library is
missing the import of a symbol fails loudly -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfeplb.so")

OK, E_INVALID, E_RANGE, E_CUDA, E_NOMEM, E_TIMEOUT, E_STATE, E_DEVICE = 0, -1, -2, -3, -4, -5, -6, -7
POLICY_LITERAL, POLICY_FIRST_FIT = 0, 1
MASK_GIVEN, MASK_REACTIVE = 0, 1
FFN_ALL, FFN_STATIC, FFN_DYNAMIC = 0, 1, 2
FORM_AUTO, FORM_SINGLE, FORM_PAIR, FORM_WEIGHT_M = -1, 0, 1, 2
HOST_SLOTS = 4            # staging sets of the pipelined host-buffer forward (FEPLB_HOST_SLOTS)


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "T", "K", "E", "R", "d", "f", "dyn", "max_num_dyn", "tau", "ranks_per_domain", "policy",
        "split", "split_granule", "row_align", "mask_policy", "phase2_copy")]


class Move(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("expert", "src", "dst", "rows")]


class Group(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("expert", "row_start", "rows", "exec_rank", "is_dynamic")]


class PlanOut(C.Structure):
    _fields_ = [("n_moves", C.c_int32), ("n_groups", C.c_int32), ("cap_moves", C.c_int32),
                ("cap_groups", C.c_int32), ("moves", C.POINTER(Move)), ("groups", C.POINTER(Group)),
                ("load_before", C.POINTER(C.c_int64)), ("load_after", C.POINTER(C.c_int64))]


class Timeline(C.Structure):
    _fields_ = [(n, C.c_double) for n in (
        "host_enqueue_static_done_us", "host_counts_ready_us", "host_plan_done_us",
        "host_upload_enqueued_us", "host_join_us", "host_return_us", "plan_us",
        "dev_hist_us", "dev_dispatch_us", "dev_static_ffn_us", "dev_dynamic_ffn_us", "dev_combine_us",
        "dev_counts_to_static_start_us", "dev_counts_to_static_end_us", "dev_total_us",
        "dev_counts_to_copies_done_us", "phase2_copy_bytes",
        "dev_ffn_pass1_us", "dev_ffn_pass2_us", "dev_plan_wait_us", "ffn_launches")]


class WeightCopy(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("expert", "src", "dst", "slot", "rows")] + [("weight_bytes", C.c_int64)]


class FeplbError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {lib().feplb_strerror(code).decode()} ({code})" + (f": {detail}" if detail else ""))


_lib = None


def lib() -> C.CDLL:
    """Opens libfeplb.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2604_19654_b200.build` "
                "(the CUDA library is the only implementation; there is no fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        sig = {
            "feplb_version": (C.c_int, []),
            "feplb_strerror": (C.c_char_p, [C.c_int]),
            "feplb_create": (C.c_int, [C.POINTER(Config), C.POINTER(vp)]),
            "feplb_destroy": (C.c_int, [vp]),
            "feplb_last_error": (C.c_char_p, [vp]),
            "feplb_check_status": (C.c_int, [vp, vp]),
            "feplb_s_pad": (C.c_size_t, [C.POINTER(Config)]),
            "feplb_select_dynamic": (C.c_int, [C.POINTER(i64), i32, i32, i32, C.POINTER(C.c_uint8)]),
            "feplb_plan": (C.c_int, [C.POINTER(Config), C.POINTER(i32), C.POINTER(C.c_uint8), C.POINTER(PlanOut)]),
            "feplb_ep_schedule": (C.c_int, [C.POINTER(Config), C.POINTER(i32), C.POINTER(C.c_uint8), i32, C.POINTER(PlanOut)] +
                                  [C.POINTER(i64)] * 6 + [C.POINTER(WeightCopy), i32, C.POINTER(i32)]),
            "feplb_ema_update": (C.c_int, [C.POINTER(C.c_double), C.POINTER(i32), i32, C.c_double]),
            "feplb_place_experts": (C.c_int, [C.POINTER(C.c_double), i32, i32, C.POINTER(i32)]),
            "feplb_route_topk": (C.c_int, [vp, vp, vp, vp, vp]),
            "feplb_route_hist": (C.c_int, [vp, vp, vp, vp, vp]),
            "feplb_dispatch": (C.c_int, [vp] * 8),
            "feplb_dispatch_noalloc": (C.c_int, [C.POINTER(Config)] + [vp] * 8),
            "feplb_home_groups": (C.c_int, [vp] * 6),
            "feplb_expert_ffn": (C.c_int, [vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]),
            "feplb_combine": (C.c_int, [vp] * 6),
            "feplb_plan_async": (C.c_int, [vp, vp, vp, vp]),
            "feplb_plan_wait": (C.c_int, [vp, i32, C.POINTER(PlanOut), C.POINTER(vp), C.POINTER(i32), vp]),
            "feplb_moe_forward": (C.c_int, [vp] * 16 + [C.POINTER(PlanOut), vp]),
            "feplb_moe_forward_host": (C.c_int, [vp] * 20 + [C.POINTER(PlanOut), vp]),
            "feplb_moe_forward_host_async": (C.c_int, [vp, i32] + [vp] * 19 + [C.POINTER(PlanOut), vp]),
            "feplb_host_wait": (C.c_int, [vp, i32]),
            "feplb_host_stage_inputs": (C.c_int, [vp, i32] + [vp] * 6),
            "feplb_set_timeline": (C.c_int, [vp, i32]),
            "feplb_get_timeline": (C.c_int, [vp, C.POINTER(Timeline)]),
            "feplb_timeline_totals": (C.c_int, [vp, C.POINTER(Timeline), C.POINTER(i64), i32]),
            "feplb_set_preact_buffer": (C.c_int, [vp, vp]),
            "feplb_transpose_weights": (C.c_int, [vp] * 8),
            "feplb_combine_bwd": (C.c_int, [vp] * 8),
            "feplb_expert_ffn_bwd": (C.c_int, [vp] * 9 + [i32, i32] + [vp] * 6 + [i32, vp]),
            "feplb_dispatch_bwd": (C.c_int, [vp] * 5),
            "feplb_moe_backward": (C.c_int, [vp] * 19 + [i32, vp]),
            "feplb_set_planner_timeout": (C.c_int, [vp, i32]),
            "feplb_set_gemm_form": (C.c_int, [vp, i32, i32]),
            "feplb_set_planner_timing": (C.c_int, [vp, i32, i32]),
            "feplb_set_launch_merging": (C.c_int, [vp, i32]),
            "feplb_pack_weights": (C.c_int, [vp] * 8),
            "feplb_selftest_bounded_wait": (C.c_int, [vp, i32, vp]),
            "feplb_launch_count": (i64, [vp]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def make_config(T, K, E, R, d, f, dyn=4, max_num_dyn=8, tau=0, ranks_per_domain=0,
                policy=POLICY_FIRST_FIT, split=0, split_granule=128, row_align=1,
                mask_policy=MASK_REACTIVE, phase2_copy=0) -> Config:
    return Config(T, K, E, R, d, f, dyn, max_num_dyn, tau, ranks_per_domain, policy, split,
                  split_granule, row_align, mask_policy, phase2_copy)


def config_from_workload(w, **kw) -> Config:
    base = dict(T=w.T, K=w.K, E=w.E, R=w.R, d=w.d, f=w.f, dyn=w.dyn, max_num_dyn=w.max_num_dyn, tau=w.tau)
    base.update(kw)
    return make_config(**base)


def s_pad(cfg: Config) -> int:
    return int(lib().feplb_s_pad(C.byref(cfg)))


class Plan:
    """Host copy of a plan: moves, groups, per-rank loads (numpy)."""

    def __init__(self, cfg: Config):
        self.cap_moves = max(1, cfg.R * cfg.max_num_dyn)
        self.cap_groups = cfg.E + cfg.R * cfg.max_num_dyn
        self._moves = (Move * self.cap_moves)()
        self._groups = (Group * self.cap_groups)()
        self._lb = (C.c_int64 * cfg.R)()
        self._la = (C.c_int64 * cfg.R)()
        self.c = PlanOut(0, 0, self.cap_moves, self.cap_groups, self._moves, self._groups, self._lb, self._la)

    @property
    def moves(self):
        return [(m.expert, m.src, m.dst, m.rows) for m in self._moves[: self.c.n_moves]]

    @property
    def groups(self):
        return [(g.expert, g.row_start, g.rows, g.exec_rank, g.is_dynamic) for g in self._groups[: self.c.n_groups]]

    @property
    def load_before(self):
        return np.array(self._lb[:], np.int64)

    @property
    def load_after(self):
        return np.array(self._la[:], np.int64)


def select_dynamic(score: Sequence[int], E: int, R: int, dyn: int) -> np.ndarray:
    sc = np.ascontiguousarray(score, np.int64)
    out = np.zeros(E, np.uint8)
    rc = lib().feplb_select_dynamic(sc.ctypes.data_as(C.POINTER(C.c_int64)), E, R, dyn,
                                    out.ctypes.data_as(C.POINTER(C.c_uint8)))
    if rc:
        raise FeplbError(rc, "feplb_select_dynamic")
    return out


def ema_update(ema: np.ndarray, counts, decay: float) -> np.ndarray:
    """In place: ema <- decay*ema + (1-decay)*counts (float64 [E])."""
    cnt = np.ascontiguousarray(counts, np.int32)
    assert ema.dtype == np.float64 and ema.flags.c_contiguous and ema.shape == cnt.shape
    rc = lib().feplb_ema_update(ema.ctypes.data_as(C.POINTER(C.c_double)), cnt.ctypes.data_as(C.POINTER(C.c_int32)),
                                cnt.shape[0], float(decay))
    if rc:
        raise FeplbError(rc, "feplb_ema_update")
    return ema


def place_experts(load, R: int) -> np.ndarray:
    """Macro-level placement: new_index[e] = position expert e moves to (host only)."""
    ld = np.ascontiguousarray(load, np.float64)
    out = np.zeros(ld.shape[0], np.int32)
    rc = lib().feplb_place_experts(ld.ctypes.data_as(C.POINTER(C.c_double)), ld.shape[0], int(R),
                                   out.ctypes.data_as(C.POINTER(C.c_int32)))
    if rc:
        raise FeplbError(rc, "feplb_place_experts")
    return out


def plan(cfg: Config, counts, dyn_mask) -> Plan:
    """Host-only greedy plan (no GPU needed)."""
    cnt = np.ascontiguousarray(counts, np.int32)
    msk = np.ascontiguousarray(dyn_mask, np.uint8)
    if cnt.shape != (cfg.E,) or msk.shape != (cfg.E,):
        raise ValueError("counts and dyn_mask must have E entries")
    p = Plan(cfg)
    rc = lib().feplb_plan(C.byref(cfg), cnt.ctypes.data_as(C.POINTER(C.c_int32)),
                          msk.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(p.c))
    if rc:
        raise FeplbError(rc, "feplb_plan")
    return p


def ep_schedule(cfg: Config, counts_by_src, dyn_mask, rank: int) -> dict:
    """What ``rank`` of R real expert-parallel ranks sends and receives (host only; see feplb_ep_schedule).

    ``counts_by_src`` int32 [R, E]: the all-gathered per-rank expert counts.  Returns the plan (identical on
    every rank), int64 [R] row counts ``p1_send/p1_recv`` (dispatch), ``p2_send/p2_recv`` (migrated rows),
    ``comb_send/comb_recv`` (combine) and ``copies``: every weight copy (expert, src, dst, slot, rows, bytes).
    """
    cbs = np.ascontiguousarray(counts_by_src, np.int32)
    msk = np.ascontiguousarray(dyn_mask, np.uint8)
    if cbs.shape != (cfg.R, cfg.E) or msk.shape != (cfg.E,):
        raise ValueError("counts_by_src must be [R, E] and dyn_mask [E]")
    p = Plan(cfg)
    arr = {k: np.zeros(cfg.R, np.int64) for k in ("p1_send", "p1_recv", "p2_send", "p2_recv", "comb_send", "comb_recv")}
    cap = max(1, cfg.R * cfg.max_num_dyn)
    copies = (WeightCopy * cap)()
    n = C.c_int32()
    rc = lib().feplb_ep_schedule(C.byref(cfg), cbs.ctypes.data_as(C.POINTER(C.c_int32)), msk.ctypes.data_as(C.POINTER(C.c_uint8)),
                                 int(rank), C.byref(p.c), *[a.ctypes.data_as(C.POINTER(C.c_int64)) for a in arr.values()],
                                 copies, cap, C.byref(n))
    if rc:
        raise FeplbError(rc, "feplb_ep_schedule")
    out = dict(arr)
    out["plan"] = p
    out["copies"] = [(c.expert, c.src, c.dst, c.slot, c.rows, c.weight_bytes) for c in copies[: n.value]]
    return out


def dispatch_noalloc(cfg: Config, x, topk_ids, counts, x_perm, slot_to_row, row_to_token, status=None, stream=None):
    """Dispatch without a context and without any allocation (scratch is built into the library).

    For callers that cannot allocate device memory at this point (their own pool owns it all, or
    they cannot take cudaMalloc's synchronisation).  Same results as ``Context.dispatch``.  Calls
    on one device must not overlap on the GPU; sizes beyond the built-in scratch raise E_NOMEM.
    """
    rc = lib().feplb_dispatch_noalloc(C.byref(cfg), _ptr(x), _ptr(topk_ids), _ptr(counts), _ptr(x_perm),
                                      _ptr(slot_to_row), _ptr(row_to_token), _ptr(status), Context._stream(stream))
    if rc:
        raise FeplbError(rc, "feplb_dispatch_noalloc")


def _ptr(t) -> Optional[int]:
    """Device/host address of a torch tensor or numpy array (None passes NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    if isinstance(t, int):
        return t
    assert t.is_contiguous()
    return t.data_ptr()


def groups_to_numpy(groups) -> np.ndarray:
    """[(expert, row_start, rows, exec_rank, is_dynamic)] -> int32 [n, 5] in the ABI's struct layout."""
    a = np.asarray(groups, np.int32).reshape(-1, 5)
    return np.ascontiguousarray(a)


class Context:
    """One layer geometry on the current CUDA device.  Calls on one context must not overlap."""

    def __init__(self, cfg: Config):
        self.cfg = cfg
        self._h = C.c_void_p()
        rc = lib().feplb_create(C.byref(cfg), C.byref(self._h))
        if rc:
            raise FeplbError(rc, "feplb_create")
        self.s_cap = s_pad(cfg)

    def close(self):
        if self._h:
            lib().feplb_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _chk(self, rc, where):
        if rc:
            raise FeplbError(rc, where, lib().feplb_last_error(self._h).decode())

    @staticmethod
    def _stream(stream) -> Optional[int]:
        if stream is None:
            import torch
            return torch.cuda.current_stream().cuda_stream or None
        return getattr(stream, "cuda_stream", stream) or None

    def check_status(self, stream=None):
        self._chk(lib().feplb_check_status(self._h, self._stream(stream)), "feplb_check_status")

    def route_topk(self, logits, topk_ids, gates, stream=None):
        self._chk(lib().feplb_route_topk(self._h, _ptr(logits), _ptr(topk_ids), _ptr(gates), self._stream(stream)),
                  "feplb_route_topk")

    def route_hist(self, topk_ids, counts, rank_load, stream=None):
        self._chk(lib().feplb_route_hist(self._h, _ptr(topk_ids), _ptr(counts), _ptr(rank_load),
                                         self._stream(stream)), "feplb_route_hist")

    def dispatch(self, x, topk_ids, counts, x_perm, slot_to_row, row_to_token, stream=None):
        self._chk(lib().feplb_dispatch(self._h, _ptr(x), _ptr(topk_ids), _ptr(counts), _ptr(x_perm),
                                       _ptr(slot_to_row), _ptr(row_to_token), self._stream(stream)), "feplb_dispatch")

    def home_groups(self, counts, dyn_mask, groups_out, dyn_mask_out=None, stream=None):
        self._chk(lib().feplb_home_groups(self._h, _ptr(counts), _ptr(dyn_mask), _ptr(groups_out),
                                          _ptr(dyn_mask_out), self._stream(stream)), "feplb_home_groups")

    def expert_ffn(self, x_perm, w1, w3, w2, groups, n_groups, h_scratch, y_perm, which=FFN_ALL, stream=None):
        self._chk(lib().feplb_expert_ffn(self._h, _ptr(x_perm), _ptr(w1), _ptr(w3), _ptr(w2), _ptr(groups),
                                         int(n_groups), int(which), _ptr(h_scratch), _ptr(y_perm),
                                         self._stream(stream)), "feplb_expert_ffn")

    def combine(self, y_perm, slot_to_row, gates, out, stream=None):
        self._chk(lib().feplb_combine(self._h, _ptr(y_perm), _ptr(slot_to_row), _ptr(gates), _ptr(out),
                                      self._stream(stream)), "feplb_combine")

    def plan_async(self, counts, dyn_mask_host=None, stream=None):
        self._mask_keepalive = None if dyn_mask_host is None else np.ascontiguousarray(dyn_mask_host, np.uint8)
        self._chk(lib().feplb_plan_async(self._h, _ptr(counts), _ptr(self._mask_keepalive), self._stream(stream)),
                  "feplb_plan_async")

    def plan_wait(self, timeout_ms=2000, stream=None):
        """Returns (Plan, device address of the dynamic group table, number of dynamic groups)."""
        p = Plan(self.cfg)
        dev = C.c_void_p()
        n = C.c_int32()
        self._chk(lib().feplb_plan_wait(self._h, int(timeout_ms), C.byref(p.c), C.byref(dev), C.byref(n),
                                        self._stream(stream)), "feplb_plan_wait")
        return p, dev.value, n.value

    def moe_forward(self, x, topk_ids, gates, w1, w3, w2, buf, dyn_mask_host=None, want_plan=True, stream=None):
        """``buf``: object with counts, rank_load, x_perm, h_scratch, y_perm, slot_to_row, row_to_token, out."""
        p = Plan(self.cfg) if want_plan else None
        mask = None if dyn_mask_host is None else np.ascontiguousarray(dyn_mask_host, np.uint8)
        self._chk(lib().feplb_moe_forward(
            self._h, _ptr(x), _ptr(topk_ids), _ptr(gates), _ptr(w1), _ptr(w3), _ptr(w2), _ptr(mask),
            _ptr(buf.counts), _ptr(buf.rank_load), _ptr(buf.x_perm), _ptr(buf.h_scratch), _ptr(buf.y_perm),
            _ptr(buf.slot_to_row), _ptr(buf.row_to_token), _ptr(buf.out),
            C.byref(p.c) if p is not None else None, self._stream(stream)), "feplb_moe_forward")
        return p

    def moe_forward_host(self, x_host, ids_host, gates_host, x_dev, ids_dev, gates_dev, w1, w3, w2, buf, out_host,
                         dyn_mask_host=None, want_plan=False, stream=None):
        p = Plan(self.cfg) if want_plan else None
        mask = None if dyn_mask_host is None else np.ascontiguousarray(dyn_mask_host, np.uint8)
        self._chk(lib().feplb_moe_forward_host(
            self._h, _ptr(x_host), _ptr(ids_host), _ptr(gates_host), _ptr(x_dev), _ptr(ids_dev), _ptr(gates_dev),
            _ptr(w1), _ptr(w3), _ptr(w2), _ptr(mask),
            _ptr(buf.counts), _ptr(buf.rank_load), _ptr(buf.x_perm), _ptr(buf.h_scratch), _ptr(buf.y_perm),
            _ptr(buf.slot_to_row), _ptr(buf.row_to_token), _ptr(buf.out), _ptr(out_host),
            C.byref(p.c) if p is not None else None, self._stream(stream)), "feplb_moe_forward_host")
        return p

    def moe_forward_host_async(self, slot, x_host, ids_host, gates_host, x_dev, ids_dev, gates_dev, w1, w3, w2, buf,
                               out_dev, out_host, dyn_mask_host=None, stream=None):
        """Pipelined host-buffer forward on staging slot 0..HOST_SLOTS-1; ``host_wait(slot)`` before reading out_host."""
        mask = None if dyn_mask_host is None else np.ascontiguousarray(dyn_mask_host, np.uint8)
        self._chk(lib().feplb_moe_forward_host_async(
            self._h, int(slot), _ptr(x_host), _ptr(ids_host), _ptr(gates_host), _ptr(x_dev), _ptr(ids_dev),
            _ptr(gates_dev), _ptr(w1), _ptr(w3), _ptr(w2), _ptr(mask),
            _ptr(buf.counts), _ptr(buf.rank_load), _ptr(buf.x_perm), _ptr(buf.h_scratch), _ptr(buf.y_perm),
            _ptr(buf.slot_to_row), _ptr(buf.row_to_token), _ptr(out_dev), _ptr(out_host), None,
            self._stream(stream)), "feplb_moe_forward_host_async")

    def host_stage_inputs(self, slot, x_host, ids_host, gates_host, x_dev, ids_dev, gates_dev):
        """Start the input copies of the next micro-batch into staging slot ``slot`` ahead of its forward."""
        self._chk(lib().feplb_host_stage_inputs(self._h, int(slot), _ptr(x_host), _ptr(ids_host), _ptr(gates_host),
                                                _ptr(x_dev), _ptr(ids_dev), _ptr(gates_dev)), "feplb_host_stage_inputs")

    def host_wait(self, slot):
        self._chk(lib().feplb_host_wait(self._h, int(slot)), "feplb_host_wait")

    def set_timeline(self, on: bool):
        self._chk(lib().feplb_set_timeline(self._h, int(bool(on))), "feplb_set_timeline")

    def get_timeline(self) -> dict:
        t = Timeline()
        self._chk(lib().feplb_get_timeline(self._h, C.byref(t)), "feplb_get_timeline")
        return {n: getattr(t, n) for n, _ in Timeline._fields_}

    def timeline_totals(self, reset=True):
        """(sums over the timed forwards since the last reset, number of forwards)."""
        t, n = Timeline(), C.c_int64()
        self._chk(lib().feplb_timeline_totals(self._h, C.byref(t), C.byref(n), int(bool(reset))), "feplb_timeline_totals")
        return {k: getattr(t, k) for k, _ in Timeline._fields_}, n.value

    # ---- backward pass ----
    def set_preact_buffer(self, ab):
        self._chk(lib().feplb_set_preact_buffer(self._h, _ptr(ab)), "feplb_set_preact_buffer")

    def transpose_weights(self, w1, w3, w2, w1t, w3t, w2t, stream=None):
        self._chk(lib().feplb_transpose_weights(self._h, _ptr(w1), _ptr(w3), _ptr(w2), _ptr(w1t), _ptr(w3t), _ptr(w2t),
                                                self._stream(stream)), "feplb_transpose_weights")

    def combine_bwd(self, d_out, y_perm, slot_to_row, gates, d_y_perm, d_gates, stream=None):
        self._chk(lib().feplb_combine_bwd(self._h, _ptr(d_out), _ptr(y_perm), _ptr(slot_to_row), _ptr(gates),
                                          _ptr(d_y_perm), _ptr(d_gates), self._stream(stream)), "feplb_combine_bwd")

    def expert_ffn_bwd(self, x_perm, ab_saved, h, d_y_perm, w1t, w3t, w2t, groups, n_groups, expert_table,
                       d_ab, d_x_perm, dw1=None, dw3=None, dw2=None, accumulate=False, which=FFN_ALL, stream=None):
        self._chk(lib().feplb_expert_ffn_bwd(
            self._h, _ptr(x_perm), _ptr(ab_saved), _ptr(h), _ptr(d_y_perm), _ptr(w1t), _ptr(w3t), _ptr(w2t), _ptr(groups),
            int(n_groups), int(which), _ptr(expert_table), _ptr(d_ab), _ptr(d_x_perm), _ptr(dw1),
            _ptr(dw3), _ptr(dw2), int(bool(accumulate)), self._stream(stream)), "feplb_expert_ffn_bwd")

    def dispatch_bwd(self, d_x_perm, slot_to_row, d_x, stream=None):
        self._chk(lib().feplb_dispatch_bwd(self._h, _ptr(d_x_perm), _ptr(slot_to_row), _ptr(d_x), self._stream(stream)),
                  "feplb_dispatch_bwd")

    def moe_backward(self, d_out, gates, w1t, w3t, w2t, buf, bwd, dw1=None, dw3=None, dw2=None, accumulate=False,
                     stream=None):
        """``buf``: the forward's Buffers; ``bwd``: a BackwardBuffers (ab, d_y_perm, d_ab, d_x_perm, d_x, d_gates)."""
        self._chk(lib().feplb_moe_backward(
            self._h, _ptr(d_out), _ptr(gates), _ptr(w1t), _ptr(w3t), _ptr(w2t), _ptr(buf.x_perm), _ptr(bwd.ab),
            _ptr(buf.h_scratch), _ptr(buf.y_perm), _ptr(buf.slot_to_row), _ptr(bwd.d_y_perm),
            _ptr(bwd.d_ab), _ptr(bwd.d_x_perm), _ptr(bwd.d_x), _ptr(bwd.d_gates), _ptr(dw1),
            _ptr(dw3), _ptr(dw2), int(bool(accumulate)), self._stream(stream)), "feplb_moe_backward")

    def set_gemm_form(self, forward_form: int = FORM_AUTO, backward_pair: int = -1):
        """Forces the grouped-GEMM form (FORM_*) of the forward launches and the pair mask of the backward GEMMs."""
        self._chk(lib().feplb_set_gemm_form(self._h, int(forward_form), int(backward_pair)), "feplb_set_gemm_form")

    def set_launch_merging(self, merged: int = -1):
        """1: one GEMM launch per pass over static, then dynamic groups; 0: launches of their own; -1: library's choice."""
        self._chk(lib().feplb_set_launch_merging(self._h, int(merged)), "feplb_set_launch_merging")

    def set_planner_timing(self, planner_delay_us: int = 0, device_wait_limit_us: int = 0):
        """Test aid: delay the planner's table, bound the GEMM's device-side wait for it."""
        self._chk(lib().feplb_set_planner_timing(self._h, int(planner_delay_us), int(device_wait_limit_us)),
                  "feplb_set_planner_timing")

    def pack_weights(self, w1_in, w3_in, w2_in, w1, w3, w2, stream=None):
        """Input-major weights ([E,d,f], [E,d,f], [E,f,d]) -> the library's output-major layout."""
        self._chk(lib().feplb_pack_weights(self._h, _ptr(w1_in), _ptr(w3_in), _ptr(w2_in), _ptr(w1), _ptr(w3), _ptr(w2),
                                           self._stream(stream)), "feplb_pack_weights")

    def set_planner_timeout(self, timeout_ms: int):
        self._chk(lib().feplb_set_planner_timeout(self._h, int(timeout_ms)), "feplb_set_planner_timeout")

    def selftest_bounded_wait(self, limit_us=2000, stream=None):
        """Raises unless a device-side wait on a barrier nobody completes gives up after limit_us."""
        self._chk(lib().feplb_selftest_bounded_wait(self._h, int(limit_us), self._stream(stream)),
                  "feplb_selftest_bounded_wait")

    def launch_count(self) -> int:
        return int(lib().feplb_launch_count(self._h))


class Buffers:
    """Caller-owned device outputs and scratch of one layer geometry (torch tensors on ``device``)."""

    def __init__(self, cfg: Config, device="cuda"):
        import torch
        cap = s_pad(cfg)
        i32, bf = torch.int32, torch.bfloat16
        self.counts = torch.zeros(cfg.E, dtype=i32, device=device)
        self.rank_load = torch.zeros(cfg.R, dtype=i32, device=device)
        self.x_perm = torch.empty(max(cap, 1), cfg.d, dtype=bf, device=device)
        self.h_scratch = torch.empty(max(cap, 1), cfg.f, dtype=bf, device=device)
        self.y_perm = torch.empty(max(cap, 1), cfg.d, dtype=bf, device=device)
        self.slot_to_row = torch.empty(max(cfg.T, 1), cfg.K, dtype=i32, device=device)
        self.row_to_token = torch.empty(max(cap, 1), dtype=i32, device=device)
        self.out = torch.empty(max(cfg.T, 1), cfg.d, dtype=bf, device=device)


class BackwardBuffers:
    """Caller-owned device buffers of the backward pass of one layer geometry."""

    def __init__(self, cfg: Config, device="cuda"):
        import torch
        cap = max(s_pad(cfg), 1)
        bf = torch.bfloat16
        self.ab = torch.zeros(cap, 2 * cfg.f, dtype=bf, device=device)          # saved pre-activations
        self.d_y_perm = torch.zeros(cap, cfg.d, dtype=bf, device=device)
        self.d_ab = torch.zeros(cap, 2 * cfg.f, dtype=bf, device=device)
        self.d_x_perm = torch.zeros(cap, cfg.d, dtype=bf, device=device)
        self.d_x = torch.zeros(max(cfg.T, 1), cfg.d, dtype=bf, device=device)
        self.d_gates = torch.zeros(max(cfg.T, 1), cfg.K, dtype=torch.float32, device=device)


def bf16_tensor(bits: np.ndarray, device="cuda"):
    """numpy uint16 bf16 bit patterns -> torch.bfloat16 tensor on ``device`` (bit copy)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device)


def bf16_bits(t) -> np.ndarray:
    """torch.bfloat16 tensor -> numpy uint16 bit patterns (bit copy)."""
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
