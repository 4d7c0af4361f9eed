"""Seeded synthetic inputs for the FEPLB MoE-layer hot path.

This module only *draws inputs*: activations, expert weights, router outputs
(top-k expert ids and gates) and the layer geometry of each named workload.  It
holds none of the method's arithmetic (no histogram, plan, permutation, FFN or
combine) and is the one module that both the CPU oracle's tests and the CUDA
path's tests/bench import.

The paper measured on routing traces of a GLM-5 training run (Section 3.1,
"Model configuration"), which are not available; the generators below stand in
for them with the paper's shape -- 128 routed experts in contiguous blocks of
E/EP experts per device, top-k routing with no balancing loss, and per
micro-batch skewed loads (Section 1, Figure 1 caption).

Conventions
-----------
* bf16 tensors travel as ``numpy.uint16`` bit patterns (numpy has no bf16);
  ``bf16_bits_to_f64`` / ``f32_to_bf16_bits`` convert exactly / with
  round-to-nearest-even.
* ``topk_ids`` int32 [T, K], ``gates`` float32 [T, K], ``x`` uint16 [T, d].
* Expert weights are stored output-major ("linear layer" layout):
  ``w1, w3`` uint16 [E, f, d] and ``w2`` uint16 [E, d, f]; row n of ``w1[e]``
  holds the d input coefficients of output feature n.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "get_workload", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "bf16_bits_to_f64", "gen_activations", "gen_weights", "gen_routing",
    "gen_microbatch", "sweep_points",
]


@dataclasses.dataclass(frozen=True)
class Workload:
    """Geometry and balancer parameters of one named workload."""
    name: str
    cfg_id: int            # 1..5, used in seeds
    T: int                 # tokens per micro-batch
    d: int                 # hidden size
    f: int                 # expert FFN width
    E: int                 # experts
    K: int                 # top-k
    R: int                 # virtual EP ranks (contiguous expert blocks)
    dyn: int               # dynamic experts per rank (Section 2.3)
    max_num_dyn: int       # received experts per rank (Section 2.3, receive buffer)
    tau: int               # minimum rows for a migration (Section 2.3)
    n_microbatches: int
    routing: str           # "zipf" | "dirichlet" | "hot3"
    alpha: float           # Zipf exponent / Dirichlet concentration
    smooth: float = 0.0    # mix-in of the uniform distribution (0 = none)

    @property
    def S(self) -> int:
        return self.T * self.K

    @property
    def L(self) -> int:
        return self.E // self.R

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    # Tiny layer, Zipf(1.2) popularity over a seeded expert order.
    "cfg1": Workload("cfg1", 1, T=256, d=128, f=64, E=8, K=2, R=2, dyn=2, max_num_dyn=2,
                     tau=4, n_microbatches=1, routing="zipf", alpha=1.2),
    # Mid layer, Dirichlet(0.3) popularity redrawn per micro-batch.
    "cfg2": Workload("cfg2", 2, T=4096, d=2048, f=768, E=64, K=6, R=4, dyn=4, max_num_dyn=8,
                     tau=64, n_microbatches=8, routing="dirichlet", alpha=0.3),
    # GLM-5-like layer: 128 experts, 3*d*f*2 B = 72 MiB per expert (Section 2.3).
    "cfg3": Workload("cfg3", 3, T=16384, d=6144, f=2048, E=128, K=8, R=8, dyn=4, max_num_dyn=8,
                     tau=64, n_microbatches=16, routing="dirichlet", alpha=0.2),
    "cfg3-smooth": Workload("cfg3-smooth", 3, T=16384, d=6144, f=2048, E=128, K=8, R=8, dyn=4,
                            max_num_dyn=8, tau=64, n_microbatches=16, routing="dirichlet",
                            alpha=0.2, smooth=0.5),
    # The GLM-5-like expert shapes on a device footprint small enough for a full ncu capture
    # (2.25 GiB of weights, ~1 GiB of activations); 1024 rows per expert on average like cfg3.
    "cfg3-prof": Workload("cfg3-prof", 3, T=4096, d=6144, f=2048, E=32, K=8, R=4, dyn=4, max_num_dyn=8,
                          tau=64, n_microbatches=2, routing="dirichlet", alpha=0.2),
    # Extreme skew: 3 experts of one rank take 35 % of all (token, k) slots.
    "cfg4": Workload("cfg4", 4, T=4096, d=2048, f=768, E=64, K=6, R=4, dyn=4, max_num_dyn=8,
                     tau=64, n_microbatches=8, routing="hot3", alpha=0.35),
}


def get_workload(name: str) -> Workload:
    """A named workload, or a point of the scaling sweep by its name (``cfg5-T8192-R8``)."""
    if name in WORKLOADS:
        return WORKLOADS[name]
    for p in sweep_points():
        if p.name == name:
            return p
    raise KeyError(name)


def sweep_points(Ts=(2048, 8192, 32768, 65536), Rs=(1, 2, 4, 8, 16)):
    """The scaling sweep: cfg3's layer at several T and virtual EP degrees R."""
    base = WORKLOADS["cfg3"]
    out = []
    for T in Ts:
        for R in Rs:
            L = base.E // R
            out.append(base.with_(name=f"cfg5-T{T}-R{R}", cfg_id=5, T=T, R=R, dyn=min(4, L),
                                  n_microbatches=4))
    return out


# ----------------------------------------------------------------------------- bf16 helpers

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------------------- tensors

def _normal_bf16(seed_key, shape, std=0.02) -> np.ndarray:
    rng = np.random.default_rng(seed_key)
    a = rng.standard_normal(shape, dtype=np.float32)
    a *= np.float32(std)
    return f32_to_bf16_bits(a)


def gen_activations(w: Workload, mb: int) -> np.ndarray:
    """x: bf16 bits [T, d], N(0, 0.02^2)."""
    return _normal_bf16([1000 * w.cfg_id + mb, 7], (w.T, w.d))


def gen_weights(w: Workload, n_threads: int | None = None):
    """(w1, w3, w2) bf16 bits, [E,f,d], [E,f,d], [E,d,f]; one seed per (config, expert, matrix)."""
    seed = 1000 * w.cfg_id + 999
    w1 = np.empty((w.E, w.f, w.d), np.uint16)
    w3 = np.empty((w.E, w.f, w.d), np.uint16)
    w2 = np.empty((w.E, w.d, w.f), np.uint16)

    def one(e):
        w1[e] = _normal_bf16([seed, e, 1], (w.f, w.d))
        w3[e] = _normal_bf16([seed, e, 3], (w.f, w.d))
        w2[e] = _normal_bf16([seed, e, 2], (w.d, w.f))

    n_threads = n_threads or min(16, os.cpu_count() or 1)
    if w.E * w.d * w.f < (1 << 22) or n_threads == 1:
        for e in range(w.E):
            one(e)
    else:
        with ThreadPoolExecutor(n_threads) as ex:
            list(ex.map(one, range(w.E)))
    return w1, w3, w2


# ----------------------------------------------------------------------------- routing

def _popularity(w: Workload, rng) -> np.ndarray:
    if w.routing == "zipf":
        order = rng.permutation(w.E)
        p = np.empty(w.E, np.float64)
        p[order] = (np.arange(w.E) + 1.0) ** (-w.alpha)
    elif w.routing == "dirichlet":
        p = rng.dirichlet(np.full(w.E, w.alpha))
        p = np.maximum(p, 1e-30)
    else:
        raise ValueError(w.routing)
    p = p / p.sum()
    if w.smooth:
        p = (1.0 - w.smooth) * p + w.smooth / w.E
    return p


def _softmax_f32(z: np.ndarray) -> np.ndarray:
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z, dtype=np.float32)
    return (e / e.sum(axis=1, keepdims=True)).astype(np.float32)


def _route_popularity(w: Workload, rng):
    """Gumbel-top-k: K distinct experts per token, drawn proportionally to p."""
    p = _popularity(w, rng)
    g = rng.gumbel(size=(w.T, w.E)).astype(np.float32)
    logit = (np.log(p).astype(np.float32)[None, :] + g).astype(np.float32)
    # K largest logits, descending; ties -> lower expert id (stable sort on the negation)
    order = np.argsort(-logit, axis=1, kind="stable")[:, : w.K]
    sel = np.take_along_axis(logit, order, axis=1)
    return order.astype(np.int32), _softmax_f32(sel)


def _route_hot3(w: Workload, rng_fixed, rng):
    """Three seeded experts of one seeded rank each receive round(alpha*T*K/3) distinct tokens;
    every token fills its remaining slots uniformly, without replacement, from the other experts."""
    L = w.E // w.R
    hot_rank = int(rng_fixed.integers(w.R))
    hot = np.sort(hot_rank * L + rng_fixed.choice(L, size=3, replace=False))
    n_hot = int(round(w.alpha * w.T * w.K / 3.0))
    assert n_hot <= w.T
    member = np.zeros((w.T, w.E), bool)
    for e in hot:
        member[rng.choice(w.T, size=n_hot, replace=False), e] = True
    cold = np.setdiff1d(np.arange(w.E), hot)
    # random priorities over the cold experts; take the top (K - #hot) per token
    pri = rng.random((w.T, cold.size))
    cold_order = np.argsort(pri, axis=1, kind="stable")
    n_hot_tok = member.sum(axis=1)
    ids = np.empty((w.T, w.K), np.int64)
    for t in range(w.T):
        h = np.flatnonzero(member[t])
        ids[t, : h.size] = h
        ids[t, h.size:] = cold[cold_order[t, : w.K - h.size]]
    del n_hot_tok
    logit = rng.standard_normal((w.T, w.K)).astype(np.float32)
    order = np.argsort(-logit, axis=1, kind="stable")
    # slot j of token t is the expert paired with the j-th largest logit
    slot_perm = rng.permuted(np.tile(np.arange(w.K), (w.T, 1)), axis=1)
    ids = np.take_along_axis(ids, slot_perm, axis=1)
    ids = np.take_along_axis(ids, order, axis=1)
    sel = np.take_along_axis(logit, order, axis=1)
    return ids.astype(np.int32), _softmax_f32(sel)


def gen_routing(w: Workload, mb: int):
    """(topk_ids int32 [T,K], gates float32 [T,K]) of micro-batch ``mb``."""
    rng = np.random.default_rng([1000 * w.cfg_id + mb, 3])
    if w.routing == "hot3":
        rng_fixed = np.random.default_rng([1000 * w.cfg_id, 5])   # hot set fixed across micro-batches
        return _route_hot3(w, rng_fixed, rng)
    return _route_popularity(w, rng)


def gen_microbatch(w: Workload, mb: int):
    """(x, topk_ids, gates) of micro-batch ``mb``."""
    ids, gates = gen_routing(w, mb)
    return gen_activations(w, mb), ids, gates
