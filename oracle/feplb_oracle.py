"""CPU oracle for the FEPLB per-micro-batch MoE-layer hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct restatement of what the hot path computes, written from
the paper (FEPLB, Sections 2.2-2.3 and 3.1) and used to check the CUDA library.  Only the
test-suite, the smoke check and the benchmark's ``cpu_baseline`` / ``--impl reference`` legs may
import it; the product path never does.  It shares no code with the CUDA path: numpy only,
fp64 for every floating-point step, no blocking, fusion or reordering beyond the definitions
below.

Notation (Section 2.3): T tokens, K experts per token (top-k), E experts, R ranks, L = E/R
experts per rank in contiguous blocks so that home(e) = e // L (Section 3.1: 128/EP experts
per device), S = T*K slots with slot index s = t*K + k, d hidden size, f expert width,
A = row alignment of expert segments (1 or 128), g = split granule.

What each function follows
--------------------------
route_hist      per-expert token counts known to every device after Phase 1 (Section 2.2);
                definition written out.                                   pinned: numpy.bincount,
                conservation, brute force
permute         the expert-order permutation of Phase 1 (Section 2.2) = stable counting sort of
                slots by expert id; definition written out.               pinned: numpy stable
                argsort, bijection invariants
gather_rows     row copies of the permutation.                            pinned: round trip
plan            the greedy load balancer of Section 2.3 (busiest dynamic expert of the most
                overloaded device -> most underloaded device, threshold tau, whole experts,
                deterministic).  The paper gives one prose paragraph and no worked example, so
                every tie-break and stopping rule is a stated reading (see the function).
                PARITY UNPINNED against the paper; pinned against invariants, closed-form
                special cases, brute-force optimum bounds on tiny inputs and hand-worked vectors.
select_dynamic  static/dynamic partition controlled by ``dyn`` (Section 2.3); a reading
                (busiest ``dyn`` experts of each rank).  PARITY UNPINNED against the paper.
expert_ffn      grouped GEMM of the experts (Sections 2.3, 3.1) with the SwiGLU expert of the
                workload definition: y = (silu(x W1) * (x W3)) W2 in fp64.  pinned: scalar loops,
                one-hot rows, linearity
expert_hidden   the first half of expert_ffn on its own (h = silu(x W1) * (x W3)), which expert_ffn
                calls; lets a test look at the CUDA path's H buffer.      pinned: through expert_ffn
_round_f64_to_bf16  round-to-nearest-even to bf16 by way of float32 (the accumulator type of the
                GPU path), used only by expert_ffn(round_h_bf16=True).    pinned: hand-picked ties
                of both parities, values next to a tie, negative and tiny values, a scalar
                integer re-implementation, the input generator's own rounding routine
combine         the Combine phase (Section 2.3) = gate-weighted sum of the K
                expert outputs of a token.                                pinned: K=1 round trip,
                scalar loops
token_straggler the paper's metric max_d T_d - mean (Section 3.1 "Metrics").  pinned: Table 3
                arithmetic
route_topk      top-k gating of the router (Sections 2.3, 3.1); gates = softmax over the selected
                logits is the workloads' definition, not the paper's.  PARITY UNPINNED against
                the paper; pinned: library stable sort, closed forms (sigmoid, plain softmax)
place_experts   macro-level expert-to-device assignment from historical load (Section 2.3, Router
                Predictor; no algorithm given): capacity-constrained LPT greedy, a reading.
                PARITY UNPINNED against the paper; pinned: permutation invariant, brute-force
                optimum and the 4/3 LPT bound on tiny inputs
ep_exchange     who sends how many rows to whom when the R ranks are real devices (Section 2.2, Phase 1:
                tokens go to their expert's home; Phase 2: the rows of migrated pieces go on to the
                receiving device with the expert's weights; Section 2.3: results return to the source
                devices), counted one row at a time from a plan.  A bookkeeping definition.  pinned:
                conservation laws, a hand-worked case
moe_layer_backward  gradients of the layer w.r.t. x, gates and the expert weights (Table 2 reports
                backward times; the pass itself is not described): the chain rule of the forward
                definition.                                               pinned: central finite
                differences of the forward definition
"""
from __future__ import annotations

import numpy as np

POLICY_LITERAL = 0
POLICY_FIRST_FIT = 1


# ----------------------------------------------------------------------------- helpers

def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def round_up(n: int, a: int) -> int:
    return (n + a - 1) // a * a


# ----------------------------------------------------------------------------- step 1: histogram

def route_hist(topk_ids: np.ndarray, E: int, R: int):
    """counts[e] = number of slots routed to expert e; load_before[r] = rows of rank r's block.

    Section 2.2: after Phase 1 every device knows the exact per-expert token counts.
    Ids outside [0, E) are an error.  Returns (counts int64 [E], load_before int64 [R]).
    """
    assert E % R == 0
    L = E // R
    counts = [0] * E
    for e in np.asarray(topk_ids).reshape(-1).tolist():
        if not 0 <= e < E:
            raise ValueError(f"expert id {e} outside [0, {E})")
        counts[e] += 1
    load = [0] * R
    for e in range(E):
        load[e // L] += counts[e]
    return np.array(counts, np.int64), np.array(load, np.int64)


# ----------------------------------------------------------------------------- step 3: permutation

def segment_offsets(counts, A: int = 1):
    """pad_off[e] = sum_{e' < e} round_up(counts[e'], A); also the padded total."""
    off, tot = [], 0
    for c in np.asarray(counts).tolist():
        off.append(tot)
        tot += round_up(int(c), A)
    return np.array(off, np.int64), tot


def permute(topk_ids: np.ndarray, E: int, A: int = 1):
    """Stable counting sort of the S slots by expert id (Section 2.2, Phase 1).

    Walking s = 0..S-1 in order, slot s goes to row pad_off[e] + (number of earlier slots of e).
    Returns (slot_to_row int64 [T,K], row_to_token int64 [S_pad] with -1 in padding rows,
             pad_off int64 [E], S_pad).
    """
    ids = np.asarray(topk_ids)
    T, K = ids.shape
    counts, _ = route_hist(ids, E, 1)
    pad_off, S_pad = segment_offsets(counts, A)
    nxt = pad_off.tolist()
    slot_to_row = [0] * (T * K)
    row_to_token = [-1] * S_pad
    for s, e in enumerate(ids.reshape(-1).tolist()):
        r = nxt[e]
        nxt[e] = r + 1
        slot_to_row[s] = r
        row_to_token[r] = s // K
    return (np.array(slot_to_row, np.int64).reshape(T, K), np.array(row_to_token, np.int64),
            pad_off, S_pad)


def gather_rows(x_bits: np.ndarray, row_to_token: np.ndarray) -> np.ndarray:
    """x_perm[row, :] = x[row_to_token[row], :] bit-copied; padding rows are zero."""
    x_bits = np.asarray(x_bits)
    out = np.zeros((row_to_token.shape[0], x_bits.shape[1]), x_bits.dtype)
    for r, t in enumerate(np.asarray(row_to_token).tolist()):
        if t >= 0:
            out[r] = x_bits[t]
    return out


# ----------------------------------------------------------------------------- step 2: plan

def select_dynamic(score, E: int, R: int, dyn: int) -> np.ndarray:
    """Mark the ``dyn`` highest-scoring experts of every rank as dynamic (ties -> lower id).

    Section 2.3: experts of a device are partitioned into static and dynamic, controlled by
    ``dyn``.  The paper does not say which experts are dynamic; this helper takes the busiest.
    """
    L = E // R
    score = np.asarray(score).tolist()
    mask = np.zeros(E, np.uint8)
    for r in range(R):
        block = list(range(r * L, (r + 1) * L))
        block.sort(key=lambda e: (-score[e], e))
        for e in block[: max(0, min(dyn, L))]:
            mask[e] = 1
    return mask


def plan(counts, dyn_mask, R: int, tau: int = 0, max_num_dyn: int = 8, ranks_per_domain: int = 0,
         policy: int = POLICY_FIRST_FIT, split: int = 0, split_granule: int = 128,
         row_align: int = 1):
    """Greedy per-micro-batch rebalancing plan (Section 2.3, load-balancer paragraph).

    Section 2.3 fixes the shape of the loop (source = most loaded device, object = its busiest
    dynamic expert, target = least loaded device, a row threshold tau, whole experts, the same
    result on every device).  Readings where it is silent:
      * load of a rank = rows ((token, k) slots) it executes, static and dynamic together;
      * most overloaded / underloaded = max / min load inside the NVLink domain, ties -> lowest
        rank id; a destination must still have a free slot in its receive buffer
        (``max_num_dyn`` received experts per rank, Section 2.3 memory paragraph);
      * busiest = most remaining rows, ties -> lowest expert id; eligible iff rows >= max(tau, 1);
      * a move is taken only if it strictly lowers the larger of the two loads, i.e. rows < gap;
        LITERAL stops when the busiest eligible expert fails this, FIRST_FIT tries the next one;
      * the source of a copy is always the expert's home rank and an expert moves at most once;
      * rebalancing never crosses a domain of ``ranks_per_domain`` consecutive ranks (0 = all R).
    ``split=1`` is an extension the paper does not have (its Conclusion lists token-level
    splitting as a limitation): a hot expert's rows may be cut, in multiples of
    ``split_granule``, and spread so that no rank is pushed across the domain mean.

    Returns a dict: moves [(expert, src, dst, rows)], load_before, load_after (int64 [R]),
    exec_rows (int64 [R, E]: rows of expert e executed on rank r) and groups
    [(expert, row_start, rows, exec_rank, is_dynamic)] in expert order -- for each expert the
    moved pieces in move order from the front of its segment, then the home remainder;
    zero-row groups are omitted.
    """
    counts = [int(c) for c in np.asarray(counts).tolist()]
    mask = [int(m) != 0 for m in np.asarray(dyn_mask).tolist()]
    E = len(counts)
    assert E % R == 0 and len(mask) == E
    L = E // R
    D = R if ranks_per_domain in (0, None) else int(ranks_per_domain)
    assert R % D == 0
    thr = max(int(tau), 1)
    g = max(int(split_granule), 1)

    load = [sum(counts[r * L:(r + 1) * L]) for r in range(R)]
    load_before = list(load)
    rem = list(counts)
    moved = [False] * E
    used = [0] * R
    pairs = set()
    moves = []

    for dom in range(R // D):
        ranks = list(range(dom * D, (dom + 1) * D))
        M = -(-sum(load[r] for r in ranks) // D)          # ceil of the domain mean
        while True:
            src = min(ranks, key=lambda r: (-load[r], r))
            if split and load[src] <= M:
                break
            dsts = [r for r in ranks if r != src and used[r] < max_num_dyn
                    and (not split or load[r] < M)]
            if not dsts:
                break
            dst = min(dsts, key=lambda r: (load[r], r))
            gap = load[src] - load[dst]
            if gap <= 0:
                break
            cand = [e for e in range(src * L, (src + 1) * L)
                    if mask[e] and not moved[e] and rem[e] >= thr and (e, dst) not in pairs]
            cand.sort(key=lambda e: (-rem[e], e))
            chosen = None
            for e in cand:
                if not split:
                    if rem[e] < gap:
                        chosen = (e, rem[e])
                        break
                else:
                    m = min(rem[e], load[src] - M, M - load[dst])
                    if m < rem[e]:
                        m = m // g * g
                    if m >= thr:
                        chosen = (e, m)
                        break
                if policy == POLICY_LITERAL:
                    break
            if chosen is None:
                break
            e, m = chosen
            if not split:
                moved[e] = True
            rem[e] -= m
            load[src] -= m
            load[dst] += m
            used[dst] += 1
            pairs.add((e, dst))
            moves.append((e, src, dst, m))

    pad_off, _ = segment_offsets(counts, row_align)
    exec_rows = np.zeros((R, E), np.int64)
    groups = []
    for e in range(E):
        p = int(pad_off[e])
        for (me, _src, dst, m) in moves:
            if me == e:
                groups.append((e, p, m, dst, int(mask[e])))
                exec_rows[dst, e] += m
                p += m
        if rem[e] > 0:
            groups.append((e, p, rem[e], e // L, int(mask[e])))
            exec_rows[e // L, e] += rem[e]
    return {
        "moves": moves,
        "load_before": np.array(load_before, np.int64),
        "load_after": np.array(load, np.int64),
        "exec_rows": exec_rows,
        "groups": groups,
    }


def token_straggler(load) -> float:
    """max_d T_d - mean_d T_d (Section 3.1, "Metrics")."""
    load = np.asarray(load, np.float64)
    return float(load.max() - load.mean())


def straggler_ratio(load) -> float:
    """max_d T_d / mean_d T_d, the scale-free form of the same metric."""
    load = np.asarray(load, np.float64)
    return float(load.max() / load.mean()) if load.mean() > 0 else 1.0


# ----------------------------------------------------------------------------- steps 4-5: expert FFN

def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def expert_ffn(x_rows_bits: np.ndarray, row_expert: np.ndarray, w1_bits, w3_bits, w2_bits,
               round_h_bf16: bool = False) -> np.ndarray:
    """y[i,:] = (silu(x_i W1[e]) * (x_i W3[e])) W2[e] with e = row_expert[i], all in fp64.

    Weights are stored output-major: w1, w3 [E, f, d], w2 [E, d, f], so x W1[e] is
    ``x @ w1[e].T``.  Rows with row_expert < 0 (padding) give zeros.  ``round_h_bf16`` rounds
    the hidden activation to bf16 (as the GPU path stores it) to localise discrepancies; the
    parity reference leaves it off.
    """
    x_rows_bits = np.asarray(x_rows_bits)
    row_expert = np.asarray(row_expert)
    n = x_rows_bits.shape[0]
    d_out = w2_bits.shape[1]
    h_all = expert_hidden(x_rows_bits, row_expert, w1_bits, w3_bits)
    if round_h_bf16:
        h_all = _round_f64_to_bf16(h_all)
    y = np.zeros((n, d_out), np.float64)
    for e in np.unique(row_expert).tolist():
        if e < 0:
            continue
        idx = np.flatnonzero(row_expert == e)
        y[idx] = h_all[idx] @ bf16_bits_to_f64(w2_bits[e]).T
    return y


def expert_hidden(x_rows_bits: np.ndarray, row_expert: np.ndarray, w1_bits, w3_bits) -> np.ndarray:
    """The hidden activation of expert_ffn on its own: h[i,:] = silu(x_i W1[e]) * (x_i W3[e]), fp64;
    padding rows give zeros."""
    x_rows_bits = np.asarray(x_rows_bits)
    row_expert = np.asarray(row_expert)
    h = np.zeros((x_rows_bits.shape[0], w1_bits.shape[1]), np.float64)
    for e in np.unique(row_expert).tolist():
        if e < 0:
            continue
        idx = np.flatnonzero(row_expert == e)
        X = bf16_bits_to_f64(x_rows_bits[idx])
        a = X @ bf16_bits_to_f64(w1_bits[e]).T
        b = X @ bf16_bits_to_f64(w3_bits[e]).T
        h[idx] = silu(a) * b
    return h


def _round_f64_to_bf16(a: np.ndarray) -> np.ndarray:
    """fp64 -> float32 (numpy's round-to-nearest-even) -> bf16 (nearest, ties to the even
    mantissa), returned as fp64.  Through float32 on purpose: the value being modelled is an fp32
    accumulator that the kernel rounds to bf16."""
    f = a.astype(np.float32)
    u = f.view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    u = ((u + r) >> np.uint32(16)) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------- step 6: combine

def combine(y_rows: np.ndarray, slot_to_row: np.ndarray, gates: np.ndarray) -> np.ndarray:
    """out[t,:] = sum_k gates[t,k] * y_rows[slot_to_row[t,k], :] in fp64 (Section 2.3, Combine)."""
    slot_to_row = np.asarray(slot_to_row)
    T, K = slot_to_row.shape
    g = np.asarray(gates, np.float64)
    out = np.zeros((T, y_rows.shape[1]), np.float64)
    for k in range(K):
        out += g[:, k:k + 1] * y_rows[slot_to_row[:, k]]
    return out


# ----------------------------------------------------------------------------- expert parallelism over real ranks

def ep_exchange(counts_by_src, plan_result, max_num_dyn: int):
    """Row traffic of expert parallelism over R real ranks for one micro-batch (Sections 2.2, 2.3).

    ``counts_by_src[s][e]`` = slots of rank s's own tokens routed to expert e.  The rows of expert e
    are ordered by source rank, then by slot (the order ``permute`` gives when the ranks' tokens are
    numbered one rank after the other); ``plan_result`` is ``plan()`` on the column sums.  Every row
    is followed on its way: source -> home of its expert (Phase 1) -> the rank that executes it, if
    its piece was migrated (Phase 2) -> back to the source (combine).  Returns
    (p1, p2, comb, copies): p1[s][r], p2[s][r], comb[s][r] = rows rank s sends to rank r in the three
    steps, copies = [(expert, src, dst, slot, rows)] with slot = dst*max_num_dyn + (earlier moves
    into dst).
    """
    cbs = [[int(v) for v in row] for row in np.asarray(counts_by_src).tolist()]
    R, E = len(cbs), len(cbs[0])
    L = E // R
    p1 = [[0] * R for _ in range(R)]
    p2 = [[0] * R for _ in range(R)]
    comb = [[0] * R for _ in range(R)]
    for e in range(E):
        exec_of_row = []
        for (ge, _start, rows, exec_rank, _dyn) in plan_result["groups"]:
            if ge == e:
                exec_of_row += [exec_rank] * rows
        assert len(exec_of_row) == sum(cbs[s][e] for s in range(R))
        pos = 0
        for s in range(R):
            for _ in range(cbs[s][e]):
                home, x = e // L, exec_of_row[pos]
                pos += 1
                p1[s][home] += 1
                if x != home:
                    p2[home][x] += 1
                comb[x][s] += 1
    used = [0] * R
    copies = []
    for (e, src, dst, rows) in plan_result["moves"]:
        copies.append((e, src, dst, dst * max_num_dyn + used[dst], rows))
        used[dst] += 1
    return np.array(p1, np.int64), np.array(p2, np.int64), np.array(comb, np.int64), copies


# ----------------------------------------------------------------------------- whole layer

def row_experts(topk_ids: np.ndarray, slot_to_row: np.ndarray, S_pad: int) -> np.ndarray:
    """Expert id owning each permuted row (-1 for padding)."""
    re = np.full(S_pad, -1, np.int64)
    re[np.asarray(slot_to_row).reshape(-1)] = np.asarray(topk_ids).reshape(-1)
    return re


def moe_layer(x_bits, topk_ids, gates, w1_bits, w3_bits, w2_bits, E: int, A: int = 1,
              tokens=None):
    """The layer output out[t,:] in fp64; with ``tokens`` only for that subset of tokens.

    The plan does not enter: migrating an expert changes where its rows are computed, never
    their value (Section 2.2: each token is still processed by the same expert with identical
    weights).
    """
    ids = np.asarray(topk_ids)
    T, K = ids.shape
    if tokens is None:
        tokens = np.arange(T)
    tokens = np.asarray(tokens)
    sub_ids = ids[tokens]                                   # [n, K]
    x_rows = np.repeat(np.asarray(x_bits)[tokens], K, axis=0)   # slot-major rows of the subset
    y = expert_ffn(x_rows, sub_ids.reshape(-1), w1_bits, w3_bits, w2_bits)
    s2r = np.arange(tokens.shape[0] * K).reshape(-1, K)
    return combine(y, s2r, np.asarray(gates)[tokens])


# ----------------------------------------------------------------------------- router, placement

def route_topk(logits: np.ndarray, K: int):
    """Top-k gating (Step 0: Section 2.3, router; Section 3.1, top-k without auxiliary loss): per token the K largest logits in descending order, ties to the
    lower expert id; gates = softmax over the K selected logits.  The paper gives no formula for
    the gates; softmax over the selected logits is the workloads' definition.  PARITY UNPINNED
    against the paper; pinned against a library sort and closed forms.
    Returns (topk_ids int64 [T,K], gates float64 [T,K]).
    """
    z = np.asarray(logits, np.float64)
    T, E = z.shape
    ids = np.empty((T, K), np.int64)
    gates = np.empty((T, K), np.float64)
    for t in range(T):
        order = sorted(range(E), key=lambda e: (-z[t, e], e))[:K]
        sel = np.array([z[t, e] for e in order])
        w = np.exp(sel - sel.max())
        ids[t] = order
        gates[t] = w / w.sum()
    return ids, gates


def ema_update(ema, counts, decay: float):
    """Historical routing statistics of the macro level (Section 2.3): ema <- decay*ema + (1-decay)*counts."""
    return decay * np.asarray(ema, np.float64) + (1.0 - decay) * np.asarray(counts, np.float64)


def place_experts(load, R: int) -> np.ndarray:
    """Expert-to-device assignment from historical load (Section 2.3, Router Predictor; the paper
    gives no algorithm).  Reading: longest-processing-time greedy under the capacity of L = E/R
    experts per rank -- experts by descending load (ties -> lower id), each to the least loaded
    rank that still has room (ties -> lower rank).  PARITY UNPINNED against the paper.
    Returns new_index int64 [E]: expert e moves to position new_index[e] (rank = position // L).
    """
    load = [float(v) for v in np.asarray(load).tolist()]
    E = len(load)
    assert E % R == 0
    L = E // R
    order = sorted(range(E), key=lambda e: (-load[e], e))
    rank_load = [0.0] * R
    fill = [0] * R
    new_index = [0] * E
    for e in order:
        r = min((r for r in range(R) if fill[r] < L), key=lambda r: (rank_load[r], r))
        new_index[e] = r * L + fill[r]
        fill[r] += 1
        rank_load[r] += load[e]
    return np.array(new_index, np.int64)


# ----------------------------------------------------------------------------- backward pass

def dsilu(z: np.ndarray) -> np.ndarray:
    """d/dz [z * sigmoid(z)] = sigmoid(z) * (1 + z * (1 - sigmoid(z)))."""
    sg = 1.0 / (1.0 + np.exp(-z))
    return sg * (1.0 + z * (1.0 - sg))


def moe_layer_backward(x_bits, topk_ids, gates, w1_bits, w3_bits, w2_bits, d_out, E: int):
    """Gradients of out[t,:] = sum_k gates[t,k] * FFN_{e(t,k)}(x[t,:]) (the layer of moe_layer)
    with respect to x, gates and the expert weights, for the upstream gradient d_out [T,d]; all
    fp64, the chain rule written out per (token, k) slot grouped by expert.  The paper reports
    forward/backward layer times (Table 2) but does not describe the backward pass; this is the
    plain derivative of the forward definition.  Pinned by central finite differences.
    Returns (dx [T,d], dgates [T,K], dw1 [E,f,d], dw3 [E,f,d], dw2 [E,d,f]) in the weights' layout.
    """
    ids = np.asarray(topk_ids)
    T, K = ids.shape
    X = bf16_bits_to_f64(x_bits)
    G = np.asarray(gates, np.float64)
    dO = np.asarray(d_out, np.float64)
    dx = np.zeros_like(X)
    dg = np.zeros((T, K), np.float64)
    dw1 = np.zeros(w1_bits.shape, np.float64)
    dw3 = np.zeros(w3_bits.shape, np.float64)
    dw2 = np.zeros(w2_bits.shape, np.float64)
    for e in range(E):
        tt, kk = np.nonzero(ids == e)
        if tt.size == 0:
            continue
        W1 = bf16_bits_to_f64(w1_bits[e])      # [f, d]
        W3 = bf16_bits_to_f64(w3_bits[e])
        W2 = bf16_bits_to_f64(w2_bits[e])      # [d, f]
        Xe = X[tt]
        a = Xe @ W1.T
        b = Xe @ W3.T
        h = silu(a) * b
        y = h @ W2.T
        dy = G[tt, kk][:, None] * dO[tt]       # out = sum_k g * y
        dg[tt, kk] = np.sum(dO[tt] * y, axis=1)
        dh = dy @ W2
        dw2[e] = dy.T @ h
        da = dh * b * dsilu(a)
        db = dh * silu(a)
        dw1[e] = da.T @ Xe
        dw3[e] = db.T @ Xe
        np.add.at(dx, tt, da @ W1 + db @ W3)
    return dx, dg, dw1, dw3, dw2
