// Host-side steps of the FEPLB hot path: the static/dynamic partition and the greedy
// per-micro-batch load balancer (paper Section 2.3).  Pure C++, no CUDA: the planner thread of
// the library and callers without a GPU run exactly this code.
#include <algorithm>
#include <climits>
#include <cstdint>
#include <vector>

#include "feplb.h"
#include "feplb_internal.h"

int feplb_validate_config(const feplb_config* c) {
  if (!c) return FEPLB_E_INVALID;
  if (c->T < 0 || c->K < 1 || c->K > 32 || c->E < 1 || c->E > FEPLB_MAX_EXPERTS || c->R < 1) return FEPLB_E_INVALID;
  if (c->E % c->R) return FEPLB_E_INVALID;
  if (c->d < 128 || c->d % 128 || c->f < 64 || c->f % 64) return FEPLB_E_INVALID;
  if (c->row_align != 1 && c->row_align != 128) return FEPLB_E_INVALID;
  if (c->split_granule < 1 || c->max_num_dyn < 0 || c->tau < 0 || c->dyn < 0) return FEPLB_E_INVALID;
  if (c->ranks_per_domain < 0 || (c->ranks_per_domain > 0 && c->R % c->ranks_per_domain)) return FEPLB_E_INVALID;
  if (c->policy != FEPLB_POLICY_LITERAL && c->policy != FEPLB_POLICY_FIRST_FIT) return FEPLB_E_INVALID;
  if (c->split != 0 && c->split != 1) return FEPLB_E_INVALID;
  if (c->mask_policy != FEPLB_MASK_GIVEN && c->mask_policy != FEPLB_MASK_REACTIVE) return FEPLB_E_INVALID;
  if (c->phase2_copy != 0 && c->phase2_copy != 1) return FEPLB_E_INVALID;
  if ((int64_t)c->T * c->K + (int64_t)c->E * (c->row_align - 1) > INT32_MAX) return FEPLB_E_INVALID;
  return FEPLB_OK;
}

extern "C" size_t feplb_s_pad(const feplb_config* c) {
  if (feplb_validate_config(c) != FEPLB_OK) return 0;
  return (size_t)c->T * c->K + (size_t)c->E * (c->row_align - 1);
}

extern "C" int feplb_select_dynamic(const int64_t* score, int32_t E, int32_t R, int32_t dyn, uint8_t* mask_out) {
  if (!score || !mask_out || E < 1 || R < 1 || E % R || dyn < 0) return FEPLB_E_INVALID;
  const int L = E / R;
  // An expert is dynamic iff fewer than `dyn` experts of its block beat it
  // (higher score, or equal score and lower id).
  for (int e = 0; e < E; ++e) {
    const int b0 = e / L * L;
    int better = 0;
    for (int o = b0; o < b0 + L; ++o)
      better += (score[o] > score[e]) || (score[o] == score[e] && o < e);
    mask_out[e] = better < dyn ? 1 : 0;
  }
  return FEPLB_OK;
}

extern "C" int feplb_plan(const feplb_config* cfg, const int32_t* counts, const uint8_t* dyn_mask, feplb_plan_out* out) {
  int rc = feplb_validate_config(cfg);
  if (rc != FEPLB_OK) return rc;
  if (!counts || !dyn_mask || !out || !out->load_before || !out->load_after) return FEPLB_E_INVALID;
  if ((out->cap_moves > 0 && !out->moves) || (out->cap_groups > 0 && !out->groups)) return FEPLB_E_INVALID;
  const int E = cfg->E, R = cfg->R, L = E / R;
  const int D = cfg->ranks_per_domain > 0 ? cfg->ranks_per_domain : R;
  const int64_t thr = std::max<int64_t>(cfg->tau, 1);
  const int64_t g = cfg->split_granule;
  const bool split = cfg->split != 0;
  for (int e = 0; e < E; ++e)
    if (counts[e] < 0) return FEPLB_E_INVALID;

  std::vector<int64_t> load(R, 0), rem(E);
  std::vector<int> used(R, 0);
  std::vector<uint8_t> moved(E, 0);
  std::vector<uint8_t> pair_used((size_t)E * R, 0);   // (expert, dst) already served
  for (int e = 0; e < E; ++e) { rem[e] = counts[e]; load[e / L] += counts[e]; }
  for (int r = 0; r < R; ++r) out->load_before[r] = load[r];

  int n_moves = 0;
  std::vector<int> cand;
  cand.reserve(L);
  for (int base = 0; base < R; base += D) {
    int64_t total = 0;
    for (int r = base; r < base + D; ++r) total += load[r];
    const int64_t mean_up = (total + D - 1) / D;       // ceil of the domain's mean load
    for (;;) {
      // most loaded rank of the domain (lowest id on ties)
      int src = base;
      for (int r = base + 1; r < base + D; ++r)
        if (load[r] > load[src]) src = r;
      if (split && load[src] <= mean_up) break;
      // least loaded rank that can still receive (lowest id on ties)
      int dst = -1;
      for (int r = base; r < base + D; ++r) {
        if (r == src || used[r] >= cfg->max_num_dyn) continue;
        if (split && load[r] >= mean_up) continue;
        if (dst < 0 || load[r] < load[dst]) dst = r;
      }
      if (dst < 0) break;
      const int64_t gap = load[src] - load[dst];
      if (gap <= 0) break;
      // eligible dynamic experts of the source, busiest first (lower id on ties)
      cand.clear();
      for (int e = src * L; e < (src + 1) * L; ++e)
        if (dyn_mask[e] && !moved[e] && rem[e] >= thr && !pair_used[(size_t)e * R + dst]) cand.push_back(e);
      std::stable_sort(cand.begin(), cand.end(), [&](int a, int b) { return rem[a] > rem[b]; });
      int pick = -1;
      int64_t rows = 0;
      for (int e : cand) {
        if (!split) {
          if (rem[e] < gap) { pick = e; rows = rem[e]; break; }
        } else {
          int64_t m = std::min(rem[e], std::min(load[src] - mean_up, mean_up - load[dst]));
          if (m < rem[e]) m = m / g * g;
          if (m >= thr) { pick = e; rows = m; break; }
        }
        if (cfg->policy == FEPLB_POLICY_LITERAL) break;
      }
      if (pick < 0) break;
      if (n_moves >= out->cap_moves) return FEPLB_E_NOMEM;
      if (!split) moved[pick] = 1;
      rem[pick] -= rows;
      load[src] -= rows;
      load[dst] += rows;
      used[dst] += 1;
      pair_used[(size_t)pick * R + dst] = 1;
      out->moves[n_moves++] = feplb_move{pick, src, dst, (int32_t)rows};
    }
  }
  out->n_moves = n_moves;
  for (int r = 0; r < R; ++r) out->load_after[r] = load[r];

  // Group table in expert order: moved pieces from the front of the segment, then the remainder.
  const int A = cfg->row_align;
  int n_groups = 0;
  int64_t off = 0;
  for (int e = 0; e < E; ++e) {
    int64_t p = off;
    for (int i = 0; i < n_moves; ++i) {
      if (out->moves[i].expert != e) continue;
      if (n_groups >= out->cap_groups) return FEPLB_E_NOMEM;
      out->groups[n_groups++] = feplb_group{e, (int32_t)p, out->moves[i].rows, out->moves[i].dst, dyn_mask[e] ? 1 : 0};
      p += out->moves[i].rows;
    }
    if (rem[e] > 0) {
      if (n_groups >= out->cap_groups) return FEPLB_E_NOMEM;
      out->groups[n_groups++] = feplb_group{e, (int32_t)p, (int32_t)rem[e], e / L, dyn_mask[e] ? 1 : 0};
    }
    off += ((int64_t)counts[e] + A - 1) / A * A;
  }
  out->n_groups = n_groups;
  return FEPLB_OK;
}

extern "C" int feplb_ep_schedule(const feplb_config* cfg, const int32_t* counts_by_src, const uint8_t* dyn_mask, int32_t rank,
                                 feplb_plan_out* plan, int64_t* p1_send, int64_t* p1_recv, int64_t* p2_send, int64_t* p2_recv,
                                 int64_t* comb_send, int64_t* comb_recv, feplb_weight_copy* copies, int32_t cap_copies,
                                 int32_t* n_copies) {
  int rc = feplb_validate_config(cfg);
  if (rc != FEPLB_OK) return rc;
  if (!counts_by_src || !dyn_mask || !plan || rank < 0 || rank >= cfg->R) return FEPLB_E_INVALID;
  const int E = cfg->E, R = cfg->R, L = E / R;
  std::vector<int32_t> counts(E, 0);
  for (int s = 0; s < R; ++s)
    for (int e = 0; e < E; ++e) {
      const int32_t c = counts_by_src[(size_t)s * E + e];
      if (c < 0 || (int64_t)counts[e] + c > INT32_MAX) return FEPLB_E_INVALID;
      counts[e] += c;
    }
  if ((rc = feplb_plan(cfg, counts.data(), dyn_mask, plan)) != FEPLB_OK) return rc;
  auto zero = [&](int64_t* a) { if (a) std::fill(a, a + R, (int64_t)0); };
  zero(p1_send); zero(p1_recv); zero(p2_send); zero(p2_recv); zero(comb_send); zero(comb_recv);
  // Phase 1: every source sends each expert's rows to the expert's home
  for (int e = 0; e < E; ++e) {
    if (p1_send) p1_send[e / L] += counts_by_src[(size_t)rank * E + e];
    if (p1_recv && e / L == rank)
      for (int s = 0; s < R; ++s) p1_recv[s] += counts_by_src[(size_t)s * E + e];
  }
  // Phase 2 and the combine: walk every expert's segment piece by piece (moved pieces from the
  // front, in move order, then the home remainder) and split each piece by source rank
  std::vector<int> next_slot(R, 0);
  int nc = 0;
  for (int i = 0; i < plan->n_moves; ++i) {
    const feplb_move& m = plan->moves[i];
    if (p2_send && m.src == rank) p2_send[m.dst] += m.rows;
    if (p2_recv && m.dst == rank) p2_recv[m.src] += m.rows;
    if (copies) {
      if (nc >= cap_copies) return FEPLB_E_NOMEM;
      copies[nc] = feplb_weight_copy{m.expert, m.src, m.dst, m.dst * cfg->max_num_dyn + next_slot[m.dst],
                                     m.rows, (int64_t)3 * cfg->d * cfg->f * 2};
    }
    ++next_slot[m.dst];
    ++nc;
  }
  if (n_copies) *n_copies = nc;
  std::vector<int64_t> seg_pos(E, 0);              // rows of expert e already handed out
  for (int gi = 0; gi < plan->n_groups; ++gi) {
    const feplb_group& g = plan->groups[gi];       // groups of one expert come in segment order
    const int e = g.expert;
    int64_t a = seg_pos[e], b = a + g.rows, off = 0;
    seg_pos[e] = b;
    for (int s = 0; s < R; ++s) {                  // source s owns [off, off + c) of the segment
      const int64_t c = counts_by_src[(size_t)s * E + e];
      const int64_t lo = std::max(a, off), hi = std::min(b, off + c);
      if (hi > lo) {
        if (comb_send && g.exec_rank == rank) comb_send[s] += hi - lo;
        if (comb_recv && s == rank) comb_recv[g.exec_rank] += hi - lo;
      }
      off += c;
    }
  }
  return FEPLB_OK;
}

extern "C" int feplb_ema_update(double* ema, const int32_t* counts, int32_t E, double decay) {
  if (!ema || !counts || E < 1 || !(decay >= 0.0 && decay <= 1.0)) return FEPLB_E_INVALID;
  for (int e = 0; e < E; ++e) ema[e] = decay * ema[e] + (1.0 - decay) * (double)counts[e];
  return FEPLB_OK;
}

extern "C" int feplb_place_experts(const double* load, int32_t E, int32_t R, int32_t* new_index) {
  if (!load || !new_index || E < 1 || R < 1 || E % R) return FEPLB_E_INVALID;
  const int L = E / R;
  std::vector<int> order(E);
  for (int e = 0; e < E; ++e) order[e] = e;
  // heaviest first, lower id on ties
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return load[a] > load[b]; });
  std::vector<double> rank_load(R, 0.0);
  std::vector<int> fill(R, 0);
  for (int e : order) {
    int best = -1;   // least loaded rank with room, lowest id on ties
    for (int r = 0; r < R; ++r)
      if (fill[r] < L && (best < 0 || rank_load[r] < rank_load[best])) best = r;
    new_index[e] = best * L + fill[best];
    fill[best] += 1;
    rank_load[best] += load[e];
  }
  return FEPLB_OK;
}
