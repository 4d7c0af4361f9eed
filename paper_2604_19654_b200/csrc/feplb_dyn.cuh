// How a running grouped-GEMM launch learns the planner's table of dynamic groups (paper Section 2.3:
// the CPU balancer computes the plan while the GPU runs the static experts, so the launch that
// goes on from the static to the dynamic groups is enqueued before the table exists).
//
// The planner thread writes the table -- 32-byte entries {expert, row_start, rows, exec_rank,
// is_dynamic, seq, 0, 0} -- and then the word (seq << 32) | number of groups into mapped host
// memory.  Of the CTAs that have run out of static work, the first one claims the transfer: it alone
// polls that word across PCIe (reads of host memory from many SMs at once queue up behind one
// another), copies the table into device memory and sets a device-side word, which is what every
// other CTA, and the launch of the second pass, look at.  So the bounded wait depends on the host
// thread alone, never on another kernel.
//
// Polling loads are relaxed (they bypass L1 and order nothing) and no fence follows them: acquire
// loads and fences were measured to cost tens of microseconds each while the other SMs saturate the
// memory system.  Every table entry carries the sequence number instead; a reader that meets an
// entry without it looks again.
#ifndef FEPLB_DYN_CUH_
#define FEPLB_DYN_CUH_

#include <cuda_runtime.h>

#include "feplb_internal.h"
#include "feplb_tc.cuh"

namespace {

constexpr int kDynGaveUp = -1;   // "number of groups" of a ready word whose writer gave up waiting for the table
constexpr int kDynAbort = -2;    // the CTA is aborting

struct DynTable {
  int4* dyn_dev;                        // device copy of the table, made by the CTA that wins `claim` from ...
  const int4* dyn_host;                 // ... the planner's own table in mapped host memory
  unsigned long long* ready_dev;        // (seq << 32) | number of dynamic groups
  const unsigned long long* ready_host;
  uint32_t* claim;                      // device word: seq of the forward whose table transfer has been claimed
  int dyn_cap;                          // capacity of dyn_dev in groups
  uint32_t seq;                         // 0: no dynamic table in this launch
  unsigned long long wait_limit_ns;     // bound of the wait for the table
};

__device__ __forceinline__ unsigned long long ld_relaxed_gpu_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed_sys_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// Entry i of the device copy; false if it does not carry the sequence number (yet).
__device__ __forceinline__ bool dyn_entry(const DynTable& d, int i, int& expert, int& row_start, int& rows, int& is_dynamic) {
  const int4 lo = __ldcg(d.dyn_dev + 2 * i), hi = __ldcg(d.dyn_dev + 2 * i + 1);
  expert = lo.x; row_start = lo.y; rows = lo.z; is_dynamic = hi.x;
  return (uint32_t)hi.y == d.seq;
}

// The number of groups a peek at the device-side word shows, or -1 if the word is not this forward's.
__device__ __forceinline__ int dyn_peek_count(const DynTable& d, unsigned long long word) {
  return (uint32_t)(word >> 32) == d.seq && (int)(uint32_t)word != kDynGaveUp ? (int)(uint32_t)word : -1;
}

// Warp-collective, called by a CTA that has nothing left to do without the table.  Waits (bounded by
// wait_limit_ns from t0; CTAs that did not win the claim wait kWaitLimitNs longer, so that the
// claimer's verdict reaches them first) until the device copy of the table is in place, making it
// itself if this CTA wins the claim.  Returns the number of groups, kDynGaveUp (FEPLB_ST_PLAN has
// been raised; go on as if the table were empty) or kDynAbort.
__device__ __forceinline__ int dyn_wait_table(const DynTable& d, int lane, volatile int* abort_flag, uint32_t* status,
                                              unsigned long long t0, bool& claimer, bool& tried_claim) {
  unsigned long long v = 0;
  int got = 0;                       // 1: the device copy is there; 2: this CTA must make it; 3: gave up; 4: abort
  if (lane == 0) {
    for (;;) {
      v = ld_relaxed_gpu_u64(d.ready_dev);
      if ((uint32_t)(v >> 32) == d.seq) { got = 1; break; }
      if (!tried_claim) {
        tried_claim = true;
        const uint32_t cur = *reinterpret_cast<volatile uint32_t*>(d.claim);
        claimer = cur != d.seq && atomicCAS(d.claim, cur, d.seq) == cur;
      }
      if (claimer) {
        v = ld_relaxed_sys_u64(d.ready_host);
        if ((uint32_t)(v >> 32) == d.seq) { got = 2; break; }
      }
      if (*abort_flag) { got = 4; break; }
      if (global_timer_ns() - t0 > d.wait_limit_ns + (claimer ? 0ull : kWaitLimitNs)) {
        atomicOr(status, FEPLB_ST_PLAN);
        got = 3;
        break;
      }
      __nanosleep(claimer ? 100 : 400);
    }
  }
  got = __shfl_sync(0xffffffffu, got, 0);
  if (got == 4) return kDynAbort;
  int n_dyn = __shfl_sync(0xffffffffu, (int)(uint32_t)v, 0);
  if (got == 3) {
    // tell the others (and the second pass) that no table came within the limit
    if (lane == 0 && claimer)
      asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(d.ready_dev),
                   "l"(((unsigned long long)d.seq << 32) | (uint32_t)kDynGaveUp) : "memory");
    return kDynGaveUp;
  }
  if (got == 1) {
    if (n_dyn == kDynGaveUp && lane == 0) atomicOr(status, FEPLB_ST_PLAN);
    return n_dyn;
  }
  // got == 2: bring the table over.  Ordinary (weak) 16-byte loads coalesce into a few PCIe reads;
  // entries that do not carry the sequence number yet are read again.
  if (n_dyn < 0 || n_dyn > d.dyn_cap) {
    if (lane == 0) atomicOr(status, FEPLB_ST_GROUP);
    n_dyn = 0;
  }
  bool good = false;
  for (int attempt = 0; attempt < 64 && !good; ++attempt) {
    good = true;
    for (int i = lane; i < n_dyn; i += 32) {
      const int4 lo = __ldcv(d.dyn_host + 2 * i), hi = __ldcv(d.dyn_host + 2 * i + 1);
      if ((uint32_t)hi.y != d.seq) { good = false; continue; }
      d.dyn_dev[2 * i] = lo;
      d.dyn_dev[2 * i + 1] = hi;
    }
    good = __all_sync(0xffffffffu, good);
  }
  if (!good) {
    if (lane == 0) atomicOr(status, FEPLB_ST_GROUP);
    n_dyn = 0;
  }
  __syncwarp();                      // the lanes' stores happen before lane 0's release below
  if (lane == 0)
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(d.ready_dev),
                 "l"(((unsigned long long)d.seq << 32) | (uint32_t)n_dyn) : "memory");
  return n_dyn;
}

// Kernel parameter from the host-side description.
inline DynTable feplb_dyn_table(const feplb_wm_dyn& dyn) {
  DynTable d;
  d.dyn_dev = reinterpret_cast<int4*>(dyn.table_dev);
  d.dyn_host = reinterpret_cast<const int4*>(dyn.table_host);
  d.ready_dev = dyn.ready_dev;
  d.ready_host = dyn.ready_host;
  d.claim = dyn.claim;
  d.dyn_cap = dyn.max_groups;
  d.seq = dyn.seq;
  d.wait_limit_ns = dyn.wait_limit_ns ? dyn.wait_limit_ns : kWaitLimitNs;
  return d;
}

}  // namespace

#endif  // FEPLB_DYN_CUH_
