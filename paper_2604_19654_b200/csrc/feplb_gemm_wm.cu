// Grouped SwiGLU expert FFN, "weights on M" form, for sm_100a (paper Section 2.3: static-expert,
// then dynamic-expert Grouped GEMM; Section 3.1: grouped GEMM over per-expert row segments whose
// cost is very sensitive to the per-expert batch size).
//
// The other form of this library (feplb_gemm.cu) puts 128 or 256 token rows on the M side of the
// MMA and the expert's weights on the N side, which wastes up to 127 (255) rows of every segment's
// last tile and reads an expert's weights from L2 once per 128 (256) rows.  Here the roles are
// exchanged, and a cluster of two CTAs (tcgen05 cta_group::2) works on one unit:
//
//   unit   = (row block of one group: n <= 256 rows, padded to a multiple of 32)
//          x (256 weight rows of the group's expert, 128 per CTA)
//   pass 1 : CTA r holds 64 rows of W1[e] followed by the same 64 rows of W3[e] (hidden units
//            u0 + 64 r ...), both CTAs stage half of the block's token rows each;
//            D = [W1; W3] X^T, so TMEM lanes 0-63 of a CTA hold a = x W1, lanes 64-127 b = x W3 of the
//            same 64 hidden units; H[rows, units] = silu(a) * b                (transposed store)
//   pass 2 : CTA r holds W2[e][c0 + 128 r : +128, :], B = H[rows, :];  Y[rows, c0 : c0 + 256] = D^T
//
// Per 64-wide K step a CTA moves 16 KiB of weights plus 64 bytes per token row for its half of a
// 256 x n x 64 MMA: an expert's weights cross the L2 ports once per <= 256 rows, a segment's ragged
// tail costs at most 31 padded rows, the accumulator of a unit takes n <= 256 of the 512 TMEM
// columns (two units in flight: the epilogue of one overlaps the MMAs of the next) and the operand
// ring holds five stages of 32 KiB, each filled by two or three TMA instructions (every instruction
// was measured to cost about a hundred cycles on top of its bytes, so the token rows come as one
// box of 16, 32, 64 or 128 rows).  Per CTA: warp 0 = TMA producer, warp 1 = tcgen05.mma issuer
// (even CTA only) and TMEM owner, warps 2..9 = epilogue.
//
// One launch walks TWO group tables in order: the table known at launch (static experts on their
// home ranks, built on the device from the counts) and then the planner's table of dynamic
// groups, which does not exist yet when the launch is enqueued (Section 2.3: the CPU balancer runs
// while the GPU computes the static experts).  A CTA that runs out of static units looks the
// dynamic table up with a bounded wait on a word in mapped host memory that the planner thread
// itself writes after the table (no kernel waits for another kernel); the first CTA to see it copies
// the table into device memory for all the others.  Every wait is bounded and ends in a status bit,
// a clean TMEM release and a normal return.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>

#include "feplb_internal.h"
#include "feplb_tc.cuh"
#include "feplb_dyn.cuh"

namespace {

constexpr int WM = 128;                 // weight rows per CTA (UMMA M = 256 over the pair)
constexpr int BK = 64;                  // K elements per stage = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int kNMax = 256;              // token rows per unit (UMMA N), half of them staged by each CTA
constexpr int kATile = WM * BK * 2;     // 16 KiB
constexpr int kBHalf = kNMax / 2 * BK * 2;          // 16 KiB
constexpr int kStageBytes = kATile + kBHalf;        // 32 KiB
constexpr int kStages = 5;
constexpr int kRingBytes = kStages * kStageBytes;   // 160 KiB
constexpr int kAccCols = 256;           // TMEM columns of one accumulator
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 8;            // two warps per TMEM lane quarter
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kEpiStageBytes = 32 * 64; // per epilogue warp: 32 tokens x 32 units of bf16
constexpr int kXchgBytes = 32 * 32 * 4; // per pair of epilogue warps (pass 1): 32 tokens x 32 units of fp32
constexpr int kXchg = 4;
constexpr int kMaxEntries = FEPLB_WM_MAX_ENTRIES;   // group entries of both tables together
constexpr int kBoxes = 4;               // token-row boxes of 128, 64, 32 and 16 rows

struct Tail {
  unsigned long long full[kStages];     // leader's: operand bytes of both CTAs
  unsigned long long empty[kStages];    // own: the leader's MMAs have read this CTA's stage
  unsigned long long tmem_full[2];      // own: accumulator complete (committed by the leader to both CTAs)
  unsigned long long tmem_empty[2];     // leader's: epilogue warps of both CTAs have read the accumulator
  unsigned long long xfull[kXchg];      // pass 1: b values of a chunk are in the exchange buffer
  unsigned long long xempty[kXchg];     // ... and have been taken out again
  unsigned long long dyn_bar;           // completed by warp 0 once the dynamic entries are in place
  uint32_t tmem_base;
  int abort_flag;
  int n_entries;                        // entries in use (static, then dynamic)
  int total_units;                      // prefix[n_entries]
  int prefix[kMaxEntries + 1];          // prefix[g] = units of the entries before g
  int row_start[kMaxEntries];
  int rows[kMaxEntries];
  int expert[kMaxEntries];              // expert id | (receive slot + 1) << 16
};
constexpr size_t kSmemBytes = 1024 + (size_t)kRingBytes + (size_t)kEpiWarps * kEpiStageBytes + (size_t)kXchg * kXchgBytes +
                              sizeof(Tail);
static_assert(kSmemBytes <= 232448, "shared memory budget");
static_assert(kSmemBytes > 116 * 1024, "one CTA per SM: each allocates all of TMEM");

struct BMaps { CUtensorMap m[kBoxes]; };

struct WmParams {
  const feplb_group* groups;            // table known at launch
  int n_groups;
  int which;                            // FEPLB_FFN_* filter on that table
  DynTable dyn;                         // the planner's table of dynamic groups (dyn.seq == 0: none in this launch)
  int E;
  int64_t s_cap;
  int n_pairs;                          // 256-row weight blocks per row block (pass 1: 128 hidden units each)
  int num_k_blocks;
  int a_rows_per_expert;                // rows of one expert in the weight maps
  int unit_rows;                        // weight-map rows a unit advances by: 128 (pass 1, in W1 and in W3) or 256 (pass 2)
  int cta_rows;                         // ... and the second CTA's offset inside it: 64 or 128
  int a1_row_off;                       // row offset of a CTA's second 64-row box inside the same map (pass 2: 64), 0 in pass 1
  int n_recv_slots;
  __nv_bfloat16* out;
  int ld_out;
  __nv_bfloat16* ab_out;                // pass 1, optional: pre-activations a | b ([rows, 2f])
  uint32_t* status;
  unsigned long long* stamps;           // optional, preset to all ones, globaltimer ns: [0] first CTA's start, [1] first
                                        // time a CTA ran out of static units, [2] ~(last CTA's end), [3] ~(longest
                                        // wait for the dynamic table); the last two are kept complemented so that
                                        // one atomicMin and one memset pattern serve all four
};

struct Unit { int row0, n_rows, n_pad, expert, slot, wt; };

__device__ __forceinline__ int units_of(int rows, int n_pairs) { return (rows + kNMax - 1) / kNMax * n_pairs; }

// unit -> (entry, row block, weight block).  The weight blocks of one row block are consecutive, so
// clusters running at the same time share the block's rows in L2 and sweep the expert's weights once.
__device__ __forceinline__ Unit unit_coord(const Tail* t, int n_entries, int n_pairs, int u) {
  int lo = 0, hi = n_entries;            // largest g with prefix[g] <= u
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (t->prefix[mid] <= u) lo = mid; else hi = mid;
  }
  const int local = u - t->prefix[lo];
  const int blk = local / n_pairs;
  const int rows = t->rows[lo];
  const int nb = (rows + kNMax - 1) / kNMax;
  const int bs = ((rows + nb - 1) / nb + 31) & ~31;      // rows per block, a multiple of 32, <= 256
  Unit c;
  c.wt = local - blk * n_pairs;
  c.row0 = t->row_start[lo] + blk * bs;
  c.n_rows = min(bs, rows - blk * bs);
  c.n_pad = (c.n_rows + 31) & ~31;
  c.expert = t->expert[lo] & 0xffff;
  c.slot = (t->expert[lo] >> 16) - 1;
  return c;
}

// One entry of a group table -> shared-memory arrays; returns its number of units (0 if not selected).
__device__ __forceinline__ int put_entry(Tail* t, int idx, int expert, int row_start, int rows, int is_dynamic, bool selected,
                                         const WmParams& p) {
  int units = 0;
  if (selected && rows > 0) {
    const bool ok = expert >= 0 && expert < p.E && row_start >= 0 && (int64_t)row_start + rows <= p.s_cap &&
                    is_dynamic - 2 < p.n_recv_slots;
    if (ok) units = units_of(rows, p.n_pairs);
    else atomicOr(p.status, FEPLB_ST_GROUP);
  }
  t->row_start[idx] = row_start;
  t->rows[idx] = rows;
  t->expert[idx] = (expert & 0xffff) | ((is_dynamic >= 2 ? is_dynamic - 1 : 0) << 16);
  return units;
}

// In-place inclusive scan of t->prefix[first+1 .. first+n] (unit counts) by one warp; prefix[first] is the base.
__device__ __forceinline__ void warp_scan_prefix(Tail* t, int first, int n, int lane) {
  const int per = (n + 31) / 32;
  const int g0 = min(n, lane * per), g1 = min(n, g0 + per);
  int sum = 0;
  for (int g = g0; g < g1; ++g) sum += t->prefix[first + g + 1];
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  int run = t->prefix[first] + incl - sum;
  __syncwarp();
  for (int g = g0; g < g1; ++g) {
    run += t->prefix[first + g + 1];
    t->prefix[first + g + 1] = run;
  }
  __syncwarp();
}

// 32 values of one weight row (this lane) for 32 consecutive token rows -> global rows, transposed
// through the warp's staging area: token j at byte j*64, this lane's unit at +lane*2; read back in
// 16-byte pieces, 8 tokens per instruction, so that a token's 32 units leave as one 64-byte run.
__device__ __forceinline__ void store_transposed(uint32_t stg, const float (&v)[32], __nv_bfloat16* out, int64_t ld, int n_valid,
                                                 int lane) {
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const unsigned short h = __bfloat16_as_ushort(__float2bfloat16_rn(v[j]));
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(stg + (uint32_t)(j * 64 + lane * 2)), "h"(h) : "memory");
  }
  __syncwarp();
  const int tj = lane >> 2, piece = lane & 3;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int j = it * 8 + tj;
    uint4 w;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w)
                 : "r"(stg + (uint32_t)(j * 64 + piece * 16)));
    if (j < n_valid) *reinterpret_cast<uint4*>(out + (int64_t)j * ld + piece * 8) = w;
  }
  __syncwarp();
}

template <bool SWIGLU>
__global__ void __launch_bounds__(kThreads, 1)
k_ffn_wm(const __grid_constant__ CUtensorMap tm_a0, const __grid_constant__ CUtensorMap tm_a1,
         const __grid_constant__ CUtensorMap tm_r0, const __grid_constant__ CUtensorMap tm_r1,
         const __grid_constant__ BMaps tm_b, const __grid_constant__ BMaps tm_rb, const WmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* epi_smem = smem + (size_t)kRingBytes;
  uint8_t* xchg_smem = epi_smem + (size_t)kEpiWarps * kEpiStageBytes;
  Tail* tail = reinterpret_cast<Tail*>(xchg_smem + (size_t)kXchg * kXchgBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t cta_rank = cluster_ctarank();          // 0 = leader: issues the MMAs of the pair
  const int worker = (int)(blockIdx.x >> 1), n_workers = (int)(gridDim.x >> 1);
  volatile int* abort_flag = &tail->abort_flag;
  const bool has_dyn = p.dyn.seq != 0;

  asm volatile("griddepcontrol.launch_dependents;");

  // ---- set-up: barriers, TMEM, the table known at launch -----------------------------------------
  if (threadIdx.x == 0) {
    prefetch_tmap(&tm_a0);
    prefetch_tmap(&tm_a1);
    for (int i = 0; i < kBoxes; ++i) prefetch_tmap(&tm_b.m[i]);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&tail->full[s]), 1);
      mbar_init(smem_u32(&tail->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&tail->tmem_full[a]), 1);
      mbar_init(smem_u32(&tail->tmem_empty[a]), 2 * kEpiWarps);   // the leader's collects both CTAs' epilogue warps
    }
    for (int x = 0; x < kXchg; ++x) {
      mbar_init(smem_u32(&tail->xfull[x]), 1);
      mbar_init(smem_u32(&tail->xempty[x]), 1);
    }
    mbar_init(smem_u32(&tail->dyn_bar), 1);
    tail->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    __syncwarp();
    tmem_alloc_pair(smem_u32(&tail->tmem_base), kTmemCols);
    tmem_relinquish_pair();
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (p.stamps && threadIdx.x == 0) atomicMin(&p.stamps[0], global_timer_ns());
  for (int g = threadIdx.x; g < p.n_groups; g += kThreads) {
    const feplb_group gr = p.groups[g];
    const bool selected = p.which == FEPLB_FFN_ALL || (p.which == FEPLB_FFN_STATIC) == (gr.is_dynamic == 0);
    tail->prefix[g + 1] = put_entry(tail, g, gr.expert, gr.row_start, gr.rows, gr.is_dynamic, selected, p);
  }
  if (threadIdx.x == 0) tail->prefix[0] = 0;
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    warp_scan_prefix(tail, 0, p.n_groups, lane);
    if (lane == 0) {
      tail->n_entries = p.n_groups;
      tail->total_units = tail->prefix[p.n_groups];
    }
  }
  __syncthreads();
  cluster_sync_all();                    // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tail->tmem_base;
  const int n_static_entries = p.n_groups;
  const int n_static_units = tail->prefix[p.n_groups];

  if (warp == 0) {
    // ---- TMA producer (lane 0 issues; the whole warp fetches the dynamic table) --------------------
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true, dyn_known = !has_dyn;
    int n_entries = n_static_entries, total = n_static_units;
    // Reads the n_dyn groups of the dynamic table from its device copy, appends its entries and tells
    // the other roles.  Every 32-byte entry carries the forward's sequence number, so no fence is
    // needed between seeing the ready word and reading the table: an entry that does not carry the
    // number yet makes the call return false, and the caller looks again.
    auto take_table = [&](int n_dyn) -> bool {
      if (n_dyn < 0 || n_static_entries + n_dyn > kMaxEntries) {
        if (lane == 0) atomicOr(p.status, FEPLB_ST_GROUP);
        n_dyn = 0;
      }
      bool good = true;
      for (int i = lane; i < n_dyn; i += 32) {
        int e, rs, rw, dy;
        if (!dyn_entry(p.dyn, i, e, rs, rw, dy)) { good = false; continue; }
        tail->prefix[n_static_entries + i + 1] = put_entry(tail, n_static_entries + i, e, rs, rw, dy, true, p);
      }
      if (!__all_sync(0xffffffffu, good)) return false;
      warp_scan_prefix(tail, n_static_entries, n_dyn, lane);
      n_entries = n_static_entries + n_dyn;
      total = tail->prefix[n_entries];
      if (lane == 0) {
        tail->n_entries = n_entries;
        tail->total_units = total;
        mbar_arrive(smem_u32(&tail->dyn_bar));      // release: the entries above are visible to the waiters
      }
      dyn_known = true;
      return true;
    };
    bool claimer = false, tried_claim = false;
    for (int u = worker; ok; u += n_workers) {
      if (!dyn_known && u >= total) {
        // Out of static units: now the table is needed (bounded wait; see feplb_dyn.cuh).
        const unsigned long long t0 = global_timer_ns();
        if (p.stamps && lane == 0) atomicMin(&p.stamps[1], t0);
        while (!dyn_known) {
          const int n_dyn = dyn_wait_table(p.dyn, lane, abort_flag, p.status, t0, claimer, tried_claim);
          if (n_dyn == kDynAbort) { ok = false; break; }
          // no table within the limit: go on as if it were empty, so that the static units still in
          // flight complete normally; the status word carries the reason
          if (!take_table(n_dyn == kDynGaveUp ? 0 : n_dyn) && global_timer_ns() - t0 > p.dyn.wait_limit_ns + kWaitLimitNs) {
            if (lane == 0) atomicOr(p.status, FEPLB_ST_PLAN);
            take_table(0);
          }
        }
        if (!ok) break;
        if (p.stamps && lane == 0) atomicMin(&p.stamps[3], ~(global_timer_ns() - t0));
      }
      if (u >= total) break;
      const Unit c = unit_coord(tail, n_entries, p.n_pairs, u);
      // While static units remain, peek at the device-side word once per unit: the load is in flight
      // during the K loop below and is looked at after it, so it costs the pipeline nothing.
      unsigned long long peek = 0;
      if (!dyn_known && lane == 0) peek = ld_relaxed_gpu_u64(p.dyn.ready_dev);
      if (lane == 0) {
        const CUtensorMap* ma0 = c.slot >= 0 ? &tm_r0 : &tm_a0;
        const CUtensorMap* ma1 = c.slot >= 0 ? &tm_r1 : &tm_a1;
        // this CTA's 128 weight rows as two boxes of 64: pass 1 W1 rows, then the same rows of W3;
        // pass 2 two consecutive boxes of W2
        const int arow0 = (c.slot >= 0 ? c.slot : c.expert) * p.a_rows_per_expert + c.wt * p.unit_rows + (int)cta_rank * p.cta_rows;
        const int arow1 = arow0 + p.a1_row_off;
        const int n_half = c.n_pad >> 1;                  // token rows this CTA stages
        const int brow0 = c.row0 + (int)cta_rank * n_half;
        // one box per operand and stage (every TMA instruction costs about a hundred cycles on top of its
        // bytes): the smallest of the 16/32/64/128-row boxes that covers this CTA's token rows; the rows
        // it brings beyond them land behind the rows the MMA reads
        int bi = kBoxes - 1;
        while (bi > 0 && ((kNMax / 2) >> bi) < n_half) --bi;
        const int brows = (kNMax / 2) >> bi;
        const uint32_t tx = (uint32_t)(2 * (kATile + brows * (BK * 2)));   // both CTAs credit the leader's barrier
        const uint32_t full0 = map_to_cta(smem_u32(&tail->full[0]), 0);
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->empty[stage]), phase ^ 1u, abort_flag, p.status))) break;
          const uint32_t full = full0 + (uint32_t)(stage * sizeof(unsigned long long));
          const uint32_t sa = smem_u32(smem + (size_t)stage * kStageBytes);
          if (cta_rank == 0) mbar_expect_tx(smem_u32(&tail->full[stage]), tx);
          if (SWIGLU) {
            tma_load_2d_pair(sa, ma0, full, kb * BK, arow0);                  // 64 rows of W1
            tma_load_2d_pair(sa + kATile / 2, ma1, full, kb * BK, arow1);     // the same 64 rows of W3
          } else {
            tma_load_2d_pair(sa, ma0, full, kb * BK, arow0);                  // 128 rows of W2
          }
          tma_load_2d_pair(sa + kATile, c.slot >= 0 ? &tm_rb.m[bi] : &tm_b.m[bi], full, kb * BK, brow0);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      if (ok && !dyn_known) {
        peek = __shfl_sync(0xffffffffu, peek, 0);
        if (dyn_peek_count(p.dyn, peek) >= 0) take_table(dyn_peek_count(p.dyn, peek));
      }
    }
    if (!ok && lane == 0) {
      for (int i = 0; i < 2000; ++i) __nanosleep(100);   // copies already issued land before the CTA's shared memory goes away
    }
  } else if (warp == 1) {
    // ---- MMA issuer (leader CTA only) ---------------------------------------------------------------
    if (lane == 0 && cta_rank == 0) {
      int stage = 0, as = 0;
      uint32_t phase = 0, aphase = 0;
      bool ok = true, dyn_known = !has_dyn;
      int n_entries = n_static_entries, total = n_static_units;
      for (int u = worker; ok; u += n_workers) {
        if (u >= total) {
          if (dyn_known) break;
          if (!(ok = mbar_wait(smem_u32(&tail->dyn_bar), 0, abort_flag, p.status, p.dyn.wait_limit_ns + 2 * kWaitLimitNs))) break;
          dyn_known = true;
          n_entries = tail->n_entries;
          total = tail->total_units;
          if (u >= total) break;
        }
        const Unit c = unit_coord(tail, n_entries, p.n_pairs, u);
        if (!(ok = mbar_wait(smem_u32(&tail->tmem_empty[as]), aphase ^ 1u, abort_flag, p.status))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * kAccCols);
        const uint32_t idesc = make_idesc(2 * WM, c.n_pad);
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->full[stage]), phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)stage * kStageBytes);
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + kATile);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (uint32_t)((kb | k) != 0));
          umma_commit_pair(smem_u32(&tail->empty[stage]));      // both CTAs' stages are free once these MMAs have read them
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(smem_u32(&tail->tmem_full[as]));       // accumulator complete, announced to both CTAs
        if (++as == 2) { as = 0; aphase ^= 1u; }
      }
    }
  } else {
    // ---- epilogue: TMEM -> registers -> (SwiGLU) -> bf16 -> transposed rows in global memory ---------
    // A thread owns one weight row of its CTA and gets 32 token rows per tcgen05.ld; two warps share
    // each TMEM lane quarter and take alternate chunks of 32 tokens.  Pass 1: lanes 0-63 hold a, lanes
    // 64-127 b of the same 64 hidden units, so the warps of quarters 2 and 3 hand their b values to the
    // warps of quarters 0 and 1 through an exchange buffer (fp32), and those compute and store H.
    const int q = warp & 3;                      // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;            // 0: even chunks of 32 tokens, 1: odd chunks
    const bool gives_b = SWIGLU && q >= 2;
    const int x = half * 2 + (q & 1);            // exchange buffer of this warp and its partner
    const uint32_t stg = smem_u32(epi_smem + (size_t)(warp - 2) * kEpiStageBytes);
    const uint32_t xb = smem_u32(xchg_smem + (size_t)x * kXchgBytes);
    const uint32_t xfull = smem_u32(&tail->xfull[x]), xempty = smem_u32(&tail->xempty[x]);
    const uint32_t empty0 = map_to_cta(smem_u32(&tail->tmem_empty[0]), 0);   // the leader's barriers
    uint32_t xphase = 0;
    int as = 0;
    uint32_t aphase = 0;
    bool ok = true, dyn_known = !has_dyn;
    int n_entries = n_static_entries, total = n_static_units;
    for (int u = worker; ok; u += n_workers) {
      if (u >= total) {
        if (dyn_known) break;
        ok = mbar_wait(smem_u32(&tail->dyn_bar), 0, abort_flag, p.status, p.dyn.wait_limit_ns + 2 * kWaitLimitNs);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        dyn_known = true;
        n_entries = tail->n_entries;
        total = tail->total_units;
        if (u >= total) break;
      }
      const Unit c = unit_coord(tail, n_entries, p.n_pairs, u);
      ok = mbar_wait(smem_u32(&tail->tmem_full[as]), aphase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * kAccCols);
      // pass 1: H[row, wt*128 + 64*rank + 32*(q&1) + lane];  pass 2: Y[row, wt*256 + 128*rank + 32*q + lane]
      const int col0 = SWIGLU ? c.wt * 128 + (int)cta_rank * 64 + (q & 1) * 32 : c.wt * 256 + (int)cta_rank * 128 + q * 32;
      const int n_chunks = c.n_pad >> 5;
      uint32_t r[32];
      int ch = half;
      if (ch < n_chunks) tmem_ld32(taddr + (uint32_t)(ch * 32), r);
      for (; ch < n_chunks && ok; ch += 2) {
        tmem_ld_wait();
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        if (ch + 2 < n_chunks) {                 // the next chunk's TMEM load flies while this one is converted and stored
          tmem_ld32(taddr + (uint32_t)((ch + 2) * 32), r);
        } else {
          // every TMEM read of this unit by this warp has completed: the accumulator may be overwritten
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(empty0 + (uint32_t)(as * sizeof(unsigned long long)));
        }
        const int r0 = c.row0 + ch * 32;
        const int n_valid = c.n_rows - ch * 32;  // valid token rows among this chunk's 32
        if (!SWIGLU) {
          store_transposed(stg, v, p.out + (int64_t)r0 * p.ld_out + col0, p.ld_out, n_valid, lane);
        } else if (gives_b) {
          ok = mbar_wait(xempty, xphase ^ 1u, abort_flag, p.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(xb + (uint32_t)(j * 128 + lane * 4)), "f"(v[j]) : "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(xfull);
          xphase ^= 1u;
          if (p.ab_out != nullptr)
            store_transposed(stg, v, p.ab_out + (int64_t)r0 * (2 * p.ld_out) + p.ld_out + col0, 2 * p.ld_out, n_valid, lane);
        } else {
          if (p.ab_out != nullptr)
            store_transposed(stg, v, p.ab_out + (int64_t)r0 * (2 * p.ld_out) + col0, 2 * p.ld_out, n_valid, lane);
          ok = mbar_wait(xfull, xphase, abort_flag, p.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            float b;
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(b) : "r"(xb + (uint32_t)(j * 128 + lane * 4)));
            v[j] = silu_f(v[j]) * b;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(xempty);
          xphase ^= 1u;
          store_transposed(stg, v, p.out + (int64_t)r0 * p.ld_out + col0, p.ld_out, n_valid, lane);
        }
      }
      if (!ok) break;
      if (half >= n_chunks) {                    // a unit of 32 rows: the odd-chunk warps read nothing, but they still hand the accumulator back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(empty0 + (uint32_t)(as * sizeof(unsigned long long)));
      }
      if (++as == 2) { as = 0; aphase ^= 1u; }
    }
  }

  // ---- teardown --------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (p.stamps && threadIdx.x == 0) atomicMin(&p.stamps[2], ~global_timer_ns());
  cluster_sync_all();                    // the leader's MMAs read the peer's shared memory: leave together
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------ host

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_fn() {
  static encode_tiled_fn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<encode_tiled_fn>(p);
  }
  return fn;
}

// Row-major bf16 matrix [rows, inner] -> tensor map with a [box_rows, 64] box, 128-byte swizzle.
bool make_tmap(CUtensorMap* m, const void* base, uint64_t rows, uint64_t inner, uint32_t box_rows) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_bmaps(BMaps* b, const void* base, uint64_t rows, uint64_t inner) {
  for (int i = 0; i < kBoxes; ++i)
    if (!make_tmap(&b->m[i], base, rows, inner, (uint32_t)((kNMax / 2) >> i))) return false;   // rows past the tensor read as zeros
  return true;
}

template <bool SWIGLU>
cudaError_t launch_wm(const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& r0, const CUtensorMap& r1,
                      const BMaps& b, const BMaps& rb, const WmParams& p, int num_sms, cudaStream_t st) {
  // per instantiation and device: the shared-memory attribute and the resident grid are set on first use
  static int grid_of[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int& grid = grid_of[dev];
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = 2;
  at[1].val.clusterDim.y = 1;
  at[1].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 2;
  if (!grid) {
    cudaError_t e = cudaFuncSetAttribute(k_ffn_wm<SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    // as many clusters of two as can be resident at once (one CTA per SM, both SMs in one GPC)
    int n_clusters = 0;
    cfg.gridDim = dim3(num_sms / 2 * 2);
    e = cudaOccupancyMaxActiveClusters(&n_clusters, k_ffn_wm<SWIGLU>, &cfg);
    if (e != cudaSuccess) return e;
    if (n_clusters < 1) return cudaErrorLaunchOutOfResources;
    grid = 2 * (n_clusters < num_sms / 2 ? n_clusters : num_sms / 2);
  }
  cfg.gridDim = dim3(grid);
  return cudaLaunchKernelEx(&cfg, k_ffn_wm<SWIGLU>, a0, a1, r0, r1, b, rb, p);
}

}  // namespace

bool feplb_wm_supported(int E, int d, int f, int n_entries_max) {
  return f % 128 == 0 && d % 256 == 0 && n_entries_max <= kMaxEntries && E <= 0xffff;
}

int feplb_launch_expert_ffn_wm(const feplb_gemm_args& a, const feplb_wm_dyn& dyn, cudaStream_t st, int64_t* n_launch,
                               char* err, size_t errn) {
  if ((a.n_groups == 0 && dyn.seq == 0) || a.s_cap == 0) return FEPLB_OK;
  if (!feplb_wm_supported(a.E, a.d, a.f, a.n_groups + dyn.max_groups)) {
    snprintf(err, errn, "expert_ffn: shape not supported by the weights-on-M form");
    return FEPLB_E_INVALID;
  }
  CUtensorMap tm_w1, tm_w3, tm_w2;      // weights in boxes of 64 rows
  BMaps bx, bh;
  if (!make_tmap(&tm_w1, a.w1, (uint64_t)a.E * a.f, (uint64_t)a.d, WM / 2) ||
      !make_tmap(&tm_w3, a.w3, (uint64_t)a.E * a.f, (uint64_t)a.d, WM / 2) ||
      !make_tmap(&tm_w2, a.w2, (uint64_t)a.E * a.d, (uint64_t)a.f, WM) ||
      !make_bmaps(&bx, a.x_perm, (uint64_t)a.s_cap, (uint64_t)a.d) ||
      !make_bmaps(&bh, a.h, (uint64_t)a.s_cap, (uint64_t)a.f)) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed (driver entry point missing or bad pointer/shape)");
    return FEPLB_E_CUDA;
  }
  CUtensorMap tm_r1 = tm_w1, tm_r3 = tm_w3, tm_r2 = tm_w2;
  const bool has_recv = a.recv_w1 && a.recv_w3 && a.recv_w2 && a.n_recv_slots > 0;
  if (has_recv && (!make_tmap(&tm_r1, a.recv_w1, (uint64_t)a.n_recv_slots * a.f, (uint64_t)a.d, WM / 2) ||
                   !make_tmap(&tm_r3, a.recv_w3, (uint64_t)a.n_recv_slots * a.f, (uint64_t)a.d, WM / 2) ||
                   !make_tmap(&tm_r2, a.recv_w2, (uint64_t)a.n_recv_slots * a.d, (uint64_t)a.f, WM))) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed for the receive buffer");
    return FEPLB_E_CUDA;
  }
  BMaps brx = bx;      // rows of migrated pieces: pass 1 reads them from the receive region when there is one
  if (has_recv && a.recv_x && !make_bmaps(&brx, a.recv_x, (uint64_t)a.s_cap, (uint64_t)a.d)) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed for the receive region of the rows");
    return FEPLB_E_CUDA;
  }
  WmParams p1;
  p1.groups = a.groups; p1.n_groups = a.n_groups; p1.which = a.which;
  p1.dyn = feplb_dyn_table(dyn);
  p1.E = a.E; p1.s_cap = a.s_cap;
  // pass 1: a unit covers 128 hidden units, 64 per CTA, each CTA taking its rows of W1 and of W3
  p1.n_pairs = a.f / 128; p1.num_k_blocks = a.d / BK; p1.a_rows_per_expert = a.f; p1.unit_rows = 128; p1.cta_rows = 64; p1.a1_row_off = 0;
  p1.n_recv_slots = has_recv ? a.n_recv_slots : 0;
  p1.out = (__nv_bfloat16*)a.h; p1.ld_out = a.f; p1.ab_out = (__nv_bfloat16*)a.ab_out;
  p1.status = a.status; p1.stamps = dyn.stamps;
  // pass 2: a unit covers 256 output columns, 128 per CTA as two consecutive boxes of W2
  WmParams p2 = p1;
  p2.n_pairs = a.d / 256; p2.num_k_blocks = a.f / BK; p2.a_rows_per_expert = a.d; p2.unit_rows = 256; p2.cta_rows = 128; p2.a1_row_off = 64;
  p2.out = (__nv_bfloat16*)a.y; p2.ld_out = a.d; p2.ab_out = nullptr;
  p2.stamps = dyn.stamps ? dyn.stamps + 4 : nullptr;

  cudaError_t e = launch_wm<true>(tm_w1, tm_w3, tm_r1, tm_r3, bx, brx, p1, a.num_sms, st);
  ++*n_launch;
  if (e == cudaSuccess) {
    e = launch_wm<false>(tm_w2, tm_w2, tm_r2, tm_r2, bh, bh, p2, a.num_sms, st);
    ++*n_launch;
  }
  if (e != cudaSuccess) {
    snprintf(err, errn, "k_ffn_wm launch: %s", cudaGetErrorString(e));
    return FEPLB_E_CUDA;
  }
  return FEPLB_OK;
}
