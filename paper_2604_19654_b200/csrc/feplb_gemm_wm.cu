// Grouped SwiGLU expert FFN, "weights on M" form, for sm_100a (paper Section 2.3: static-expert,
// then dynamic-expert Grouped GEMM; Section 3.1: grouped GEMM over per-expert row segments whose
// cost is very sensitive to the per-expert batch size).
//
// The other form of this library (feplb_gemm.cu) puts 128 or 256 token rows on the M side of the
// MMA and the expert's weights on the N side.  With a few hundred rows per expert that wastes up
// to 127 (255) rows of every segment's last tile and, worse, makes a CTA pull 48 KiB of operands
// through its L2 port per 64-wide K step of a 128 x 256 tile, more than the port delivers while
// the tensor pipe works on it.  Here the roles are exchanged:
//
//   unit   = (row block of one group: n <= 256 rows, padded to a multiple of 16)
//          x (a pair of 128-row weight tiles of the group's expert)
//   pass 1 : A0 = W1[e][u0:u0+128, :], A1 = W3[e][u0:u0+128, :], B = X[rows, :]
//            acc_a = A0 B^T, acc_b = A1 B^T  (128 hidden units x n tokens each, fp32 in TMEM)
//            H[rows, u0:u0+128] = silu(acc_a) * acc_b                          (transposed store)
//   pass 2 : A0 = W2[e][c0:c0+128, :], A1 = W2[e][c0+128:c0+256, :], B = H[rows, :]
//            Y[rows, c0:c0+256] = (acc_a | acc_b)^T
//
// so a K step moves 32 KiB of weights plus 128 bytes per token row for two MMAs of 128 x n x 64,
// an expert's weights cross the L2 port once per <= 256 rows instead of once per 128, and a
// segment's ragged tail costs at most 15 padded rows.  One CTA per SM, persistent, warp-specialised:
// warp 0 = TMA producer, warp 1 = tcgen05.mma issuer and TMEM owner, warps 2..9 = epilogue.
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

namespace {

constexpr int WM = 128;                 // weight rows per A tile (UMMA M)
#ifndef FEPLB_WM_EXP
#define FEPLB_WM_EXP 0
#endif
#ifndef FEPLB_WM_BK
#define FEPLB_WM_BK 64
#endif
constexpr int BK = FEPLB_WM_BK;         // K elements per stage = one swizzle row (128 or 64 bytes)
constexpr int UMMA_K = 16;
constexpr int kNMax = 256;              // token rows per unit (UMMA N)
constexpr int kATile = WM * BK * 2;     // 16 / 8 KiB
constexpr int kBBytes = kNMax * BK * 2; // 32 / 16 KiB
constexpr int kStageBytes = 2 * kATile + kBBytes;   // 64 / 32 KiB
constexpr int kStages = 3 * 64 / BK;
constexpr int kRingBytes = kStages * kStageBytes;   // 192 KiB
constexpr int kEpiWarps = 8;            // two warps per TMEM lane quarter
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kEpiStageBytes = 32 * 64; // per epilogue warp: 32 tokens x 32 units of bf16
constexpr int kTmemCols = 512;
constexpr int kMaxEntries = FEPLB_WM_MAX_ENTRIES;   // group entries of both tables together
constexpr int kBoxes = 5;               // token-row boxes of 256, 128, 64, 32 and 16 rows

struct Tail {
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
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
constexpr size_t kSmemBytes = 1024 + (size_t)kRingBytes + (size_t)kEpiWarps * kEpiStageBytes + sizeof(Tail);
static_assert(kSmemBytes <= 232448, "shared memory budget");
static_assert(kSmemBytes > 116 * 1024, "one CTA per SM: each allocates all of TMEM");

struct BMaps { CUtensorMap m[kBoxes]; };

struct WmParams {
  const feplb_group* groups;            // table known at launch
  int n_groups;
  int which;                            // FEPLB_FFN_* filter on that table
  int4* dyn_dev;                        // dynamic table, 32 bytes per group {expert, row_start, rows, exec_rank, is_dynamic,
                                        // seq, 0, 0}: device copy, made by the CTA that wins `claim` from ...
  const int4* dyn_host;                 // ... the planner's own table in mapped host memory
  unsigned long long* ready_dev;        // (seq << 32) | number of dynamic groups
  const unsigned long long* ready_host;
  uint32_t* claim;                      // device word: seq of the forward whose table transfer has been claimed
  int dyn_cap;                          // capacity of dyn_dev in groups
  uint32_t seq;                         // 0: no dynamic table in this launch
  int E;
  int64_t s_cap;
  int n_pairs;                          // weight-tile pairs per row block
  int num_k_blocks;
  int a_rows_per_expert;                // rows of one expert in the weight maps
  int a1_row_off;                       // row offset of the second tile of a pair inside the same map (pass 2), 0 in pass 1
  int pair_rows;                        // weight rows a pair advances by (128 in pass 1, 256 in pass 2)
  int n_recv_slots;
  __nv_bfloat16* out;
  int ld_out;
  __nv_bfloat16* ab_out;                // pass 1, optional: pre-activations a | b ([rows, 2f])
  uint32_t* status;
  unsigned long long* stamps;           // optional, preset to all ones, globaltimer ns: [0] first CTA's start, [1] first
                                        // time a CTA ran out of static units, [2] ~(last CTA's end), [3] ~(longest
                                        // wait for the dynamic table); the last two are kept complemented so that
                                        // one atomicMin and one memset pattern serve all four
  unsigned long long wait_limit_ns;     // bound of the wait for the dynamic table
};

// Shared-memory descriptor of a K-major tile whose rows are BK bf16 wide: 128-byte rows with the
// 128-byte swizzle (8-row groups 1024 bytes apart) or 64-byte rows with the 64-byte swizzle (512 apart).
__device__ __forceinline__ uint64_t wm_desc(uint32_t saddr) {
  if (BK == 64) return make_smem_desc(saddr);
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(512 >> 4) << 32) | (1ull << 46) | (4ull << 61);
}

struct Unit { int row0, n_rows, n_pad, expert, slot, wt; };

__device__ __forceinline__ int units_of(int rows, int n_pairs) { return (rows + kNMax - 1) / kNMax * n_pairs; }

// unit -> (entry, row block, weight-tile pair).  The pairs of one row block are consecutive, so CTAs
// running at the same time share the block's rows in L2 and sweep the expert's weights once.
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
  const int bs = ((rows + nb - 1) / nb + 15) & ~15;      // rows per block, a multiple of 16, <= 256
  Unit c;
  c.wt = local - blk * n_pairs;
  c.row0 = t->row_start[lo] + blk * bs;
  c.n_rows = min(bs, rows - blk * bs);
  c.n_pad = (c.n_rows + 15) & ~15;
  c.expert = t->expert[lo] & 0xffff;
  c.slot = (t->expert[lo] >> 16) - 1;
  return c;
}

// Polling loads are relaxed (they bypass L1 and order nothing), and no fence follows them: acquire
// loads and fences were measured to cost tens of microseconds each while the other SMs saturate the
// memory system.  The table entries carry the sequence number themselves instead.
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
constexpr int kGaveUp = -1;            // "number of groups" of a ready word whose writer gave up waiting for the table

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
         const __grid_constant__ BMaps tm_b, const WmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* epi_smem = smem + (size_t)kRingBytes;
  Tail* tail = reinterpret_cast<Tail*>(epi_smem + (size_t)kEpiWarps * kEpiStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int worker = (int)blockIdx.x, n_workers = (int)gridDim.x;
  volatile int* abort_flag = &tail->abort_flag;
  const bool has_dyn = p.seq != 0;

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
      mbar_init(smem_u32(&tail->tmem_empty[a]), kEpiWarps);
    }
    mbar_init(smem_u32(&tail->dyn_bar), 1);
    tail->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    __syncwarp();
    tmem_alloc(smem_u32(&tail->tmem_base), kTmemCols);
    tmem_relinquish();
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
        const int4 lo = __ldcg(p.dyn_dev + 2 * i), hi = __ldcg(p.dyn_dev + 2 * i + 1);   // expert, row_start, rows, exec_rank | is_dynamic, seq
        if ((uint32_t)hi.y != p.seq) { good = false; continue; }
        tail->prefix[n_static_entries + i + 1] = put_entry(tail, n_static_entries + i, lo.x, lo.y, lo.z, hi.x, true, p);
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
        // Out of static units: now the table is needed.  It reaches the device like this: the planner
        // thread writes it, and then a word with this forward's sequence number, into mapped host
        // memory.  The first CTA to get here claims the transfer: it alone polls that word across
        // PCIe (reads of host memory from many SMs at once queue up behind one another), copies the
        // table into device memory and sets the device-side word, which is what every other CTA,
        // and the second pass, look at.  So the bounded wait depends on the host thread alone.
        const unsigned long long t0 = global_timer_ns();
        if (p.stamps && lane == 0) atomicMin(&p.stamps[1], t0);
        while (!dyn_known) {
          unsigned long long v = 0;
          int got = 0;                       // 1: the device copy is there; 2: this CTA must make it
          if (lane == 0) {
            for (;;) {
              v = ld_relaxed_gpu_u64(p.ready_dev);
              if ((uint32_t)(v >> 32) == p.seq) { got = 1; break; }
              if (!tried_claim) {
                tried_claim = true;
                const uint32_t cur = *reinterpret_cast<volatile uint32_t*>(p.claim);
                claimer = cur != p.seq && atomicCAS(p.claim, cur, p.seq) == cur;
              }
              if (claimer) {
                v = ld_relaxed_sys_u64(p.ready_host);
                if ((uint32_t)(v >> 32) == p.seq) { got = 2; break; }
              }
              if (*abort_flag) { ok = false; break; }
              // the claimer gives up first and tells the others; they keep their own, longer, bound
              if (global_timer_ns() - t0 > p.wait_limit_ns + (claimer ? 0ull : kWaitLimitNs)) {
                atomicOr(p.status, FEPLB_ST_PLAN);
                got = 3;
                break;
              }
              __nanosleep(claimer ? 100 : 400);
            }
          }
          ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          if (!ok) break;
          got = __shfl_sync(0xffffffffu, got, 0);
          int n_dyn = __shfl_sync(0xffffffffu, (int)(uint32_t)v, 0);
          if (got == 3 || n_dyn == kGaveUp) {
            // no table within the limit: go on as if it were empty, so that the static units still in
            // flight in this CTA complete normally; the status word carries the reason
            if (got == 3 && lane == 0 && claimer)
              asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.ready_dev),
                           "l"(((unsigned long long)p.seq << 32) | (uint32_t)kGaveUp) : "memory");
            if (n_dyn == kGaveUp && lane == 0) atomicOr(p.status, FEPLB_ST_PLAN);
            take_table(0);
            break;
          }
          if (got == 2) {
            if (n_dyn < 0 || n_dyn > p.dyn_cap) {
              if (lane == 0) atomicOr(p.status, FEPLB_ST_GROUP);
              n_dyn = 0;
            }
            // ordinary (weak) 16-byte loads: they coalesce into a few PCIe reads.  Entries that do not
            // carry the sequence number yet are read again.
            bool good = false;
            for (int attempt = 0; attempt < 64 && !good; ++attempt) {
              good = true;
              for (int i = lane; i < n_dyn; i += 32) {
                const int4 lo = __ldcv(p.dyn_host + 2 * i), hi = __ldcv(p.dyn_host + 2 * i + 1);
                if ((uint32_t)hi.y != p.seq) { good = false; continue; }
                p.dyn_dev[2 * i] = lo;
                p.dyn_dev[2 * i + 1] = hi;
              }
              good = __all_sync(0xffffffffu, good);
            }
            if (!good) {
              if (lane == 0) atomicOr(p.status, FEPLB_ST_GROUP);
              n_dyn = 0;
            }
            __syncwarp();                    // the lanes' stores happen before lane 0's release below
            if (lane == 0)
              asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.ready_dev),
                           "l"(((unsigned long long)p.seq << 32) | (uint32_t)n_dyn) : "memory");
          }
          if (!take_table(n_dyn) && global_timer_ns() - t0 > p.wait_limit_ns + kWaitLimitNs) {
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
      if (!dyn_known && lane == 0) peek = ld_relaxed_gpu_u64(p.ready_dev);
      if (lane == 0) {
        const CUtensorMap* ma0 = c.slot >= 0 ? &tm_r0 : &tm_a0;
        const CUtensorMap* ma1 = c.slot >= 0 ? &tm_r1 : &tm_a1;
        const int arow0 = (c.slot >= 0 ? c.slot : c.expert) * p.a_rows_per_expert + c.wt * p.pair_rows;
        const int arow1 = arow0 + p.a1_row_off;
        const uint32_t tx = (uint32_t)(2 * kATile + c.n_pad * (BK * 2));
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->empty[stage]), phase ^ 1u, abort_flag, p.status))) break;
          const uint32_t full = smem_u32(&tail->full[stage]);
          const uint32_t sa = smem_u32(smem + (size_t)stage * kStageBytes);
#if FEPLB_WM_EXP == 1
          mbar_arrive(full);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
          continue;
#endif
          mbar_expect_tx(full, tx);
          tma_load_2d(sa, ma0, full, kb * BK, arow0);
          tma_load_2d(sa + kATile, ma1, full, kb * BK, arow1);
          uint32_t sb = sa + 2 * kATile;
          int r = 0;
#pragma unroll
          for (int i = 0; i < kBoxes; ++i) {
            const int box = kNMax >> i;
            if (c.n_pad - r >= box) {
              tma_load_2d(sb, &tm_b.m[i], full, kb * BK, c.row0 + r);
              r += box;
              sb += (uint32_t)(box * BK * 2);
            }
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      if (ok && !dyn_known) {
        peek = __shfl_sync(0xffffffffu, peek, 0);
        if ((uint32_t)(peek >> 32) == p.seq && (int)(uint32_t)peek != kGaveUp) take_table((int)(uint32_t)peek);
      }
    }
    if (!ok && lane == 0) {
      for (int i = 0; i < 2000; ++i) __nanosleep(100);   // copies already issued land before the CTA's shared memory goes away
    }
  } else if (warp == 1) {
    // ---- MMA issuer ------------------------------------------------------------------------------
    if (lane == 0) {
      int stage = 0, slot = 0;
      uint32_t phase = 0, ephase[2] = {0, 0};
      bool ok = true, dyn_known = !has_dyn;
      int n_entries = n_static_entries, total = n_static_units;
      for (int u = worker; ok; u += n_workers) {
        if (u >= total) {
          if (dyn_known) break;
          if (!(ok = mbar_wait(smem_u32(&tail->dyn_bar), 0, abort_flag, p.status, p.wait_limit_ns + 2 * kWaitLimitNs))) break;
          dyn_known = true;
          n_entries = tail->n_entries;
          total = tail->total_units;
          if (u >= total) break;
        }
        const Unit c = unit_coord(tail, n_entries, p.n_pairs, u);
        const bool big = c.n_pad > 128;          // both accumulators of a big unit take 256 columns each: all of TMEM
        uint32_t col_a, col_b;
        if (big) {
          if (!(ok = mbar_wait(smem_u32(&tail->tmem_empty[0]), ephase[0] ^ 1u, abort_flag, p.status))) break;
          if (!(ok = mbar_wait(smem_u32(&tail->tmem_empty[1]), ephase[1] ^ 1u, abort_flag, p.status))) break;
          col_a = 0; col_b = 256;
        } else {
          if (!(ok = mbar_wait(smem_u32(&tail->tmem_empty[slot]), ephase[slot] ^ 1u, abort_flag, p.status))) break;
          col_a = (uint32_t)(slot * 256); col_b = col_a + 128;
        }
        tc_fence_after();
        const uint32_t idesc = make_idesc(WM, c.n_pad);
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->full[stage]), phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)stage * kStageBytes);
          const uint64_t da0 = wm_desc(sa), da1 = wm_desc(sa + kATile), db = wm_desc(sa + 2 * kATile);
#if FEPLB_WM_EXP != 2
#ifdef FEPLB_WM_REORDER
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(tmem_base + col_a, da0 + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (uint32_t)((kb | k) != 0));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(tmem_base + col_b, da1 + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (uint32_t)((kb | k) != 0));
#else
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint32_t acc = (uint32_t)((kb | k) != 0);
            umma_bf16(tmem_base + col_a, da0 + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, acc);
            umma_bf16(tmem_base + col_b, da1 + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, acc);
          }
#endif
#endif
          umma_commit(smem_u32(&tail->empty[stage]));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (big) {
          umma_commit(smem_u32(&tail->tmem_full[0]));
          umma_commit(smem_u32(&tail->tmem_full[1]));
          ephase[0] ^= 1u; ephase[1] ^= 1u;
        } else {
          umma_commit(smem_u32(&tail->tmem_full[slot]));
          ephase[slot] ^= 1u;
          slot ^= 1;
        }
      }
    }
  } else {
    // ---- epilogue: TMEM -> registers -> (SwiGLU) -> bf16 -> transposed rows in global memory ---------
    // A thread owns one weight row (a hidden unit in pass 1, an output column in pass 2) and gets 32
    // token rows per tcgen05.ld.  Two warps share each TMEM lane quarter and take alternate chunks.
    const int q = warp & 3;                      // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;            // 0: even chunks of 32 tokens, 1: odd chunks
    const uint32_t stg = smem_u32(epi_smem + (size_t)(warp - 2) * kEpiStageBytes);
    int slot = 0;
    uint32_t fphase[2] = {0, 0};
    bool ok = true, dyn_known = !has_dyn;
    int n_entries = n_static_entries, total = n_static_units;
    for (int u = worker; ok; u += n_workers) {
      if (u >= total) {
        if (dyn_known) break;
        ok = mbar_wait(smem_u32(&tail->dyn_bar), 0, abort_flag, p.status, p.wait_limit_ns + 2 * kWaitLimitNs);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        dyn_known = true;
        n_entries = tail->n_entries;
        total = tail->total_units;
        if (u >= total) break;
      }
      const Unit c = unit_coord(tail, n_entries, p.n_pairs, u);
      const bool big = c.n_pad > 128;
      uint32_t col_a, col_b;
      if (big) {
        ok = mbar_wait(smem_u32(&tail->tmem_full[0]), fphase[0], abort_flag, p.status) &&
             mbar_wait(smem_u32(&tail->tmem_full[1]), fphase[1], abort_flag, p.status);
        col_a = 0; col_b = 256;
      } else {
        ok = mbar_wait(smem_u32(&tail->tmem_full[slot]), fphase[slot], abort_flag, p.status);
        col_a = (uint32_t)(slot * 256); col_b = col_a + 128;
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
      // pass 1: H[row, wt*128 + wrow];  pass 2: Y[row, wt*256 + wrow] and Y[row, wt*256 + 128 + wrow]
      const int col0 = c.wt * p.pair_rows + q * 32;
      const int n_chunks = (c.n_pad + 31) >> 5;
      uint32_t ra[32], rb[32];
      int ch = half;
#if FEPLB_WM_EXP == 3
      ch = n_chunks + 2;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (big) { mbar_arrive(smem_u32(&tail->tmem_empty[0])); mbar_arrive(smem_u32(&tail->tmem_empty[1])); }
        else mbar_arrive(smem_u32(&tail->tmem_empty[slot]));
      }
#endif
      if (ch < n_chunks) {
        tmem_ld32(lane_base + col_a + (uint32_t)(ch * 32), ra);
        tmem_ld32(lane_base + col_b + (uint32_t)(ch * 32), rb);
      }
      for (; ch < n_chunks; ch += 2) {
        tmem_ld_wait();
        float va[32], vb[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) { va[j] = __uint_as_float(ra[j]); vb[j] = __uint_as_float(rb[j]); }
        const bool more = ch + 2 < n_chunks;
        if (more) {                              // the next chunk's TMEM loads fly while this one is converted and stored
          tmem_ld32(lane_base + col_a + (uint32_t)((ch + 2) * 32), ra);
          tmem_ld32(lane_base + col_b + (uint32_t)((ch + 2) * 32), rb);
        } else {
          // every TMEM read of this unit by this warp has completed: the accumulator may be overwritten
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (big) { mbar_arrive(smem_u32(&tail->tmem_empty[0])); mbar_arrive(smem_u32(&tail->tmem_empty[1])); }
            else mbar_arrive(smem_u32(&tail->tmem_empty[slot]));
          }
        }
        const int r0 = c.row0 + ch * 32;
        const int n_valid = c.n_rows - ch * 32;  // valid token rows among this chunk's 32
        if (SWIGLU) {
          if (p.ab_out != nullptr) {
            __nv_bfloat16* ab = p.ab_out + (int64_t)r0 * (2 * p.ld_out) + col0;
            store_transposed(stg, va, ab, 2 * p.ld_out, n_valid, lane);
            store_transposed(stg, vb, ab + p.ld_out, 2 * p.ld_out, n_valid, lane);
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) va[j] = silu_f(va[j]) * vb[j];
          store_transposed(stg, va, p.out + (int64_t)r0 * p.ld_out + col0, p.ld_out, n_valid, lane);
        } else {
          __nv_bfloat16* o = p.out + (int64_t)r0 * p.ld_out + col0;
          store_transposed(stg, va, o, p.ld_out, n_valid, lane);
          store_transposed(stg, vb, o + WM, p.ld_out, n_valid, lane);
        }
      }
#if FEPLB_WM_EXP != 3
      if (half >= n_chunks)
#else
      if (false)
#endif
      {                    // a unit of at most 32 rows: this warp read nothing, but it still hands the slot back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tail->tmem_empty[slot]));
      }
      if (big) { fphase[0] ^= 1u; fphase[1] ^= 1u; }
      else { fphase[slot] ^= 1u; slot ^= 1; }
    }
  }

  // ---- teardown --------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (p.stamps && threadIdx.x == 0) {
    const unsigned long long te = global_timer_ns();
    atomicMin(&p.stamps[2], ~te);
#ifdef FEPLB_PROBE
    if (SWIGLU) { atomicMin(&p.stamps[9], te); atomicAdd(&p.stamps[10], te - p.stamps[8]); }
    else { atomicMin(&p.stamps[11], te); atomicAdd(&p.stamps[12], te - p.stamps[8]); }
#endif
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
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
            CU_TENSOR_MAP_INTERLEAVE_NONE, BK == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_bmaps(BMaps* b, const void* base, uint64_t rows, uint64_t inner) {
  for (int i = 0; i < kBoxes; ++i) {
    if (!make_tmap(&b->m[i], base, rows, inner, (uint32_t)(kNMax >> i))) return false;   // rows past the tensor read as zeros
  }
  return true;
}

template <bool SWIGLU>
cudaError_t launch_wm(const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& r0, const CUtensorMap& r1,
                      const BMaps& b, const WmParams& p, int num_sms, cudaStream_t st) {
  static bool attr_set[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(k_ffn_wm<SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(num_sms);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_ffn_wm<SWIGLU>, a0, a1, r0, r1, b, p);
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
  CUtensorMap tm_w1, tm_w3, tm_w2;
  BMaps bx, bh;
  if (!make_tmap(&tm_w1, a.w1, (uint64_t)a.E * a.f, (uint64_t)a.d, WM) ||
      !make_tmap(&tm_w3, a.w3, (uint64_t)a.E * a.f, (uint64_t)a.d, WM) ||
      !make_tmap(&tm_w2, a.w2, (uint64_t)a.E * a.d, (uint64_t)a.f, WM) ||
      !make_bmaps(&bx, a.x_perm, (uint64_t)a.s_cap, (uint64_t)a.d) ||
      !make_bmaps(&bh, a.h, (uint64_t)a.s_cap, (uint64_t)a.f)) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed (driver entry point missing or bad pointer/shape)");
    return FEPLB_E_CUDA;
  }
  CUtensorMap tm_r1 = tm_w1, tm_r3 = tm_w3, tm_r2 = tm_w2;
  const bool has_recv = a.recv_w1 && a.recv_w3 && a.recv_w2 && a.n_recv_slots > 0;
  if (has_recv && (!make_tmap(&tm_r1, a.recv_w1, (uint64_t)a.n_recv_slots * a.f, (uint64_t)a.d, WM) ||
                   !make_tmap(&tm_r3, a.recv_w3, (uint64_t)a.n_recv_slots * a.f, (uint64_t)a.d, WM) ||
                   !make_tmap(&tm_r2, a.recv_w2, (uint64_t)a.n_recv_slots * a.d, (uint64_t)a.f, WM))) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed for the receive buffer");
    return FEPLB_E_CUDA;
  }
  WmParams p1;
  p1.groups = a.groups; p1.n_groups = a.n_groups; p1.which = a.which;
  p1.dyn_dev = reinterpret_cast<int4*>(dyn.table_dev); p1.dyn_host = reinterpret_cast<const int4*>(dyn.table_host); p1.ready_dev = dyn.ready_dev; p1.ready_host = dyn.ready_host;
  p1.claim = dyn.claim; p1.dyn_cap = dyn.max_groups;
  p1.seq = dyn.seq;
  p1.E = a.E; p1.s_cap = a.s_cap;
  p1.n_pairs = a.f / WM; p1.num_k_blocks = a.d / BK; p1.a_rows_per_expert = a.f; p1.a1_row_off = 0; p1.pair_rows = WM;
  p1.n_recv_slots = has_recv ? a.n_recv_slots : 0;
  p1.out = (__nv_bfloat16*)a.h; p1.ld_out = a.f; p1.ab_out = (__nv_bfloat16*)a.ab_out;
  p1.status = a.status; p1.stamps = dyn.stamps; p1.wait_limit_ns = dyn.wait_limit_ns ? dyn.wait_limit_ns : kWaitLimitNs;
  WmParams p2 = p1;
  p2.n_pairs = a.d / (2 * WM); p2.num_k_blocks = a.f / BK; p2.a_rows_per_expert = a.d; p2.a1_row_off = WM; p2.pair_rows = 2 * WM;
  p2.out = (__nv_bfloat16*)a.y; p2.ld_out = a.d; p2.ab_out = nullptr;
  p2.stamps = dyn.stamps ? dyn.stamps + 4 : nullptr;

  cudaError_t e = launch_wm<true>(tm_w1, tm_w3, tm_r1, tm_r3, bx, p1, a.num_sms, st);
  ++*n_launch;
  if (e == cudaSuccess) {
    e = launch_wm<false>(tm_w2, tm_w2, tm_r2, tm_r2, bh, p2, a.num_sms, st);
    ++*n_launch;
  }
  if (e != cudaSuccess) {
    snprintf(err, errn, "k_ffn_wm launch: %s", cudaGetErrorString(e));
    return FEPLB_E_CUDA;
  }
  return FEPLB_OK;
}
