// Grouped SwiGLU expert FFN of the FEPLB hot path on sm_100a (paper Section 2.3: static-expert,
// then dynamic-expert Grouped GEMM; Section 3.1: grouped GEMM over per-expert row segments).
//
// Two launches of one persistent, warp-specialised kernel:
//   pass 1 (SwiGLU): H[rows, n0:n0+bn] = silu(X W1[e]) * (X W3[e])   -- one MMA of N = 2*bn whose
//                    B tile is the W1 tile followed by the W3 tile; the epilogue multiplies
//                    the two halves of the accumulator and rounds to bf16
//   pass 2 (plain):  Y[rows, n0:n0+2bn] = H W2[e]
// Per CTA: warp 0 = TMA producer (one lane), warp 1 = tcgen05.mma issuer (one lane) and TMEM
// owner, the other warps = epilogue (tcgen05.ld -> registers -> global).  A and B tiles are
// staged by TMA (128-byte swizzle, K-major) through a shared-memory ring; the fp32 accumulators
// live in TMEM.  A tile covers rows of ONE group (row segment of one expert); the last tile of
// a group is ragged and its surplus rows are computed but never stored.
//
// Every mbarrier wait is bounded: when it gives up the CTA raises FEPLB_ST_WAIT in the status
// word, all roles leave their loops, TMEM is released and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>

#include "feplb_internal.h"
#include "feplb_tc.cuh"
#include "feplb_dyn.cuh"

namespace {

constexpr int BM = FEPLB_TILE_M;       // rows per MMA (UMMA M) = rows of one sub-tile
constexpr int BK = 64;                 // K elements per stage = one 128-byte swizzle row
constexpr int UMMA_K = 16;             // K per tcgen05.mma for 16-bit inputs
constexpr int kAccCols = 256;          // TMEM columns of one accumulator
constexpr int kTmemCols = 512;         // all of TMEM: one CTA per SM
constexpr int kABytes = BM * BK * 2;               // 16 KiB per sub-tile
constexpr int kBBytesMax = 256 * BK * 2;           // 32 KiB

// Two forms of one kernel.
//   single (PAIR = false): one CTA computes a 128 x 256 tile (UMMA M x N, cta_group::1); K step 64;
//     4 stages of 48 KiB (A 16 KiB + B 32 KiB).  The mainloop needs 96 bytes per MMA cycle from L2.
//   pair (PAIR = true): a cluster of two CTAs computes a 256 x 256 tile with cta_group::2 MMAs
//     issued by the even CTA: each CTA stages its own 128 rows of A and HALF of the B tile (the
//     W1 tile in the even CTA and the W3 tile in the odd one in pass 1), so a CTA needs only
//     64 bytes per MMA cycle from L2 and the ring holds 6 stages of 32 KiB.  No load is shared
//     between the CTAs: each brings its own halves.  Used for launches whose groups are large
//     (a 256-row tile wastes more on a ragged tail).
// Both keep two accumulators in TMEM so that the epilogue of tile i overlaps the MMAs of tile i+1.
template <bool PAIR> struct Ring {
  static constexpr int kStages = PAIR ? 6 : 4;
  static constexpr int kStageBytes = kABytes + (PAIR ? kBBytesMax / 2 : kBBytesMax);   // multiple of 1024
  static constexpr int kTileRows = PAIR ? 2 * BM : BM;
};
constexpr int kMaxStages = 6;
constexpr int kAccStages = 2;
constexpr int kRingBytes = 4 * (kABytes + kBBytesMax);   // 192 KiB in both forms
static_assert(Ring<false>::kStages * Ring<false>::kStageBytes == kRingBytes &&
              Ring<true>::kStages * Ring<true>::kStageBytes == kRingBytes, "ring size");
constexpr int kEpiWarps = 4;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kEpiStageBytes = 32 * 128;            // per epilogue warp: 32 rows x 64 bf16

struct SmemTail {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long tmem_full[kAccStages];
  unsigned long long tmem_empty[kAccStages];
  unsigned long long dyn_bar;         // completed by warp 0 once the dynamic entries are in place
  uint32_t tmem_base;
  int abort_flag;
  int n_entries;                      // entries in use (the table known at launch, then the planner's dynamic groups)
  int total_mtiles;                   // prefix[n_entries]
  int prefix[FEPLB_MAX_GROUPS + 1];   // prefix[g] = M tiles of groups before g
  int g_row_start[FEPLB_MAX_GROUPS];
  int g_rows[FEPLB_MAX_GROUPS];
  int g_expert[FEPLB_MAX_GROUPS];
};
constexpr size_t kSmemBytes = 1024 /* alignment slack */ + (size_t)kRingBytes +
                              (size_t)kEpiWarps * kEpiStageBytes + sizeof(SmemTail);
static_assert(kSmemBytes <= 232448, "shared memory budget");
static_assert(kSmemBytes > 116 * 1024, "two CTAs must never share an SM: each allocates all of TMEM");

struct GemmParams {
  const feplb_group* groups;
  int n_groups;
  int which;            // FEPLB_FFN_*
  int E;
  int64_t s_cap;        // rows of the A and output buffers
  int n_tiles_n;        // N tiles per M tile
  int num_k_blocks;     // K / 64
  int b_rows_per_expert;  // rows of one expert in the B tensor maps
  int n_recv_slots;     // slots of the receive buffer of migrated experts' weights (0 = none)
  int bn;               // rows of one B half tile (64 or 128); the MMA has N = 2*bn
  __nv_bfloat16* out;
  int ld_out;           // elements between output rows
  uint32_t* status;
  __nv_bfloat16* ab_out;   // pass 1, optional: pre-activations a | b saved for the backward pass ([rows, 2f])
  DynTable dyn;            // the planner's table of dynamic groups, walked after `groups` (dyn.seq == 0: none in this launch)
  unsigned long long* stamps;   // optional, preset to all ones, globaltimer ns: [0] first CTA's start, [1] first time a CTA
                                // ran out of static tiles, [2] ~(last CTA's end), [3] ~(longest wait for the dynamic table)
};


struct TileCoord { int row0, rows_valid, expert, slot, nt; };   // slot >= 0: weights in that receive slot

// tile -> (group, M tile, N tile); N tiles of one M tile are consecutive so that CTAs running at
// the same time share the A rows and sweep one expert's weights together (both stay in L2).
template <int kRows>
__device__ __forceinline__ TileCoord tile_coord(const SmemTail* t, int n_groups, int n_tiles_n, int tile) {
  const int mt = tile / n_tiles_n;
  int lo = 0, hi = n_groups;   // largest g with prefix[g] <= mt
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (t->prefix[mid] <= mt) lo = mid; else hi = mid;
  }
  const int local = mt - t->prefix[lo];
  TileCoord c;
  c.row0 = t->g_row_start[lo] + local * kRows;
  c.rows_valid = min(kRows, t->g_rows[lo] - local * kRows);
  c.expert = t->g_expert[lo] & 0xffff;
  c.slot = (t->g_expert[lo] >> 16) - 1;
  c.nt = tile - mt * n_tiles_n;
  return c;
}

// fp32 accumulator registers of 32 columns -> 16 packed bf16 pairs (SwiGLU: silu(a) * b first).
template <bool SWIGLU>
__device__ __forceinline__ void convert_slice(const uint32_t (&a)[32], const uint32_t (&b)[32], uint32_t* packed) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    float v0 = __uint_as_float(a[2 * i]), v1 = __uint_as_float(a[2 * i + 1]);
    if (SWIGLU) {
      v0 = silu_f(v0) * __uint_as_float(b[2 * i]);
      v1 = silu_f(v1) * __uint_as_float(b[2 * i + 1]);
    }
    packed[i] = pack_bf16x2(v0, v1);
  }
}

// 32 rows x 64 bf16 columns, one row per lane in packed[32]: through the warp's staging area (row
// `lane`, 16-byte chunk j at position j ^ (lane & 7)) and out again 4 rows per instruction, so
// that every global store covers whole 128-byte lines; rows >= rows_here are not written.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(m)), "r"(src), "r"(c0), "r"(c1) : "memory");
}
// The warp's staging area may still be read by the TMA store of its previous slice.
__device__ __forceinline__ void staging_ready(int lane) {
  if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  __syncwarp();
}

// Full slices (all 32 rows valid) leave through one TMA store: the staging layout below IS the
// 128-byte-swizzled box layout, so lane 0 hands the 4 KiB to the copy unit and the warp moves on.
__device__ __forceinline__ void stage_and_tma_store(uint32_t stg, const uint32_t* packed, const CUtensorMap* m, int gcol,
                                                    int grow, int lane) {
  staging_ready(lane);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t addr = stg + (uint32_t)(lane * 128 + ((j ^ (lane & 7)) << 4));
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(packed[4 * j]), "r"(packed[4 * j + 1]),
                 "r"(packed[4 * j + 2]), "r"(packed[4 * j + 3]) : "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  if (lane == 0) {
    tma_store_2d(m, stg, gcol, grow);
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  }
}

__device__ __forceinline__ void stage_and_store(uint32_t stg, const uint32_t* packed, __nv_bfloat16* obase, int ld,
                                                int col, int rows_here, int lane) {
  const int rd_row = lane >> 3, rd_chunk = lane & 7;
  staging_ready(lane);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t addr = stg + (uint32_t)(lane * 128 + ((j ^ (lane & 7)) << 4));
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(packed[4 * j]), "r"(packed[4 * j + 1]),
                 "r"(packed[4 * j + 2]), "r"(packed[4 * j + 3]) : "memory");
  }
  __syncwarp();
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int r = it * 4 + rd_row;
    const uint32_t addr = stg + (uint32_t)(r * 128 + ((rd_chunk ^ (r & 7)) << 4));
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    if (r < rows_here) *reinterpret_cast<uint4*>(obase + (int64_t)r * ld + col + rd_chunk * 8) = v;
  }
  __syncwarp();
}

// One entry of a group table -> shared-memory arrays; returns its number of M tiles (0 if not selected).
template <int kRows>
__device__ __forceinline__ int put_group(SmemTail* t, int idx, int expert, int row_start, int rows, int is_dynamic, bool selected,
                                         const GemmParams& p) {
  int tiles = 0;
  if (selected && rows > 0) {
    const bool ok = expert >= 0 && expert < p.E && row_start >= 0 && (int64_t)row_start + rows <= p.s_cap &&
                    is_dynamic - 2 < p.n_recv_slots;
    if (ok) tiles = (rows + kRows - 1) / kRows;
    else atomicOr(p.status, FEPLB_ST_GROUP);
  }
  t->g_row_start[idx] = row_start;
  t->g_rows[idx] = rows;
  // expert id in the low half; receive slot + 1 in the high half (0 = weights at home)
  t->g_expert[idx] = (expert & 0xffff) | ((is_dynamic >= 2 ? is_dynamic - 1 : 0) << 16);
  return tiles;
}

// In-place inclusive scan of t->prefix[first+1 .. first+n] (tile counts) by one warp; prefix[first] is the base.
__device__ __forceinline__ void warp_scan_prefix(SmemTail* t, int first, int n, int lane) {
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

template <bool SWIGLU, bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
k_grouped_gemm(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_ra,
               const __grid_constant__ CUtensorMap tm_b0,
               const __grid_constant__ CUtensorMap tm_b1, const __grid_constant__ CUtensorMap tm_r0,
               const __grid_constant__ CUtensorMap tm_r1, const __grid_constant__ CUtensorMap tm_out, const GemmParams p) {
  constexpr int kStages = Ring<PAIR>::kStages, kStageBytes = Ring<PAIR>::kStageBytes;
  constexpr int kTileRows = Ring<PAIR>::kTileRows;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* epi_smem = smem + (size_t)kRingBytes;
  // pair form: rank of this CTA in its cluster of two (0 = leader, issues the MMAs), work is dealt
  // per cluster; single form: every CTA is its own leader
  const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  SmemTail* tail = reinterpret_cast<SmemTail*>(epi_smem + (size_t)kEpiWarps * kEpiStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &tail->abort_flag;

  // Programmatic dependent launch: the next kernel of the stream may be scheduled as soon as SMs
  // free up (its set-up then overlaps this grid's tail); it waits for this grid's results itself.
  asm volatile("griddepcontrol.launch_dependents;");

  // ---- set-up: barriers, TMEM, group table ------------------------------------------------
  if (threadIdx.x == 0) {
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_ra);
    prefetch_tmap(&tm_b0);
    prefetch_tmap(&tm_b1);
    prefetch_tmap(&tm_r0);
    prefetch_tmap(&tm_r1);
    prefetch_tmap(&tm_out);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&tail->full[s]), 1);
      mbar_init(smem_u32(&tail->empty[s]), 1);
    }
    for (int a = 0; a < kAccStages; ++a) {
      mbar_init(smem_u32(&tail->tmem_full[a]), 1);
      // one arrival per epilogue warp (of both CTAs in the pair form: the leader's barrier collects them)
      mbar_init(smem_u32(&tail->tmem_empty[a]), PAIR ? 2 * kEpiWarps : kEpiWarps);
    }
    mbar_init(smem_u32(&tail->dyn_bar), 1);
    tail->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    __syncwarp();
    if (PAIR) {
      tmem_alloc_pair(smem_u32(&tail->tmem_base), kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(&tail->tmem_base), kTmemCols);
      tmem_relinquish();
    }
  }
  // everything above touched only this CTA's resources; from here on the results of the kernels
  // before this one (rows, group table) are read
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (p.stamps && threadIdx.x == 0) atomicMin(&p.stamps[0], global_timer_ns());
  for (int g = threadIdx.x; g < p.n_groups; g += kThreads) {
    const feplb_group gr = p.groups[g];
    const bool selected = p.which == FEPLB_FFN_ALL || (p.which == FEPLB_FFN_STATIC) == (gr.is_dynamic == 0);
    tail->prefix[g + 1] = put_group<kTileRows>(tail, g, gr.expert, gr.row_start, gr.rows, gr.is_dynamic, selected, p);   // scanned below
  }
  if (threadIdx.x == 0) tail->prefix[0] = 0;
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    warp_scan_prefix(tail, 0, p.n_groups, lane);
    if (lane == 0) {
      tail->n_entries = p.n_groups;
      tail->total_mtiles = tail->prefix[p.n_groups];
    }
  }
  __syncthreads();
  if (PAIR) cluster_sync_all();   // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tail->tmem_base;
  const bool has_dyn = p.dyn.seq != 0;
  const int n_static_entries = p.n_groups;
  const int n_static_tiles = tail->prefix[p.n_groups] * p.n_tiles_n;
  const uint32_t b_half_bytes = (uint32_t)p.bn * BK * 2;
  const uint32_t stage_tx = PAIR ? 2 * (kABytes + b_half_bytes) : kABytes + 2 * b_half_bytes;

  if (warp == 0) {
    // ---- TMA producer (lane 0 issues; the whole warp fetches the dynamic table) ----------------
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true, dyn_known = !has_dyn;
    int n_entries = n_static_entries, total = n_static_tiles;
    // Reads the n_dyn groups of the dynamic table from its device copy, appends its entries and tells
    // the other roles; false if an entry does not carry this forward's sequence number yet.
    auto take_table = [&](int n_dyn) -> bool {
      if (n_dyn < 0 || n_static_entries + n_dyn > FEPLB_MAX_GROUPS) {
        if (lane == 0) atomicOr(p.status, FEPLB_ST_GROUP);
        n_dyn = 0;
      }
      bool good = true;
      for (int i = lane; i < n_dyn; i += 32) {
        int e, rs, rw, dy;
        if (!dyn_entry(p.dyn, i, e, rs, rw, dy)) { good = false; continue; }
        tail->prefix[n_static_entries + i + 1] = put_group<kTileRows>(tail, n_static_entries + i, e, rs, rw, dy, true, p);
      }
      if (!__all_sync(0xffffffffu, good)) return false;
      warp_scan_prefix(tail, n_static_entries, n_dyn, lane);
      n_entries = n_static_entries + n_dyn;
      total = tail->prefix[n_entries] * p.n_tiles_n;
      if (lane == 0) {
        tail->n_entries = n_entries;
        tail->total_mtiles = tail->prefix[n_entries];
        mbar_arrive(smem_u32(&tail->dyn_bar));      // release: the entries above are visible to the waiters
      }
      dyn_known = true;
      return true;
    };
    bool claimer = false, tried_claim = false;
    for (int tile = worker; ok; tile += n_workers) {
      if (!dyn_known && tile >= total) {
        // Out of static tiles: now the table is needed (bounded wait; see feplb_dyn.cuh).
        const unsigned long long t0 = global_timer_ns();
        if (p.stamps && lane == 0) atomicMin(&p.stamps[1], t0);
        while (!dyn_known) {
          const int n_dyn = dyn_wait_table(p.dyn, lane, abort_flag, p.status, t0, claimer, tried_claim);
          if (n_dyn == kDynAbort) { ok = false; break; }
          // no table within the limit: go on as if it were empty, so that the static tiles still in
          // flight in this CTA complete normally; the status word carries the reason
          if (!take_table(n_dyn == kDynGaveUp ? 0 : n_dyn) && global_timer_ns() - t0 > p.dyn.wait_limit_ns + kWaitLimitNs) {
            if (lane == 0) atomicOr(p.status, FEPLB_ST_PLAN);
            take_table(0);
          }
        }
        if (!ok) break;
        if (p.stamps && lane == 0) atomicMin(&p.stamps[3], ~(global_timer_ns() - t0));
      }
      if (tile >= total) break;
      const TileCoord c = tile_coord<kTileRows>(tail, n_entries, p.n_tiles_n, tile);
      // While static tiles remain, peek at the device-side word once per tile: the load is in flight
      // during the K loop below and is looked at after it, so it costs the pipeline nothing.
      unsigned long long peek = 0;
      if (!dyn_known && lane == 0) peek = ld_relaxed_gpu_u64(p.dyn.ready_dev);
      if (lane == 0) {
        // weights of a migrated expert come from its slot of the receive buffer, and in pass 1 its
        // rows from the receive region of the rows (same row numbers as the permuted buffer)
        const CUtensorMap* ma = c.slot >= 0 ? &tm_ra : &tm_a;
        const CUtensorMap* mb0 = c.slot >= 0 ? &tm_r0 : &tm_b0;
        const CUtensorMap* mb1 = c.slot >= 0 ? &tm_r1 : &tm_b1;
        const int brow0 = (c.slot >= 0 ? c.slot : c.expert) * p.b_rows_per_expert + (SWIGLU ? c.nt * p.bn : c.nt * 2 * p.bn);
        const int brow1 = SWIGLU ? brow0 : brow0 + p.bn;
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->empty[stage]), phase ^ 1u, abort_flag, p.status))) break;
          const uint32_t full = smem_u32(&tail->full[stage]);
          const uint32_t sa = smem_u32(smem + (size_t)stage * kStageBytes);
          const uint32_t sb = sa + kABytes;
          if (PAIR) {
            // both CTAs credit the LEADER's barrier; the leader announces the bytes of both.  A tile
            // whose second 128 rows hold no valid row (a group of at most 128 rows, or a ragged
            // tail) needs no A rows in the peer: it skips that load (the MMA then multiplies
            // whatever its stage holds into accumulator rows nobody stores), so a small group costs
            // the pair no more operand traffic than it would cost a single CTA.
            const uint32_t full0 = map_to_cta(full, 0);
            const bool peer_rows = c.rows_valid > BM;
            if (cta_rank == 0) mbar_expect_tx(full, peer_rows ? stage_tx : stage_tx - kABytes);
            if (cta_rank == 0 || peer_rows) tma_load_2d_pair(sa, ma, full0, kb * BK, c.row0 + (int)cta_rank * BM);
            if (cta_rank == 0) tma_load_2d_pair(sb, mb0, full0, kb * BK, brow0);
            else tma_load_2d_pair(sb, mb1, full0, kb * BK, brow1);
          } else {
            mbar_expect_tx(full, stage_tx);
            tma_load_2d(sa, ma, full, kb * BK, c.row0);
            tma_load_2d(sb, mb0, full, kb * BK, brow0);
            tma_load_2d(sb + b_half_bytes, mb1, full, kb * BK, brow1);
          }
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
      // leave time for copies already issued to land before the CTA's shared memory goes away
      for (int i = 0; i < 2000; ++i) __nanosleep(100);
    }
  } else if (warp == 1) {
    // ---- MMA issuer -------------------------------------------------------------------------
    if (lane == 0 && cta_rank == 0) {
      const uint32_t idesc = make_idesc(kTileRows, 2 * p.bn);
      int stage = 0, as = 0;
      uint32_t phase = 0, aphase = 0;
      bool ok = true, dyn_known = !has_dyn;
      int total = n_static_tiles;
      for (int tile = worker; ok; tile += n_workers) {
        if (tile >= total) {
          if (dyn_known) break;
          if (!(ok = mbar_wait(smem_u32(&tail->dyn_bar), 0, abort_flag, p.status, p.dyn.wait_limit_ns + 2 * kWaitLimitNs))) break;
          dyn_known = true;
          total = tail->total_mtiles * p.n_tiles_n;
          if (tile >= total) break;
        }
        if (!(ok = mbar_wait(smem_u32(&tail->tmem_empty[as]), aphase ^ 1u, abort_flag, p.status))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * kAccCols);
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->full[stage]), phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)stage * kStageBytes);
          const uint64_t da = make_smem_desc(sa);
          const uint64_t db = make_smem_desc(sa + kABytes);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // +32 bytes (>> 4 = 2) per K step inside the 128-byte swizzle row
            if (PAIR) umma_bf16_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (uint32_t)((kb | k) != 0));
            else umma_bf16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (uint32_t)((kb | k) != 0));
          }
          // stage reusable (in both CTAs of a pair) once these MMAs have read it
          if (PAIR) umma_commit_pair(smem_u32(&tail->empty[stage]));
          else umma_commit(smem_u32(&tail->empty[stage]));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        // accumulator complete (announced to the epilogue warps of both CTAs of a pair)
        if (PAIR) umma_commit_pair(smem_u32(&tail->tmem_full[as]));
        else umma_commit(smem_u32(&tail->tmem_full[as]));
        if (++as == kAccStages) { as = 0; aphase ^= 1u; }
      }
    }
  } else {
    // ---- epilogue: TMEM -> registers -> bf16 -> (warp-private smem transpose) -> global -------
    // A thread owns one accumulator row, so storing straight from registers would scatter 16-byte
    // pieces over 32 rows per instruction.  Instead each warp stages 32 rows x 64 columns (128 B
    // per row, 16-byte chunks XOR-swizzled by row) and writes them back out 4 rows per
    // instruction: every store covers whole 128-byte lines, masked per row for ragged tiles.
    const int q = warp & 3;                   // TMEM lane quarter this warp may read
    const uint32_t stg = smem_u32(epi_smem + (size_t)(warp - 2) * kEpiStageBytes);
    const int out_cols = SWIGLU ? p.bn : 2 * p.bn;
    int as = 0;
    uint32_t aphase = 0;
    bool ok = true, dyn_known = !has_dyn;
    int n_entries = n_static_entries, total = n_static_tiles;
    for (int tile = worker; ok; tile += n_workers) {
      if (tile >= total) {
        if (dyn_known) break;
        ok = mbar_wait(smem_u32(&tail->dyn_bar), 0, abort_flag, p.status, p.dyn.wait_limit_ns + 2 * kWaitLimitNs);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        dyn_known = true;
        n_entries = tail->n_entries;
        total = tail->total_mtiles * p.n_tiles_n;
        if (tile >= total) break;
      }
      const TileCoord c = tile_coord<kTileRows>(tail, n_entries, p.n_tiles_n, tile);
      ok = mbar_wait(smem_u32(&tail->tmem_full[as]), aphase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * kAccCols);
      const int row_off = (int)cta_rank * BM + q * 32;    // this warp's first row inside the tile
      const int rows_here = c.rows_valid - row_off;       // valid rows among this warp's 32
      __nv_bfloat16* obase = p.out + (int64_t)(c.row0 + row_off) * p.ld_out + (int64_t)c.nt * out_cols;
      uint32_t a0[32], a1[32], b0[32], b1[32], packed[32];
      tmem_ld32(taddr, a0);
      tmem_ld32(taddr + 32u, a1);
      if (SWIGLU) {
        tmem_ld32(taddr + (uint32_t)p.bn, b0);
        tmem_ld32(taddr + (uint32_t)p.bn + 32u, b1);
      }
      for (int col = 0; col < out_cols; col += 64) {
        tmem_ld_wait();
        if (SWIGLU && p.ab_out != nullptr) {
          // training: also keep the pre-activations a | b of these 64 hidden units (bf16) for the
          // backward pass, in [rows, 2f] with b at column offset f
          __nv_bfloat16* abase = p.ab_out + (int64_t)(c.row0 + row_off) * (2 * p.ld_out);
          const int hcol = c.nt * out_cols + col;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            packed[i] = pack_bf16x2(__uint_as_float(a0[2 * i]), __uint_as_float(a0[2 * i + 1]));
            packed[16 + i] = pack_bf16x2(__uint_as_float(a1[2 * i]), __uint_as_float(a1[2 * i + 1]));
          }
          stage_and_store(stg, packed, abase, 2 * p.ld_out, hcol, rows_here, lane);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            packed[i] = pack_bf16x2(__uint_as_float(b0[2 * i]), __uint_as_float(b0[2 * i + 1]));
            packed[16 + i] = pack_bf16x2(__uint_as_float(b1[2 * i]), __uint_as_float(b1[2 * i + 1]));
          }
          stage_and_store(stg, packed, abase, 2 * p.ld_out, p.ld_out + hcol, rows_here, lane);
        }
        convert_slice<SWIGLU>(a0, b0, packed);
        convert_slice<SWIGLU>(a1, b1, packed + 16);
        if (col + 64 < out_cols) {           // next slice's TMEM loads fly while this one is stored
          tmem_ld32(taddr + (uint32_t)(col + 64), a0);
          tmem_ld32(taddr + (uint32_t)(col + 96), a1);
          if (SWIGLU) {
            tmem_ld32(taddr + (uint32_t)(p.bn + col + 64), b0);
            tmem_ld32(taddr + (uint32_t)(p.bn + col + 96), b1);
          }
        }
        if (rows_here >= 32) stage_and_tma_store(stg, packed, &tm_out, c.nt * out_cols + col, c.row0 + row_off, lane);
        else stage_and_store(stg, packed, obase, p.ld_out, col, rows_here, lane);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tail->tmem_empty[as]), 0));
        else mbar_arrive(smem_u32(&tail->tmem_empty[as]));
      }
      if (++as == kAccStages) { as = 0; aphase ^= 1u; }
    }
    staging_ready(lane);      // the staging area must outlive the last TMA store that reads it
  }

  // ---- teardown ---------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (p.stamps && threadIdx.x == 0) atomicMin(&p.stamps[2], ~global_timer_ns());
  if (PAIR) cluster_sync_all();   // the leader's MMAs read the peer's shared memory: leave together
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing will ever complete.
// The wait must give up after limit_ns, raise FEPLB_ST_WAIT and let the kernel return normally.
__global__ void k_wait_selftest(uint32_t* status, unsigned long long limit_ns, int* gave_up) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    fence_barrier_init();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, limit_ns);
    *gave_up = ok ? 0 : 1;
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

template <bool SWIGLU, bool PAIR>
cudaError_t launch_one(const CUtensorMap& ta, const CUtensorMap& tra, const CUtensorMap& tb0, const CUtensorMap& tb1, const CUtensorMap& tr0,
                       const CUtensorMap& tr1, const CUtensorMap& tout, const GemmParams& p, int num_sms, cudaStream_t st) {
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
  cfg.attrs = at;
  cfg.numAttrs = 1;
  if (PAIR) {
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = 2;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  if (!grid) {
    cudaError_t e = cudaFuncSetAttribute(k_grouped_gemm<SWIGLU, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    int g = num_sms;
    if (PAIR) {
      // as many clusters of two as can be resident at once (one CTA per SM, both SMs in one GPC)
      int n_clusters = 0;
      cfg.gridDim = dim3(num_sms / 2 * 2);
      e = cudaOccupancyMaxActiveClusters(&n_clusters, k_grouped_gemm<SWIGLU, PAIR>, &cfg);
      if (e != cudaSuccess) return e;
      if (n_clusters < 1) return cudaErrorLaunchOutOfResources;
      g = 2 * (n_clusters < num_sms / 2 ? n_clusters : num_sms / 2);
    }
    grid = g;
  }
  cfg.gridDim = dim3(grid);
  return cudaLaunchKernelEx(&cfg, k_grouped_gemm<SWIGLU, PAIR>, ta, tra, tb0, tb1, tr0, tr1, tout, p);
}

}  // namespace

int feplb_launch_expert_ffn(const feplb_gemm_args& a, cudaStream_t st, int64_t* n_launch, char* err, size_t errn,
                            const feplb_wm_dyn* dyn) {
  if ((a.n_groups == 0 && !(dyn && dyn->seq)) || a.s_cap == 0) return FEPLB_OK;
  if (dyn && a.n_groups + dyn->max_groups > FEPLB_MAX_GROUPS) {
    snprintf(err, errn, "expert_ffn: the two group tables of a merged launch exceed %d entries", FEPLB_MAX_GROUPS);
    return FEPLB_E_INVALID;
  }
  // pass 1: H = silu(X W1) * (X W3);  N tile = bn columns of H, MMA N = 2*bn
  const int bn1 = (a.f % 128 == 0) ? 128 : 64;
  // pass 2: Y = H W2;  N tile = 2*bn columns of Y
  const int bn2 = (a.d % 256 == 0) ? 128 : 64;
  CUtensorMap tm_x, tm_w1, tm_w3, tm_h, tm_w2, tm_ho, tm_yo;     // tm_ho, tm_yo: outputs in boxes of 32 rows x 64 columns
  if (!make_tmap(&tm_x, a.x_perm, (uint64_t)a.s_cap, (uint64_t)a.d, BM) ||
      !make_tmap(&tm_w1, a.w1, (uint64_t)a.E * a.f, (uint64_t)a.d, bn1) ||
      !make_tmap(&tm_w3, a.w3, (uint64_t)a.E * a.f, (uint64_t)a.d, bn1) ||
      !make_tmap(&tm_h, a.h, (uint64_t)a.s_cap, (uint64_t)a.f, BM) ||
      !make_tmap(&tm_w2, a.w2, (uint64_t)a.E * a.d, (uint64_t)a.f, bn2) ||
      !make_tmap(&tm_ho, a.h, (uint64_t)a.s_cap, (uint64_t)a.f, 32) ||
      !make_tmap(&tm_yo, a.y, (uint64_t)a.s_cap, (uint64_t)a.d, 32)) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed (driver entry point missing or bad pointer/shape)");
    return FEPLB_E_CUDA;
  }
  // receive buffer of migrated experts' weights, addressed by slot like the home weights by expert
  CUtensorMap tm_r1 = tm_w1, tm_r3 = tm_w3, tm_r2 = tm_w2;
  const bool has_recv = a.recv_w1 && a.recv_w3 && a.recv_w2 && a.n_recv_slots > 0;
  if (has_recv && (!make_tmap(&tm_r1, a.recv_w1, (uint64_t)a.n_recv_slots * a.f, (uint64_t)a.d, bn1) ||
                   !make_tmap(&tm_r3, a.recv_w3, (uint64_t)a.n_recv_slots * a.f, (uint64_t)a.d, bn1) ||
                   !make_tmap(&tm_r2, a.recv_w2, (uint64_t)a.n_recv_slots * a.d, (uint64_t)a.f, bn2))) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed for the receive buffer");
    return FEPLB_E_CUDA;
  }
  // rows of migrated pieces: pass 1 reads them from the receive region when there is one
  CUtensorMap tm_rx = tm_x;
  if (has_recv && a.recv_x && !make_tmap(&tm_rx, a.recv_x, (uint64_t)a.s_cap, (uint64_t)a.d, BM)) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed for the receive region of the rows");
    return FEPLB_E_CUDA;
  }
  GemmParams p1;
  p1.n_recv_slots = has_recv ? a.n_recv_slots : 0;
  p1.groups = a.groups; p1.n_groups = a.n_groups; p1.which = a.which; p1.E = a.E; p1.s_cap = a.s_cap;
  p1.n_tiles_n = a.f / bn1; p1.num_k_blocks = a.d / BK; p1.b_rows_per_expert = a.f; p1.bn = bn1;
  p1.out = (__nv_bfloat16*)a.h; p1.ld_out = a.f; p1.status = a.status; p1.ab_out = (__nv_bfloat16*)a.ab_out;
  const feplb_wm_dyn none;
  p1.dyn = feplb_dyn_table(dyn ? *dyn : none);
  p1.stamps = dyn ? dyn->stamps : nullptr;
  GemmParams p2 = p1;
  p2.n_tiles_n = a.d / (2 * bn2); p2.num_k_blocks = a.f / BK; p2.b_rows_per_expert = a.d; p2.bn = bn2;
  p2.out = (__nv_bfloat16*)a.y; p2.ld_out = a.d; p2.ab_out = nullptr;
  p2.stamps = p1.stamps ? p1.stamps + 4 : nullptr;

  cudaError_t e = a.pair ? launch_one<true, true>(tm_x, tm_rx, tm_w1, tm_w3, tm_r1, tm_r3, tm_ho, p1, a.num_sms, st)
                         : launch_one<true, false>(tm_x, tm_rx, tm_w1, tm_w3, tm_r1, tm_r3, tm_ho, p1, a.num_sms, st);
  ++*n_launch;
  if (e == cudaSuccess) {
    e = a.pair ? launch_one<false, true>(tm_h, tm_h, tm_w2, tm_w2, tm_r2, tm_r2, tm_yo, p2, a.num_sms, st)
               : launch_one<false, false>(tm_h, tm_h, tm_w2, tm_w2, tm_r2, tm_r2, tm_yo, p2, a.num_sms, st);
    ++*n_launch;
  }
  if (e != cudaSuccess) {
    snprintf(err, errn, "k_grouped_gemm launch: %s", cudaGetErrorString(e));
    return FEPLB_E_CUDA;
  }
  return FEPLB_OK;
}

cudaError_t feplb_launch_wait_selftest(uint32_t* status, unsigned long long limit_ns, int* gave_up, cudaStream_t st) {
  k_wait_selftest<<<1, 32, 0, st>>>(status, limit_ns, gave_up);
  return cudaGetLastError();
}
