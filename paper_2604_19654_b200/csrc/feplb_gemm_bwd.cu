// Backward pass of the grouped SwiGLU expert FFN on sm_100a (the paper reports backward layer times
// in Table 2 but does not describe the pass; this is the derivative of the forward definition,
// computed over the same groups).  One warp-specialised tcgen05 kernel in three kinds, operands
// staged by TMA.  DH and DX take K-major operands (the weights are transposed once per weight
// update, their contraction runs over the forward layout's slow dimension); WG takes MN-major
// operands, i.e. the row-major activations as they lie, the contraction running over rows:
//   DH: dH = dY W2 (A = dY rows, B = W2^T tiles), epilogue applies the SwiGLU derivative with the
//       saved pre-activations:  dA = dH * b * silu'(a),  dB = dH * silu(a)  -> dAB [rows, 2f]
//   DX: dX = dA W1^T + dB W3^T as ONE contraction over K = 2f ([dA|dB] against W1^T then W3^T)
//   WG: weight gradients, one (expert, M tile, N tile) per tile with the contraction running over
//       that expert's rows:  dW[e] = P_e^T Q_e  (fp32 out, optionally accumulated), P [rows, M] and
//       Q [rows, N] read in boxes of 64 columns x 64 rows, padding rows zeroed beforehand
// Pipeline as in the forward kernel: warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps
// 2..5 epilogue; 4-stage ring of 48 KiB; two TMEM accumulators; every mbarrier wait bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>

#include "feplb_internal.h"
#include "feplb_tc.cuh"

namespace {

enum { KIND_DH = 0, KIND_DX = 1, KIND_WG = 2 };

constexpr int BM = FEPLB_TILE_M;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int kAccCols = 256;
constexpr int kTmemCols = 512;
constexpr int kABytes = BM * BK * 2;
constexpr int kBBytesMax = 256 * BK * 2;
constexpr int kStages = 4;
constexpr int kAccStages = 2;
constexpr int kStageBytes = kABytes + kBBytesMax;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kEpiStageBytes = 32 * 128;
// The weight-gradient kind gives up one ring stage for output staging: each epilogue warp owns
// kWgBufs buffers of 32 rows x 32 fp32 (4 KiB, 128-byte swizzled) that TMA stores or reduce-adds
// drain to dW while the warp fills the next one.
constexpr int kWgStages = 3;
constexpr int kWgBufs = 4;
static_assert(kWgBufs * kEpiWarps * kEpiStageBytes <= kABytes + kBBytesMax + kEpiWarps * kEpiStageBytes, "staging fits the freed stage");
// Pair form (cta_group::2): a cluster of two CTAs computes a 256 x 256 tile; each CTA stages its own
// 128 rows (columns, for the MN-major kind) of A and half of the B tile, 32 KiB per stage.
constexpr int kPairStageBytes = kABytes + 128 * BK * 2;
constexpr int kPairStages = 6;
constexpr int kPairWgStages = 4;
constexpr int kMaxStages = 6;

template <int KIND, bool PAIR>
struct Ring {
  static constexpr int kNS = PAIR ? (KIND == 2 ? kPairWgStages : kPairStages) : (KIND == 2 ? kWgStages : kStages);
  static constexpr int kBytes = PAIR ? kPairStageBytes : kStageBytes;
  static constexpr int kTileRows = PAIR ? 2 * BM : BM;
  static_assert(kNS <= kMaxStages && kNS * kBytes + (KIND == 2 ? kWgBufs : 1) * kEpiWarps * kEpiStageBytes <=
                kStages * kStageBytes + kEpiWarps * kEpiStageBytes, "ring + staging fit below the tail");
};

struct Tail {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long tmem_full[kAccStages];
  unsigned long long tmem_empty[kAccStages];
  uint32_t tmem_base;
  int abort_flag;
  int prefix[FEPLB_MAX_GROUPS + 1];
  int g_row_start[FEPLB_MAX_GROUPS];
  int g_rows[FEPLB_MAX_GROUPS];
  int g_expert[FEPLB_MAX_GROUPS];
};
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + (size_t)kEpiWarps * kEpiStageBytes + sizeof(Tail);
static_assert(kSmemBytes <= 232448 && kSmemBytes > 116 * 1024, "one CTA per SM: each allocates all of TMEM");

struct BwdParams {
  const feplb_group* groups;   // DH/DX: the group table; WG: the E-entry home table (one entry per expert)
  int n_groups;
  int which;
  int E;
  int64_t s_cap;
  int n_tiles_n;               // N tiles per M tile
  int num_k_blocks;            // DH: d/64, DX: 2f/64, WG: unused (ceil(rows/64) per expert)
  int k_switch;                // DX: first K block served by the second B map (f/64)
  int n_limit;                 // DH/DX: valid output columns (a last N tile may overhang)
  int b_rows_per_expert;       // DH: f, DX: d, WG: 0 (B^T is not per expert)
  int bn;                      // rows of one B half tile; the MMA has N = 2*bn
  __nv_bfloat16* out;          // DH: dAB [s_cap, 2f]; DX: dX_perm [s_cap, d]
  int ld_out;
  const __nv_bfloat16* ab;     // DH: saved pre-activations [s_cap, 2f] (a | b)
  int f;                       // DH: columns of a (and offset of b)
  float* wout;                 // WG: fp32 [E, m_total, n_total]
  int m_total, n_total;        // WG
  int m_tiles;                 // WG: M tiles per expert
  int accumulate;              // WG: add to wout instead of overwriting it
  uint32_t* status;
};

struct Coord { int row0, rows_valid, expert, mt, nt, kblocks; };

template <int KIND, int TR>
__device__ __forceinline__ Coord tile_coord(const Tail* t, const BwdParams& p, int tile) {
  Coord c;
  if (KIND == KIND_WG) {
    const int per = p.m_tiles * p.n_tiles_n;
    const int g = tile / per;
    const int r = tile - g * per;
    c.mt = r / p.n_tiles_n;
    c.nt = r - c.mt * p.n_tiles_n;
    c.expert = t->g_expert[g];
    c.row0 = t->g_row_start[g];               // first row of the expert's segment = start of its K range
    c.rows_valid = t->g_rows[g];
    c.kblocks = (t->g_rows[g] + BK - 1) / BK;
    return c;
  }
  const int mt = tile / p.n_tiles_n;
  int lo = 0, hi = p.n_groups;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (t->prefix[mid] <= mt) lo = mid; else hi = mid;
  }
  const int local = mt - t->prefix[lo];
  c.row0 = t->g_row_start[lo] + local * TR;
  c.rows_valid = min(TR, t->g_rows[lo] - local * TR);
  c.expert = t->g_expert[lo];
  c.mt = mt;
  c.nt = tile - mt * p.n_tiles_n;
  c.kblocks = p.num_k_blocks;
  return c;
}

// Shared-memory descriptor of an MN-major operand tile staged as 64-element (128-byte) wide boxes of
// 64 K rows each, 128-byte swizzled: consecutive K rows are 128 bytes apart, groups of 8 K rows
// 1024 bytes (stride byte offset), consecutive 64-element chunks along M or N one box = 8192 bytes
// (leading byte offset) apart.
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(8192 >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor as make_idesc, with both operands MN-major (bits 15 and 16).
__device__ __forceinline__ uint32_t make_idesc_mn(int m, int n) { return make_idesc(m, n) | (1u << 15) | (1u << 16); }

__device__ __forceinline__ float sigmoid_f(float a) { return __fdividef(1.f, 1.f + __expf(-a)); }
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Stage 32 rows x 64 bf16 columns (packed[32] per lane = its row) through the warp's swizzled
// staging area and write them out 4 rows per instruction, whole 128-byte lines, row-masked.
__device__ __forceinline__ void staged_store(uint32_t stg, const uint32_t* packed, __nv_bfloat16* obase, int ld_out,
                                             int col, int rows_here, int lane) {
  const int rd_row = lane >> 3, rd_chunk = lane & 7;
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
    if (r < rows_here) *reinterpret_cast<uint4*>(obase + (int64_t)r * ld_out + col + rd_chunk * 8) = v;
  }
  __syncwarp();
}

// 3-d tiled TMA load (the MN-major operands: 64 columns x 64 rows x several 64-column chunks).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// The same, in the pair form: the byte count is credited to an mbarrier of the pair's leader.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// TMA store / reduce-add of one staged 32 x 32 fp32 box to dW[e] (tensor map over [E, M, N]).
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* m, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(m), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* m, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(m), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int KIND, bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
k_ffn_bwd_gemm(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
               const __grid_constant__ CUtensorMap tm_b1, const __grid_constant__ CUtensorMap tm_out, const BwdParams p) {
  constexpr int NS = Ring<KIND, PAIR>::kNS;                       // ring stages
  constexpr int kSB = Ring<KIND, PAIR>::kBytes;                   // bytes per stage
  constexpr int TR = Ring<KIND, PAIR>::kTileRows;                 // rows (WG: M columns) of a tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* epi_smem = smem + (size_t)NS * kSB;
  // pair form: rank in the cluster of two (0 = leader, issues the MMAs); tiles are dealt per cluster
  const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  Tail* tail = reinterpret_cast<Tail*>(smem + (size_t)kStages * kStageBytes + (size_t)kEpiWarps * kEpiStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &tail->abort_flag;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b0);
    prefetch_tmap(&tm_b1);
    if (KIND == KIND_WG) prefetch_tmap(&tm_out);
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&tail->full[s]), 1);
      mbar_init(smem_u32(&tail->empty[s]), 1);
    }
    for (int a = 0; a < kAccStages; ++a) {
      mbar_init(smem_u32(&tail->tmem_full[a]), 1);
      mbar_init(smem_u32(&tail->tmem_empty[a]), PAIR ? 2 * kEpiWarps : kEpiWarps);
    }
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
  for (int g = threadIdx.x; g < p.n_groups; g += kThreads) {
    const feplb_group gr = p.groups[g];
    const bool selected = p.which == FEPLB_FFN_ALL || (p.which == FEPLB_FFN_STATIC) == (gr.is_dynamic == 0);
    int tiles = 0, rows = 0;
    if (selected && gr.rows > 0) {
      const bool ok = gr.expert >= 0 && gr.expert < p.E && gr.row_start >= 0 && (int64_t)gr.row_start + gr.rows <= p.s_cap;
      if (ok) { tiles = (gr.rows + TR - 1) / TR; rows = gr.rows; }
      else atomicOr(p.status, FEPLB_ST_GROUP);
    }
    tail->prefix[g + 1] = tiles;
    tail->g_row_start[g] = gr.row_start;
    tail->g_rows[g] = rows;                      // 0 for unselected or malformed entries
    tail->g_expert[g] = gr.expert;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    const int per = (p.n_groups + 31) / 32;
    const int g0 = lane * per, g1 = min(p.n_groups, g0 + per);
    int sum = 0;
    for (int g = g0; g < g1; ++g) sum += tail->prefix[g + 1];
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    int run = incl - sum;
    for (int g = g0; g < g1; ++g) {
      const int t = tail->prefix[g + 1];
      run += t;
      tail->prefix[g + 1] = run;
    }
    if (lane == 0) tail->prefix[0] = 0;
  }
  __syncthreads();
  if (PAIR) cluster_sync_all();   // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tail->tmem_base;
  const int total_tiles = KIND == KIND_WG ? p.n_groups * p.m_tiles * p.n_tiles_n : tail->prefix[p.n_groups] * p.n_tiles_n;
  const uint32_t b_half_bytes = (uint32_t)p.bn * BK * 2;
  const uint32_t stage_tx = PAIR ? 2 * (kABytes + b_half_bytes) : kABytes + 2 * b_half_bytes;

  if (warp == 0) {
    // ---- TMA producer ---------------------------------------------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
        const Coord c = tile_coord<KIND, TR>(tail, p, tile);
        for (int kb = 0; kb < c.kblocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->empty[stage]), phase ^ 1u, abort_flag, p.status))) break;
          const uint32_t full = smem_u32(&tail->full[stage]);
          const uint32_t sa = smem_u32(smem + (size_t)stage * kSB);
          const uint32_t sb = sa + kABytes;
          if (PAIR) {
            // both CTAs credit the LEADER's barrier; the leader announces the bytes of both.  Each
            // CTA brings its own 128 rows (WG: columns) of A and its half of the B tile.
            const uint32_t full0 = map_to_cta(full, 0);
            if (cta_rank == 0) mbar_expect_tx(full, stage_tx);
            if (KIND == KIND_WG) {
              const int k0 = c.row0 + kb * BK;
              tma_load_3d_pair(sa, &tm_a, full0, 0, k0, c.mt * (TR / 64) + (int)cta_rank * (BM / 64));
              tma_load_3d_pair(sb, &tm_b0, full0, 0, k0, c.nt * (2 * p.bn / 64) + (int)cta_rank * (p.bn / 64));
            } else {
              const CUtensorMap* mb = (KIND == KIND_DX && kb >= p.k_switch) ? &tm_b1 : &tm_b0;
              const int kb_b = (KIND == KIND_DX && kb >= p.k_switch) ? kb - p.k_switch : kb;
              const int brow = c.expert * p.b_rows_per_expert + c.nt * 2 * p.bn + (int)cta_rank * p.bn;
              tma_load_2d_pair(sa, &tm_a, full0, kb * BK, c.row0 + (int)cta_rank * BM);
              tma_load_2d_pair(sb, mb, full0, kb_b * BK, brow);
            }
            if (++stage == NS) { stage = 0; phase ^= 1u; }
            continue;
          }
          mbar_expect_tx(full, stage_tx);
          if (KIND == KIND_WG) {
            // K runs along the expert's rows: both operands are read as they lie in memory (row = K,
            // columns = M resp. N contiguous).  The maps see a matrix as [64-column chunk][row][64
            // columns], so one load brings 64 rows of all the tile's chunks, 8 KiB per chunk.
            const int k0 = c.row0 + kb * BK;
            tma_load_3d(sa, &tm_a, full, 0, k0, c.mt * (TR / 64));
            tma_load_3d(sb, &tm_b0, full, 0, k0, c.nt * (2 * p.bn / 64));
          } else {
            const CUtensorMap* mb = (KIND == KIND_DX && kb >= p.k_switch) ? &tm_b1 : &tm_b0;
            const int kb_b = (KIND == KIND_DX && kb >= p.k_switch) ? kb - p.k_switch : kb;
            const int brow = c.expert * p.b_rows_per_expert + c.nt * 2 * p.bn;
            tma_load_2d(sa, &tm_a, full, kb * BK, c.row0);
            tma_load_2d(sb, mb, full, kb_b * BK, brow);
            tma_load_2d(sb + b_half_bytes, mb, full, kb_b * BK, brow + p.bn);
          }
          if (++stage == NS) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(100);
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer -------------------------------------------------------------------------
    if (lane == 0 && cta_rank == 0) {
      const uint32_t idesc = KIND == KIND_WG ? make_idesc_mn(TR, 2 * p.bn) : make_idesc(TR, 2 * p.bn);
      int stage = 0, as = 0;
      uint32_t phase = 0, aphase = 0;
      bool ok = true;
      for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
        const Coord c = tile_coord<KIND, TR>(tail, p, tile);
        if (!(ok = mbar_wait(smem_u32(&tail->tmem_empty[as]), aphase ^ 1u, abort_flag, p.status))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * kAccCols);
        for (int kb = 0; kb < c.kblocks; ++kb) {
          if (!(ok = mbar_wait(smem_u32(&tail->full[stage]), phase, abort_flag, p.status))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)stage * kSB);
          // descriptor step per UMMA_K: MN-major 16 K rows of 128 bytes (2048 >> 4), K-major 32 bytes (>> 4)
          const uint64_t da = KIND == KIND_WG ? make_smem_desc_mn(sa) : make_smem_desc(sa);
          const uint64_t db = KIND == KIND_WG ? make_smem_desc_mn(sa + kABytes) : make_smem_desc(sa + kABytes);
          constexpr uint64_t kStep = KIND == KIND_WG ? 128 : 2;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            if (PAIR) umma_bf16_pair(d_tmem, da + kStep * k, db + kStep * k, idesc, (uint32_t)((kb | k) != 0));
            else umma_bf16(d_tmem, da + kStep * k, db + kStep * k, idesc, (uint32_t)((kb | k) != 0));
          }
          if (PAIR) umma_commit_pair(smem_u32(&tail->empty[stage]));
          else umma_commit(smem_u32(&tail->empty[stage]));
          if (++stage == NS) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (c.kblocks > 0) {
          if (PAIR) umma_commit_pair(smem_u32(&tail->tmem_full[as]));
          else umma_commit(smem_u32(&tail->tmem_full[as]));
        } else {                                                 // an expert without rows: nothing was issued
          mbar_arrive(smem_u32(&tail->tmem_full[as]));
          if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tail->tmem_full[as]), 1));
        }
        if (++as == kAccStages) { as = 0; aphase ^= 1u; }
      }
    }
  } else {
    // ---- epilogue -----------------------------------------------------------------------------
    const int q = warp & 3;
    const uint32_t stg = smem_u32(epi_smem + (size_t)(warp - 2) * kEpiStageBytes * (KIND == KIND_WG ? kWgBufs : 1));
    int wg_buf = 0;
    int as = 0;
    uint32_t aphase = 0;
    bool ok = true;
    for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
      const Coord c = tile_coord<KIND, TR>(tail, p, tile);
      ok = mbar_wait(smem_u32(&tail->tmem_full[as]), aphase, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * kAccCols);
      const int out_cols = 2 * p.bn;
      if (KIND == KIND_WG) {
        // fp32 tile of dW[e]: this warp's 32 rows, 32 columns at a time: TMEM -> registers ->
        // swizzled staging buffer -> one TMA store (or reduce-add into dW) of the 32 x 32 box.
        // An expert without rows adds nothing; without accumulation it gets zeros.
        const int m0 = c.mt * TR + (int)cta_rank * BM + q * 32;
        const bool emit = m0 < p.m_total && !(c.kblocks == 0 && p.accumulate);
        // one 32-column chunk: registers -> staging buffer -> TMA store / reduce-add
        auto put = [&](const uint32_t (&a)[32], int col) {
          const int n0 = c.nt * out_cols + col;
          if (n0 >= p.n_total) return;                        // warp-uniform; M and N are multiples of 32
          const uint32_t buf = stg + (uint32_t)(wg_buf * kEpiStageBytes);
          if (lane == 0) bulk_wait_read<kWgBufs - 1>();     // the store that read this buffer kWgBufs boxes ago
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t addr = buf + (uint32_t)(lane * 128 + ((j ^ (lane & 7)) << 4));
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a[4 * j]), "r"(a[4 * j + 1]),
                         "r"(a[4 * j + 2]), "r"(a[4 * j + 3]) : "memory");
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (p.accumulate) tma_reduce_add_3d(&tm_out, buf, n0, m0, c.expert);
            else tma_store_3d(&tm_out, buf, n0, m0, c.expert);
            bulk_commit();
          }
          if (++wg_buf == kWgBufs) wg_buf = 0;
        };
        if (emit) {
          uint32_t a0[32], a1[32];
          if (c.kblocks > 0) {
            // the TMEM load of the next chunk is in flight while the current one is staged and sent
            tmem_ld32(taddr, a0);
            for (int col = 0; col < out_cols; col += 64) {
              tmem_ld_wait();
              tmem_ld32(taddr + (uint32_t)(col + 32), a1);
              put(a0, col);
              tmem_ld_wait();
              if (col + 64 < out_cols) tmem_ld32(taddr + (uint32_t)(col + 64), a0);
              put(a1, col + 32);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) a0[i] = 0u;
            for (int col = 0; col < out_cols; col += 32) put(a0, col);
          }
        }
      } else {
        const int row_off = (int)cta_rank * BM + q * 32;
        const int rows_here = c.rows_valid - row_off;
        const int my_row = c.row0 + row_off + lane;
        const bool row_ok = lane < rows_here;
        for (int col = 0; col < out_cols; col += 64) {
          uint32_t a0[32], a1[32];
          tmem_ld32(taddr + (uint32_t)col, a0);
          tmem_ld32(taddr + (uint32_t)(col + 32), a1);
          tmem_ld_wait();
          const int gcol = c.nt * out_cols + col;      // first of this slice's 64 output columns
          if (gcol >= p.n_limit) continue;             // overhang of the last N tile (warp-uniform)
          if (KIND == KIND_DX) {
            uint32_t packed[32];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              packed[i] = pack_bf16x2(__uint_as_float(a0[2 * i]), __uint_as_float(a0[2 * i + 1]));
              packed[16 + i] = pack_bf16x2(__uint_as_float(a1[2 * i]), __uint_as_float(a1[2 * i + 1]));
            }
            staged_store(stg, packed, p.out + (int64_t)(c.row0 + row_off) * p.ld_out, p.ld_out, gcol, rows_here, lane);
          } else {
            // SwiGLU derivative: this thread's row, 64 columns of a and b (128 bytes each)
            uint32_t pa[32], pb[32];
            if (row_ok) {
              const uint4* ap = reinterpret_cast<const uint4*>(p.ab + (int64_t)my_row * (2 * p.f) + gcol);
              const uint4* bp = reinterpret_cast<const uint4*>(p.ab + (int64_t)my_row * (2 * p.f) + p.f + gcol);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const uint4 va = ap[i], vb = bp[i];
                pa[4 * i] = va.x; pa[4 * i + 1] = va.y; pa[4 * i + 2] = va.z; pa[4 * i + 3] = va.w;
                pb[4 * i] = vb.x; pb[4 * i + 1] = vb.y; pb[4 * i + 2] = vb.z; pb[4 * i + 3] = vb.w;
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) { pa[i] = 0u; pb[i] = 0u; }
            }
            uint32_t pda[32], pdb[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float dh0 = __uint_as_float(i < 16 ? a0[2 * i] : a1[2 * (i - 16)]);
              const float dh1 = __uint_as_float(i < 16 ? a0[2 * i + 1] : a1[2 * (i - 16) + 1]);
              const float x0 = bf16_lo(pa[i]), x1 = bf16_hi(pa[i]);
              const float y0 = bf16_lo(pb[i]), y1 = bf16_hi(pb[i]);
              const float s0 = sigmoid_f(x0), s1 = sigmoid_f(x1);
              // silu(a) = a*s;  silu'(a) = s * (1 + a * (1 - s))
              pda[i] = pack_bf16x2(dh0 * y0 * s0 * (1.f + x0 * (1.f - s0)), dh1 * y1 * s1 * (1.f + x1 * (1.f - s1)));
              pdb[i] = pack_bf16x2(dh0 * x0 * s0, dh1 * x1 * s1);
            }
            __nv_bfloat16* obase = p.out + (int64_t)(c.row0 + row_off) * p.ld_out;
            staged_store(stg, pda, obase, p.ld_out, gcol, rows_here, lane);
            staged_store(stg, pdb, obase, p.ld_out, p.f + gcol, rows_here, lane);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&tail->tmem_empty[as]), 0));
        else mbar_arrive(smem_u32(&tail->tmem_empty[as]));
      }
      if (++as == kAccStages) { as = 0; aphase ^= 1u; }
    }
    if (KIND == KIND_WG && lane == 0) bulk_wait_read<0>();      // staging must outlive the stores that read it
  }

  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();   // the leader's MMAs read the peer's shared memory: leave together
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- bandwidth kernels of the backward pass ---------------------------------------------------

// dst[c, r] = src[r, c] for a batch of bf16 matrices (32 x 32 tiles through shared memory); used
// once per weight update for the transposed weight copies, not per micro-batch.
__global__ void __launch_bounds__(256)
k_transpose_bf16(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows, int cols,
                 int64_t ld_src, int64_t ld_dst, int64_t batch_src, int64_t batch_dst) {
  __shared__ __nv_bfloat16 t[32][34];
  src += (int64_t)blockIdx.z * batch_src;
  dst += (int64_t)blockIdx.z * batch_dst;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;    // 32 x 8
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty + 8 * i, c = c0 + tx;
    const bool live = r < rows && c < cols;
    t[ty + 8 * i][tx] = live ? src[(int64_t)r * ld_src + c] : __float2bfloat16(0.f);
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = c0 + ty + 8 * i, r = r0 + tx;
    if (c < cols && r < rows) dst[(int64_t)c * ld_dst + r] = t[tx][ty + 8 * i];
  }
}

__device__ __forceinline__ uint4 ld_nc_v4(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Backward of the combine: for every slot (t, k) with row r = slot_to_row[t, k]
//   dY_perm[r, :] = gates[t, k] * dOut[t, :]         dGates[t, k] = <dOut[t, :], y_perm[r, :]>
// One warp per slot, slots dealt out in equal contiguous ranges.
__global__ void __launch_bounds__(256)
k_combine_bwd(const uint4* __restrict__ d_out, const uint4* __restrict__ y_perm, const int32_t* __restrict__ slot_to_row,
              const float* __restrict__ gates, uint4* __restrict__ d_y_perm, float* __restrict__ d_gates,
              int64_t S, int K, int chunks) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * 256) >> 5;
  const int64_t s0 = S * warp / nwarps, s1 = S * (warp + 1) / nwarps;
  for (int64_t s = s0; s < s1; ++s) {
    const int row = slot_to_row[s];
    const float g = gates[s];
    const int64_t t = s / K;
    float dot = 0.f;
    if (row >= 0) {
      for (int c = lane; c < chunks; c += 32) {
        const uint4 o = ld_nc_v4(d_out + t * chunks + c);
        const uint4 y = ld_nc_v4(y_perm + (int64_t)row * chunks + c);
        uint4 w;
        const uint32_t ov[4] = {o.x, o.y, o.z, o.w}, yv[4] = {y.x, y.y, y.z, y.w};
        uint32_t wv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float o0 = bf16_lo(ov[i]), o1 = bf16_hi(ov[i]);
          dot = fmaf(o0, bf16_lo(yv[i]), dot);
          dot = fmaf(o1, bf16_hi(yv[i]), dot);
          wv[i] = pack_bf16x2(g * o0, g * o1);
        }
        w.x = wv[0]; w.y = wv[1]; w.z = wv[2]; w.w = wv[3];
        d_y_perm[(int64_t)row * chunks + c] = w;
      }
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (lane == 0) d_gates[s] = row >= 0 ? dot : 0.f;
  }
}

// Zero the rows that pad each expert's segment to a multiple of 128 rows in up to three row-major
// buffers (blockIdx.y picks one): the weight gradients contract over whole 64-row blocks of a segment,
// and the GEMM epilogues that produce these buffers write the valid rows only.  gridDim.z blocks
// share one (expert, buffer).
struct PadBufs { uint4* buf[3]; int chunks[3]; };
__global__ void __launch_bounds__(256)
k_zero_pad_rows(const feplb_group* __restrict__ table, PadBufs b) {
  const feplb_group g = table[blockIdx.x];
  const int chunks = b.chunks[blockIdx.y];
  const int64_t r0 = (int64_t)g.row_start + g.rows, r1 = (r0 + 127) / 128 * 128;
  uint4* p = b.buf[blockIdx.y] + r0 * chunks;
  const int64_t n = (r1 - r0) * chunks;
  for (int64_t i = blockIdx.z * 256 + threadIdx.x; i < n; i += 256 * gridDim.z) p[i] = make_uint4(0, 0, 0, 0);
}

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

// Row-major bf16 matrix [rows, inner] with a row pitch of ld elements -> [box_rows, 64] boxes, 128-byte swizzle.
bool make_tmap(CUtensorMap* m, const void* base, uint64_t rows, uint64_t inner, uint64_t ld, uint32_t box_rows) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major bf16 [rows, cols] (pitch ld) as the 3-d tensor {64 columns, rows, cols/64 chunks}: a box of
// 64 x 64 x `chunks` lands in shared memory chunk after chunk, each 64 rows of 128 bytes, 128-byte
// swizzled: the MN-major operand layout of the weight-gradient kind.
bool make_tmap_mn(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t chunks) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {64, rows, cols / 64};
  cuuint64_t strides[2] = {ld * 2, 128};
  cuuint32_t box[3] = {64, (cuuint32_t)BK, chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 [E, M, N] as a 3-d map with boxes of 32 x 32 x 1, 128-byte swizzled (the epilogue's staging layout);
// a box never crosses into the next expert's matrix.
bool make_tmap_out(CUtensorMap* m, float* base, uint64_t E, uint64_t M, uint64_t N) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {N, M, E};
  cuuint64_t strides[2] = {N * 4, M * N * 4};
  cuuint32_t box[3] = {32, 32, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int KIND, bool PAIR>
cudaError_t launch_kind(const CUtensorMap& ta, const CUtensorMap& tb0, const CUtensorMap& tb1, const CUtensorMap& tout,
                        const BwdParams& p, int num_sms, cudaStream_t st) {
  // per instantiation and device: the shared-memory attribute and the resident grid are set on first use
  static int grid_of[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int& grid = grid_of[dev];
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  cfg.attrs = at;
  cfg.numAttrs = 0;
  if (PAIR) {
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.numAttrs = 1;
  }
  if (!grid) {
    cudaError_t e = cudaFuncSetAttribute(k_ffn_bwd_gemm<KIND, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    int g = num_sms;
    if (PAIR) {
      // as many clusters of two as can be resident at once (one CTA per SM, both SMs in one GPC)
      int n_clusters = 0;
      cfg.gridDim = dim3(num_sms / 2 * 2);
      e = cudaOccupancyMaxActiveClusters(&n_clusters, k_ffn_bwd_gemm<KIND, PAIR>, &cfg);
      if (e != cudaSuccess) return e;
      if (n_clusters < 1) return cudaErrorLaunchOutOfResources;
      g = 2 * (n_clusters < num_sms / 2 ? n_clusters : num_sms / 2);
    }
    grid = g;
  }
  cfg.gridDim = dim3(grid);
  return cudaLaunchKernelEx(&cfg, k_ffn_bwd_gemm<KIND, PAIR>, ta, tb0, tb1, tout, p);
}

cudaError_t transpose(const void* src, void* dst, int rows, int cols, int64_t ld_src, int64_t ld_dst, int batch,
                      int64_t batch_src, int64_t batch_dst, cudaStream_t st, int64_t* n_launch) {
  if (rows == 0 || cols == 0 || batch == 0) return cudaSuccess;
  dim3 grid((cols + 31) / 32, (rows + 31) / 32, batch);
  k_transpose_bf16<<<grid, 256, 0, st>>>((const __nv_bfloat16*)src, (__nv_bfloat16*)dst, rows, cols, ld_src, ld_dst,
                                         batch_src, batch_dst);
  ++*n_launch;
  return cudaGetLastError();
}

}  // namespace

cudaError_t feplb_launch_transpose_weights(const void* w1, const void* w3, const void* w2, void* w1t, void* w3t, void* w2t,
                                           int E, int d, int f, cudaStream_t st, int64_t* n_launch) {
  const int64_t per = (int64_t)d * f;
  cudaError_t e = transpose(w1, w1t, f, d, d, f, E, per, per, st, n_launch);       // [E,f,d] -> [E,d,f]
  if (e == cudaSuccess) e = transpose(w3, w3t, f, d, d, f, E, per, per, st, n_launch);
  if (e == cudaSuccess) e = transpose(w2, w2t, d, f, f, d, E, per, per, st, n_launch);   // [E,d,f] -> [E,f,d]
  return e;
}

cudaError_t feplb_launch_combine_bwd(const void* d_out, const void* y_perm, const int32_t* slot_to_row, const float* gates,
                                     void* d_y_perm, float* d_gates, int T, int K, int d, int num_sms, cudaStream_t st,
                                     int64_t* n_launch) {
  const int64_t S = (int64_t)T * K;
  if (S == 0) return cudaSuccess;
  int blocks = num_sms * 6;
  const int64_t need = (S + 7) / 8;
  if (need < blocks) blocks = (int)need;
  k_combine_bwd<<<blocks, 256, 0, st>>>((const uint4*)d_out, (const uint4*)y_perm, slot_to_row, gates, (uint4*)d_y_perm,
                                        d_gates, S, K, d / 8);
  ++*n_launch;
  return cudaGetLastError();
}

int feplb_launch_expert_ffn_bwd(const feplb_bwd_args& a, cudaStream_t st, int64_t* n_launch, char* err, size_t errn) {
  if (a.n_groups == 0 || a.s_cap == 0) return FEPLB_OK;
  const int d = a.d, f = a.f;
  cudaError_t e = cudaSuccess;
  auto fail_cuda = [&](const char* what) {
    snprintf(err, errn, "%s: %s", what, cudaGetErrorString(e));
    return FEPLB_E_CUDA;
  };
  // ---- dH and the SwiGLU derivative: dAB = SwiGLU'(a, b; dY W2) ----------------------------------
  const int bn_h = (f % 256 == 0) ? 128 : 64;      // N = f in tiles of 2*bn columns (the last may overhang)
  const int bn_x = (d % 256 == 0) ? 128 : 64;
  CUtensorMap tm_dy, tm_w2t, tm_dab, tm_w1t, tm_w3t;
  if (!make_tmap(&tm_dy, a.d_y_perm, (uint64_t)a.s_cap, (uint64_t)d, (uint64_t)d, BM) ||
      !make_tmap(&tm_w2t, a.w2t, (uint64_t)a.E * f, (uint64_t)d, (uint64_t)d, bn_h) ||
      !make_tmap(&tm_dab, a.d_ab, (uint64_t)a.s_cap, (uint64_t)2 * f, (uint64_t)2 * f, BM) ||
      !make_tmap(&tm_w1t, a.w1t, (uint64_t)a.E * d, (uint64_t)f, (uint64_t)f, bn_x) ||
      !make_tmap(&tm_w3t, a.w3t, (uint64_t)a.E * d, (uint64_t)f, (uint64_t)f, bn_x)) {
    snprintf(err, errn, "cuTensorMapEncodeTiled failed (backward)");
    return FEPLB_E_CUDA;
  }
  BwdParams p = {};
  p.groups = a.groups; p.n_groups = a.n_groups; p.which = a.which; p.E = a.E; p.s_cap = a.s_cap; p.status = a.status;
  BwdParams ph = p;
  ph.n_tiles_n = (f + 2 * bn_h - 1) / (2 * bn_h); ph.n_limit = f; ph.num_k_blocks = d / BK; ph.b_rows_per_expert = f; ph.bn = bn_h;
  ph.out = (__nv_bfloat16*)a.d_ab; ph.ld_out = 2 * f; ph.ab = (const __nv_bfloat16*)a.ab_saved; ph.f = f;
  e = a.pair_dgrad ? launch_kind<KIND_DH, true>(tm_dy, tm_w2t, tm_w2t, tm_dy, ph, a.num_sms, st)
                   : launch_kind<KIND_DH, false>(tm_dy, tm_w2t, tm_w2t, tm_dy, ph, a.num_sms, st);
  ++*n_launch;
  if (e != cudaSuccess) return fail_cuda("k_ffn_bwd_gemm<DH>");
  // ---- dX = [dA | dB] [W1^T ; W3^T] ------------------------------------------------------------------
  BwdParams px = p;
  px.n_tiles_n = d / (2 * bn_x); px.n_limit = d; px.num_k_blocks = 2 * f / BK; px.k_switch = f / BK; px.b_rows_per_expert = d; px.bn = bn_x;
  px.out = (__nv_bfloat16*)a.d_x_perm; px.ld_out = d;
  e = a.pair_dgrad ? launch_kind<KIND_DX, true>(tm_dab, tm_w1t, tm_w3t, tm_dab, px, a.num_sms, st)
                   : launch_kind<KIND_DX, false>(tm_dab, tm_w1t, tm_w3t, tm_dab, px, a.num_sms, st);
  ++*n_launch;
  if (e != cudaSuccess) return fail_cuda("k_ffn_bwd_gemm<DX>");
  if (!a.dw1) return FEPLB_OK;
  // ---- weight gradients: contraction over each expert's rows, operands read as they lie (MN-major) ------
  // dW2[e] [d, f] = dY_e^T H_e;   dW1[e] [f, d] = dA_e^T X_e;   dW3[e] [f, d] = dB_e^T X_e
  PadBufs pb;
  pb.buf[0] = (uint4*)a.h; pb.chunks[0] = f / 8;
  pb.buf[1] = (uint4*)a.d_y_perm; pb.chunks[1] = d / 8;
  pb.buf[2] = (uint4*)a.d_ab; pb.chunks[2] = 2 * f / 8;
  k_zero_pad_rows<<<dim3(a.E, 3, 8), 256, 0, st>>>(a.expert_table, pb);
  ++*n_launch;
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda("k_zero_pad_rows");
  struct WG { const void* p; int m_total; int ld_p; const void* q; int n_total; float* out; };
  const WG jobs[3] = {
      {a.d_y_perm, d, d, a.h, f, a.dw2},
      {a.d_ab, f, 2 * f, a.x_perm, d, a.dw1},
      {(const char*)a.d_ab + (size_t)f * 2, f, 2 * f, a.x_perm, d, a.dw3},
  };
  for (const WG& j : jobs) {
    const int bn = (j.n_total % 256 == 0) ? 128 : 64;
    CUtensorMap tm_at, tm_bt, tm_o;
    if (!make_tmap_mn(&tm_at, j.p, (uint64_t)a.s_cap, (uint64_t)j.m_total, (uint64_t)j.ld_p, BM / 64) ||
        !make_tmap_mn(&tm_bt, j.q, (uint64_t)a.s_cap, (uint64_t)j.n_total, (uint64_t)j.n_total, (a.pair_wgrad ? bn : 2 * bn) / 64) ||
        !make_tmap_out(&tm_o, j.out, (uint64_t)a.E, (uint64_t)j.m_total, (uint64_t)j.n_total)) {
      snprintf(err, errn, "cuTensorMapEncodeTiled failed (weight gradient)");
      return FEPLB_E_CUDA;
    }
    BwdParams pw = p;
    pw.groups = a.expert_table; pw.n_groups = a.E; pw.which = FEPLB_FFN_ALL;
    pw.bn = bn; pw.n_tiles_n = (j.n_total + 2 * bn - 1) / (2 * bn); pw.m_tiles = a.pair_wgrad ? (j.m_total + 2 * BM - 1) / (2 * BM) : (j.m_total + BM - 1) / BM;
    pw.m_total = j.m_total; pw.n_total = j.n_total; pw.wout = j.out; pw.accumulate = a.accumulate;
    e = a.pair_wgrad ? launch_kind<KIND_WG, true>(tm_at, tm_bt, tm_bt, tm_o, pw, a.num_sms, st)
                     : launch_kind<KIND_WG, false>(tm_at, tm_bt, tm_bt, tm_o, pw, a.num_sms, st);
    ++*n_launch;
    if (e != cudaSuccess) return fail_cuda("k_ffn_bwd_gemm<WG>");
  }
  return FEPLB_OK;
}
