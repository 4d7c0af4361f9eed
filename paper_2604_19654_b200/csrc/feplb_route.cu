// Integer side of the FEPLB hot path on sm_100a: routing histogram (paper Section 2.2: per-expert
// token counts known after Phase 1), the stable counting-sort permutation of (token, k) slots
// into expert-contiguous rows (Section 2.2, Phase 1: expert order for the grouped GEMM), the row
// gather, and the home (pre-plan) group table the static-expert GEMM runs on (Section 2.3).
//
// Ranks inside an expert's segment must not depend on the order in which atomics land, so
// ranking is done in three deterministic levels: a warp ranks its 32 slots with match_any and
// a lane mask, warps of a CTA are chained through per-warp histograms in shared memory, CTAs
// are chained through an exclusive scan of per-CTA histograms.  Atomics are used only for the
// per-expert totals (integer adds commute).  The first two levels run in the histogram kernel,
// which already holds the ids and match masks and leaves each slot's rank inside its CTA's 1024
// slots behind; the gather kernel adds the segment offset and the CTA's base from the scan, so no
// ranking kernel of its own sits between the counts and the row copies.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "feplb_internal.h"

namespace {

// Programmatic dependent launch: a kernel launched with the attribute below may be scheduled
// while the kernel before it in the stream drains; pdl_sync() holds it until that kernel's
// results are complete (a no-op for ordinary launches) and lets its own successor do the same.
__device__ __forceinline__ void pdl_sync() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, bool programmatic,
                   Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = programmatic ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kChunks = FEPLB_SLOTS_PER_BLOCK / kThreads;   // 32-slot chunks per warp (4)
static_assert(FEPLB_SLOTS_PER_BLOCK == kWarps * kChunks * 32, "slot tiling");

// Warp w of CTA b owns slots [b*1024 + w*128, +128) as kChunks chunks of 32 consecutive slots.
// Fills the per-warp histograms wh[kWarps][E] and returns each lane's ids and match masks.
__device__ __forceinline__ bool warp_histograms(const int32_t* __restrict__ ids, int64_t S, int E, int* wh,
                                                int (&id)[kChunks], unsigned (&mk)[kChunks]) {
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < kWarps * E; i += kThreads) wh[i] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * FEPLB_SLOTS_PER_BLOCK + w * (kChunks * 32);
  bool bad = false;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    const int64_t s = base + c * 32 + lane;
    int v = -1;
    if (s < S) {
      v = ids[s];
      if ((unsigned)v >= (unsigned)E) { bad = true; v = -1; }
    }
    id[c] = v;
    mk[c] = __match_any_sync(0xffffffffu, v);
    if (v >= 0 && lane == __ffs(mk[c]) - 1) wh[w * E + v] += __popc(mk[c]);
    __syncwarp();
  }
  return bad;
}

// A slot's rank among the slots of its expert inside its CTA's 1024 slots, as k_block_hist leaves it in
// slot_to_row for the gather kernel: -2 - rank (final rows are >= 0, -1 marks an id outside [0, E)).
__device__ __forceinline__ int encode_local_rank(int r) { return -2 - r; }

// Step 1: per-CTA histograms; with counts != nullptr also the totals (one atomic per CTA and expert);
// with local_rank != nullptr also every slot's encoded rank inside this CTA's slots.
__global__ void __launch_bounds__(kThreads)
k_block_hist(const int32_t* __restrict__ ids, int64_t S, int E, int L, int32_t* __restrict__ block_hist,
             int32_t* __restrict__ counts, int32_t* __restrict__ rank_load, uint32_t* status,
             int32_t* __restrict__ local_rank) {
  extern __shared__ int wh[];
  int id[kChunks];
  unsigned mk[kChunks];
  pdl_sync();
  if (warp_histograms(ids, S, E, wh, id, mk)) atomicOr(status, FEPLB_ST_RANGE);
  __syncthreads();
  // chain the warps: wh[w][e] becomes the rank of warp w's first slot of expert e; the sum is the CTA's count
  for (int e = threadIdx.x; e < E; e += kThreads) {
    int sum = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const int t = wh[w * E + e];
      wh[w * E + e] = sum;
      sum += t;
    }
    if (block_hist) block_hist[(int64_t)blockIdx.x * E + e] = sum;
    if (counts && sum) {
      atomicAdd(&counts[e], sum);
      atomicAdd(&rank_load[e / L], sum);
    }
  }
  if (!local_rank) return;
  __syncthreads();
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned lt = (1u << lane) - 1u;
  const int64_t base = (int64_t)blockIdx.x * FEPLB_SLOTS_PER_BLOCK + w * (kChunks * 32);
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    const int64_t s = base + c * 32 + lane;
    const int v = id[c];
    int r = 0;
    if (v >= 0) r = wh[w * E + v] + __popc(mk[c] & lt);
    __syncwarp();
    if (v >= 0 && lane == __ffs(mk[c]) - 1) wh[w * E + v] += __popc(mk[c]);
    __syncwarp();
    if (s < S) local_rank[s] = v >= 0 ? encode_local_rank(r) : -1;
  }
}

// Block-wide exclusive scan of v over the 1024 threads of the block; tmp holds 64 values.
template <typename V = int>
__device__ __forceinline__ V block_exclusive_scan(V v, V* tmp, V* total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  V x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    V y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) tmp[w] = x;
  __syncthreads();
  if (w == 0) {
    V s = tmp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      V y = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s += y;
    }
    tmp[32 + lane] = s;   // inclusive scan of the warp sums
  }
  __syncthreads();
  const V warp_off = w ? tmp[32 + w - 1] : 0;
  if (total) *total = tmp[32 + 31];
  return warp_off + x - v;
}

// Exclusive scan of the per-CTA histograms over CTAs (in place), check against counts, and
// pad_off[e] = sum_{e'<e} round_up(counts[e'], A); pad_off[E] = padded total.
// The counts are the caller's: when they disagree with the ids (FEPLB_ST_COUNTS) the result is
// wrong but every later access stays inside the caller's buffers -- a negative count is taken as
// zero, offsets are summed in 64 bits and clamped to s_cap, a padded total beyond s_cap is reported;
// the gather kernel then drops the rows that do not fit.
__global__ void __launch_bounds__(1024)
k_scan(int32_t* __restrict__ block_hist, int nb, int E, int A, const int32_t* __restrict__ counts,
       int32_t* __restrict__ pad_off, int64_t s_cap, uint32_t* status, int32_t* __restrict__ row_to_token) {
  __shared__ long long tmp[64];
  const int e = threadIdx.x;
  int c = 0;
  pdl_sync();
  if (e < E) {
    int run = 0;
    for (int b = 0; b < nb; ++b) {
      const int v = block_hist[(int64_t)b * E + e];
      block_hist[(int64_t)b * E + e] = run;
      run += v;
    }
    c = counts[e];
    if (run != c) atomicOr(status, FEPLB_ST_COUNTS);
    if (c < 0) c = 0;
  }
  long long total;
  const long long off = block_exclusive_scan<long long>(((long long)c + A - 1) / A * A, tmp, &total);
  if (e < E) pad_off[e] = (int32_t)(off < s_cap ? off : s_cap);
  if (e == 0) {
    pad_off[E] = (int32_t)(total < s_cap ? total : s_cap);
    if (total > s_cap) atomicOr(status, FEPLB_ST_COUNTS);
  }
  // rows behind the last segment hold no token (the padding rows inside segments are marked by k_zero_pad,
  // the live rows by k_gather: with counts that agree with the ids that covers every row)
  for (int64_t i = total + threadIdx.x; i < s_cap; i += blockDim.x) row_to_token[i] = -1;
}

// Whole-layer variant of k_scan: from the per-CTA histograms alone it produces everything the
// rest of the pass needs -- counts, per-rank loads, segment offsets, the home group table (with
// the dynamic-expert mask, given or derived from the counts) and the -1 tail of row_to_token --
// so that no memset, atomic or extra launch sits between the histogram and the plan.
__global__ void __launch_bounds__(1024)
k_scan_fused(int32_t* __restrict__ block_hist, int nb, int E, int L, int A, int dyn,
             const uint8_t* __restrict__ mask_in, int32_t* __restrict__ counts_out,
             int32_t* __restrict__ rank_load_out, int32_t* __restrict__ pad_off,
             feplb_group* __restrict__ groups, uint8_t* __restrict__ mask_out,
             int32_t* __restrict__ row_to_token, int64_t s_cap,
             unsigned long long* __restrict__ counts_host_tagged, int32_t seq, unsigned long long* t_counts) {
  __shared__ int tmp[64];
  __shared__ int sc[FEPLB_MAX_EXPERTS];
  const int e = threadIdx.x;
  int c = 0;
  pdl_sync();
  if (e < E) {
    // exclusive scan over CTAs, eight independent loads in flight per round (the in-place stores
    // would otherwise serialise every load behind the previous store)
    int run = 0;
    for (int b0 = 0; b0 < nb; b0 += 8) {
      int v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = b0 + j < nb ? block_hist[(int64_t)(b0 + j) * E + e] : 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (b0 + j < nb) block_hist[(int64_t)(b0 + j) * E + e] = run;
        run += v[j];
      }
    }
    c = run;
    counts_out[e] = c;
    sc[e] = c;
    // Straight into pinned host memory for the planner thread, each count in one 8-byte word that
    // carries this forward's sequence number: the reader polls until every word shows the
    // number, so no system-scope fence and no separate flag hold this kernel up (under bulk
    // host<->device copies such a fence was measured to cost tens of microseconds).
    if (counts_host_tagged)
      *reinterpret_cast<volatile unsigned long long*>(counts_host_tagged + e) =
          ((unsigned long long)(uint32_t)seq << 32) | (uint32_t)c;
  }
  if (t_counts && e == 0) {            // timeline: when the counts left for the host (globaltimer, ns)
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    *t_counts = t;
  }
  int total;
  const int off = block_exclusive_scan((c + A - 1) / A * A, tmp, &total);   // also orders sc[] for all threads
  if (e < E) {
    pad_off[e] = off;
    int is_dyn;
    if (mask_in) {
      is_dyn = mask_in[e] != 0;
    } else {
      const int b0 = e / L * L;
      int better = 0;
      for (int o = b0; o < b0 + L; ++o) better += (sc[o] > c) || (sc[o] == c && o < e);
      is_dyn = better < dyn;
    }
    groups[e] = feplb_group{e, off, c, e / L, is_dyn};
    if (mask_out) mask_out[e] = (uint8_t)is_dyn;
  }
  if (e == 0) pad_off[E] = total;
  if (e < E / L) {
    int sum = 0;
    for (int o = e * L; o < (e + 1) * L; ++o) sum += sc[o];
    rank_load_out[e] = sum;
  }
  for (int64_t i = (int64_t)total + threadIdx.x; i < s_cap; i += blockDim.x) row_to_token[i] = -1;
}

__device__ __forceinline__ uint4 ld_nc_v4(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Row gather, token-major: one warp reads a token's row once (16-byte vectors, coalesced) and
// writes it to the K rows of its slots.  A slot's row = segment offset of its expert + first row of
// its CTA-of-1024-slots within the segment (both from the scan) + its rank inside that CTA (left in
// slot_to_row by k_block_hist); the warp that copies the first slice of a token writes the final
// slot_to_row and row_to_token entries.  Another warp working on a later slice of the same token may
// read either form of the entry, and gets the same row from both.
constexpr int kGatherUnroll = 4;
// Work unit = (token, slice of 4 x 32 chunks = 2 KiB of its row); equal contiguous ranges of units
// per warp over a grid sized to the machine, so that no tail wave forms.
__global__ void __launch_bounds__(kThreads)
k_gather(const uint4* __restrict__ x, const int32_t* __restrict__ ids, const int32_t* __restrict__ pad_off,
         const int32_t* __restrict__ block_base, int32_t* slot_to_row, int32_t* __restrict__ row_to_token,
         uint4* __restrict__ x_perm, int T, int K, int E, int chunks, int64_t s_cap) {
  pdl_sync();
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  const int slices = (chunks + 32 * kGatherUnroll - 1) / (32 * kGatherUnroll);
  const int64_t units = (int64_t)T * slices;
  const int64_t u0 = units * warp / nwarps, u1 = units * (warp + 1) / nwarps;
  int cur_t = -1, myrow = -1;
  for (int64_t u = u0; u < u1; ++u) {
    const int t = (int)(u / slices);
    const int c0 = (int)(u - (int64_t)t * slices) * 32 * kGatherUnroll;
    const uint4* src = x + (int64_t)t * chunks;
    uint4 v[kGatherUnroll];
#pragma unroll
    for (int i = 0; i < kGatherUnroll; ++i) {
      const int c = c0 + i * 32 + lane;
      if (c < chunks) v[i] = ld_nc_v4(src + c);
    }
    if (t != cur_t) {            // warp-uniform
      cur_t = t;
      myrow = -1;
      if (lane < K) {
        const int64_t s = (int64_t)t * K + lane;
        const int r = __ldcg(slot_to_row + s);
        const int e = ids[s];    // in flight together with r; its offsets follow in one more round trip
        if (r >= 0) {
          myrow = r;             // already final
        } else if (r <= -2) {    // implies 0 <= e < E (checked by k_block_hist)
          const int64_t row = (int64_t)pad_off[e] + block_base[s / FEPLB_SLOTS_PER_BLOCK * E + e] + (-2 - r);
          // rows beyond the buffer: only with counts that disagree with the ids (reported by the scan)
          myrow = row < s_cap ? (int)row : -1;
        }
        if (c0 == 0) {           // the token's first slice: this warp publishes the rows
          slot_to_row[s] = myrow;
          if (myrow >= 0) row_to_token[myrow] = t;
        }
      }
    }
    for (int k = 0; k < K; ++k) {
      const int row = __shfl_sync(0xffffffffu, myrow, k);
      if (row < 0) continue;
      uint4* dst = x_perm + (int64_t)row * chunks;
#pragma unroll
      for (int i = 0; i < kGatherUnroll; ++i) {
        const int c = c0 + i * 32 + lane;
        if (c < chunks) dst[c] = v[i];
      }
    }
  }
}

// Zero the padding rows at the end of every expert's segment (row_align > 1 only).
__global__ void __launch_bounds__(kThreads)
k_zero_pad(const int32_t* __restrict__ counts, const int32_t* __restrict__ pad_off, uint4* __restrict__ x_perm,
           int chunks, int32_t* __restrict__ row_to_token, int64_t s_cap) {
  pdl_sync();
  const int e = blockIdx.x;
  // clamped to the buffer: counts that disagree with the ids must not turn into wild writes
  const int c = counts[e] > 0 ? counts[e] : 0;
  int64_t r1 = pad_off[e + 1];
  if (r1 > s_cap) r1 = s_cap;
  int64_t r0 = (int64_t)pad_off[e] + c;
  if (r0 > r1) r0 = r1;
  if (r0 < 0) r0 = 0;
  if (row_to_token)
    for (int64_t r = r0 + threadIdx.x; r < r1; r += kThreads) row_to_token[r] = -1;
  const int64_t n = (r1 - r0) * chunks;
  uint4* p = x_perm + r0 * chunks;
  const uint4 z = make_uint4(0, 0, 0, 0);
  for (int64_t i = threadIdx.x; i < n; i += kThreads) p[i] = z;
}

// Home group table {e, pad_off[e], counts[e], home(e), dynamic?} for all E experts.
__global__ void __launch_bounds__(1024)
k_home_groups(const int32_t* __restrict__ counts, const uint8_t* __restrict__ mask_in, int E, int L, int A, int dyn,
              feplb_group* __restrict__ groups, uint8_t* __restrict__ mask_out) {
  __shared__ int tmp[64];
  __shared__ int sc[FEPLB_MAX_EXPERTS];
  const int e = threadIdx.x;
  const int c = e < E ? counts[e] : 0;
  if (e < E) sc[e] = c;
  const int off = block_exclusive_scan<int>((c + A - 1) / A * A, tmp, nullptr);
  if (e >= E) return;
  int is_dyn;
  if (mask_in) {
    is_dyn = mask_in[e] != 0;
  } else {
    // dynamic iff fewer than `dyn` experts of the block are busier (ties: lower id is busier)
    const int b0 = e / L * L;
    int better = 0;
    for (int o = b0; o < b0 + L; ++o) better += (sc[o] > c) || (sc[o] == c && o < e);
    is_dyn = better < dyn;
  }
  groups[e] = feplb_group{e, off, c, e / L, is_dyn};
  if (mask_out) mask_out[e] = (uint8_t)is_dyn;
}

// Router top-k gating (paper Sections 2.3 and 3.1: top-k routing, no auxiliary loss): one warp per
// token.  Lane l holds logits l, l+32, ...; K rounds of a warp arg-max (larger value, then lower
// expert id) pick the experts in descending order; gates = softmax over the K selected logits.
template <int NPER>
__global__ void __launch_bounds__(kThreads)
k_route_topk(const float* __restrict__ logits, int T, int E, int K, int32_t* __restrict__ ids,
             float* __restrict__ gates) {
  const int lane = threadIdx.x & 31;
  const int warp = (blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int nwarps = (gridDim.x * kThreads) >> 5;
  for (int t = warp; t < T; t += nwarps) {
    float v[NPER];
#pragma unroll
    for (int i = 0; i < NPER; ++i) {
      const int e = i * 32 + lane;
      v[i] = e < E ? logits[(int64_t)t * E + e] : -INFINITY;
    }
    unsigned taken = 0;
    float sel_val = 0.f;
    int sel_idx = 0;
    for (int k = 0; k < K; ++k) {
      float best = -INFINITY;
      int bidx = 0x7fffffff;
#pragma unroll
      for (int i = 0; i < NPER; ++i) {
        const int e = i * 32 + lane;
        if (e < E && !((taken >> i) & 1u) && (v[i] > best || bidx == 0x7fffffff)) { best = v[i]; bidx = e; }
      }
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
        if (oi != 0x7fffffff && (bidx == 0x7fffffff || ov > best || (ov == best && oi < bidx))) { best = ov; bidx = oi; }
      }
      if ((bidx & 31) == lane) taken |= 1u << (bidx >> 5);
      if (lane == k) { sel_val = best; sel_idx = bidx; }
    }
    const float m = __shfl_sync(0xffffffffu, sel_val, 0);       // the first pick is the maximum
    float ex = lane < K ? expf(sel_val - m) : 0.f;
    float sum = ex;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane < K) {
      ids[(int64_t)t * K + lane] = sel_idx;
      gates[(int64_t)t * K + lane] = ex / sum;
    }
  }
}

}  // namespace

cudaError_t feplb_launch_block_hist(const int32_t* ids, int64_t S, int E, int R, int32_t* block_hist,
                                    int32_t* counts, int32_t* rank_load, uint32_t* status,
                                    cudaStream_t st, int64_t* n_launch) {
  cudaError_t err;
  if (counts) {
    if ((err = cudaMemsetAsync(counts, 0, sizeof(int32_t) * E, st)) != cudaSuccess) return err;
    if ((err = cudaMemsetAsync(rank_load, 0, sizeof(int32_t) * R, st)) != cudaSuccess) return err;
  }
  const int nb = (int)((S + FEPLB_SLOTS_PER_BLOCK - 1) / FEPLB_SLOTS_PER_BLOCK);
  if (nb == 0) return cudaSuccess;
  k_block_hist<<<nb, kThreads, sizeof(int) * kWarps * E, st>>>(ids, S, E, E / R, block_hist, counts, rank_load, status,
                                                                (int32_t*)nullptr);
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t feplb_launch_permute(const int32_t* ids, int64_t S, int K, int E, int A, const int32_t* counts,
                                 int32_t* block_hist, int32_t* pad_off, int32_t* slot_to_row,
                                 int32_t* row_to_token, int64_t s_cap, uint32_t* status,
                                 cudaStream_t st, int64_t* n_launch) {
  // two kernels chained by a programmatic launch (the second one's launch latency hides under the first);
  // feplb_launch_gather, which must follow, turns the ranks they leave in slot_to_row into rows
  (void)K;
  cudaError_t err;
  const int nb = (int)((S + FEPLB_SLOTS_PER_BLOCK - 1) / FEPLB_SLOTS_PER_BLOCK);
  if (nb) {
    err = launch(k_block_hist, nb, kThreads, sizeof(int) * kWarps * E, st, false, ids, S, E, E, block_hist,
                 (int32_t*)nullptr, (int32_t*)nullptr, status, slot_to_row);
    ++*n_launch;
    if (err != cudaSuccess) return err;
  }
  err = launch(k_scan, 1, 1024, 0, st, nb > 0, block_hist, nb, E, A, counts, pad_off, s_cap, status, row_to_token);
  ++*n_launch;
  return err;
}

cudaError_t feplb_launch_gather(const void* x, const int32_t* ids, const int32_t* block_base, int32_t* slot_to_row,
                                const int32_t* counts, const int32_t* pad_off, void* x_perm, int T, int K, int E, int d,
                                int A, int64_t s_cap, int num_sms, cudaStream_t st, int64_t* n_launch,
                                int32_t* row_to_token, bool programmatic) {
  cudaError_t err;
  const int chunks = d / 8;
  if (A > 1) {
    err = launch(k_zero_pad, E, kThreads, 0, st, programmatic, counts, pad_off, (uint4*)x_perm, chunks, row_to_token,
                 s_cap);
    ++*n_launch;
    if (err != cudaSuccess) return err;
  }
  if (T == 0) return cudaSuccess;
  const int64_t units = (int64_t)T * ((chunks + 32 * kGatherUnroll - 1) / (32 * kGatherUnroll));
  int blocks = num_sms * 8;   // 8 CTAs of 256 threads per SM are resident
  const int64_t need = (units + kWarps - 1) / kWarps;
  if (need < blocks) blocks = (int)need;
  ++*n_launch;
  return launch(k_gather, blocks, kThreads, 0, st, programmatic, (const uint4*)x, ids, pad_off, block_base, slot_to_row,
                row_to_token, (uint4*)x_perm, T, K, E, chunks, s_cap);
}

// Copies the planner's table of dynamic groups from mapped pinned host memory to the device.  A
// kernel rather than a host-to-device memcpy: a memcpy would queue on the copy engine behind
// whatever bulk input transfer is in flight, and the dynamic GEMM waits for this table.
__global__ void __launch_bounds__(256) k_upload_groups(const int4* __restrict__ src_host, int4* __restrict__ dst, int n16) {
  for (int i = threadIdx.x; i < n16; i += 256) dst[i] = src_host[i];
}

cudaError_t feplb_launch_upload_groups(const feplb_group* src_host_mapped, feplb_group* dst, int n, cudaStream_t st) {
  const int n16 = (int)(((size_t)n * sizeof(feplb_group) + 15) / 16);      // both tables are allocated in 16-byte multiples
  if (n16 == 0) return cudaSuccess;
  k_upload_groups<<<1, 256, 0, st>>>(reinterpret_cast<const int4*>(src_host_mapped), reinterpret_cast<int4*>(dst), n16);
  return cudaGetLastError();
}

cudaError_t feplb_launch_home_groups(const int32_t* counts, const uint8_t* mask_in, int E, int R, int A, int dyn,
                                     feplb_group* groups, uint8_t* mask_out, cudaStream_t st, int64_t* n_launch) {
  k_home_groups<<<1, 1024, 0, st>>>(counts, mask_in, E, E / R, A, dyn, groups, mask_out);
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t feplb_launch_route_fused(const int32_t* ids, int64_t S, int E, int R, int A, int dyn,
                                     const uint8_t* mask_in, int32_t* block_hist, int32_t* counts,
                                     int32_t* rank_load, int32_t* pad_off, feplb_group* groups, uint8_t* mask_out,
                                     int32_t* slot_to_row, int32_t* row_to_token, int64_t s_cap, uint32_t* status,
                                     unsigned long long* counts_host_tagged, int32_t seq, unsigned long long* t_counts,
                                     cudaStream_t st, int64_t* n_launch) {
  cudaError_t err;
  const int nb = (int)((S + FEPLB_SLOTS_PER_BLOCK - 1) / FEPLB_SLOTS_PER_BLOCK);
  if (nb) {
    err = launch(k_block_hist, nb, kThreads, sizeof(int) * kWarps * E, st, true, ids, S, E, E, block_hist,
                 (int32_t*)nullptr, (int32_t*)nullptr, status, slot_to_row);
    ++*n_launch;
    if (err != cudaSuccess) return err;
  }
  ++*n_launch;
  return launch(k_scan_fused, 1, 1024, 0, st, true, block_hist, nb, E, E / R, A, dyn, mask_in, counts, rank_load, pad_off,
                groups, mask_out, row_to_token, s_cap, counts_host_tagged, seq, t_counts);
}

cudaError_t feplb_launch_route_topk(const float* logits, int T, int E, int K, int32_t* ids, float* gates,
                                    int num_sms, cudaStream_t st, int64_t* n_launch) {
  if (T == 0) return cudaSuccess;
  int blocks = (T + kWarps - 1) / kWarps;
  if (blocks > num_sms * 8) blocks = num_sms * 8;
  const int nper = (E + 31) / 32;
  ++*n_launch;
  if (nper <= 1) k_route_topk<1><<<blocks, kThreads, 0, st>>>(logits, T, E, K, ids, gates);
  else if (nper <= 2) k_route_topk<2><<<blocks, kThreads, 0, st>>>(logits, T, E, K, ids, gates);
  else if (nper <= 4) k_route_topk<4><<<blocks, kThreads, 0, st>>>(logits, T, E, K, ids, gates);
  else if (nper <= 8) k_route_topk<8><<<blocks, kThreads, 0, st>>>(logits, T, E, K, ids, gates);
  else if (nper <= 16) k_route_topk<16><<<blocks, kThreads, 0, st>>>(logits, T, E, K, ids, gates);
  else k_route_topk<32><<<blocks, kThreads, 0, st>>>(logits, T, E, K, ids, gates);
  return cudaGetLastError();
}
