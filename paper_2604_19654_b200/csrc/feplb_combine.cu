// Gated combine of the FEPLB hot path on sm_100a (paper Section 2.3: the Combine phase returns
// the expert results to their tokens): out[t,:] = sum_k gates[t,k] * y_perm[slot_to_row[t,k],:],
// k ascending, fp32 accumulation, one bf16 rounding.  HBM-bound: every y_perm row is read once
// with 16-byte loads (K independent loads in flight per lane), every out row written once.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "feplb_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 8;   // rows loaded before they are accumulated

__device__ __forceinline__ uint4 ld_nc_v4(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ void fma_bf16x2(float& a0, float& a1, float g, uint32_t packed) {
  // bf16 -> fp32 is a 16-bit shift
  a0 = fmaf(g, __uint_as_float(packed << 16), a0);
  a1 = fmaf(g, __uint_as_float(packed & 0xffff0000u), a1);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Work unit = (token, 32-chunk slice of its row) = 512 output bytes; the units are dealt out in
// equal contiguous ranges to all warps of a grid sized to the machine, so that no tail wave forms.
__global__ void __launch_bounds__(kThreads, 3)
k_combine(const uint4* __restrict__ y_perm, const int32_t* __restrict__ slot_to_row,
          const float* __restrict__ gates, uint4* __restrict__ out, int T, int K, int chunks) {
  // launched with programmatic stream serialization: CTAs may become resident while the expert
  // GEMM before them drains; its y_perm is complete only after this wait
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  const int slices = (chunks + 31) / 32;
  const int64_t units = (int64_t)T * slices;
  const int64_t u0 = units * warp / nwarps, u1 = units * (warp + 1) / nwarps;
  int cur_t = -1, myrow = -1;
  float myg = 0.f;
  for (int64_t u = u0; u < u1; ++u) {
    const int t = (int)(u / slices);
    const int c = (int)(u - (int64_t)t * slices) * 32 + lane;
    if (t != cur_t) {            // warp-uniform
      cur_t = t;
      myrow = -1;
      myg = 0.f;
      if (lane < K) {
        myrow = slot_to_row[(int64_t)t * K + lane];
        myg = gates ? gates[(int64_t)t * K + lane] : 1.f;   // no gates: plain sum (backward of the dispatch)
      }
    }
    const bool on = c < chunks;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    for (int k0 = 0; k0 < K; k0 += kBatch) {
      uint4 v[kBatch];
      float g[kBatch];
#pragma unroll
      for (int j = 0; j < kBatch; ++j) {
        const int k = k0 + j;
        const int row = __shfl_sync(0xffffffffu, myrow, k & 31);
        g[j] = __shfl_sync(0xffffffffu, myg, k & 31);
        v[j] = make_uint4(0, 0, 0, 0);
        if (k >= K || row < 0) g[j] = 0.f;
        else if (on) v[j] = ld_nc_v4(y_perm + (int64_t)row * chunks + c);
      }
#pragma unroll
      for (int j = 0; j < kBatch; ++j) {
        if (k0 + j < K) {
          fma_bf16x2(acc[0], acc[1], g[j], v[j].x);
          fma_bf16x2(acc[2], acc[3], g[j], v[j].y);
          fma_bf16x2(acc[4], acc[5], g[j], v[j].z);
          fma_bf16x2(acc[6], acc[7], g[j], v[j].w);
        }
      }
    }
    if (on) {
      uint4 o;
      o.x = pack_bf16x2(acc[0], acc[1]);
      o.y = pack_bf16x2(acc[2], acc[3]);
      o.z = pack_bf16x2(acc[4], acc[5]);
      o.w = pack_bf16x2(acc[6], acc[7]);
      out[(int64_t)t * chunks + c] = o;
    }
  }
}

}  // namespace

cudaError_t feplb_launch_combine(const void* y_perm, const int32_t* slot_to_row, const float* gates, void* out,
                                 int T, int K, int d, int num_sms, cudaStream_t st, int64_t* n_launch) {
  if (T == 0) return cudaSuccess;
  // a grid that fills every SM exactly once at 3 CTAs per SM (fewer CTAs if there is less work)
  const int64_t units = (int64_t)T * ((d / 8 + 31) / 32);
  int blocks = num_sms * 3;
  const int64_t need = (units + kThreads / 32 - 1) / (kThreads / 32);
  if (need < blocks) blocks = (int)need;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  ++*n_launch;
  return cudaLaunchKernelEx(&cfg, k_combine, (const uint4*)y_perm, slot_to_row, gates, (uint4*)out, T, K, d / 8);
}
