// feplb_dispatch_noalloc: the dispatch step for callers that must not allocate device memory.
//
// Some users of this library cannot call cudaMalloc at the point where they need a dispatch:
// a serving process that has already handed all free device memory to its own pool (so a late
// cudaMalloc fails or eats into memory the pool believes it owns), or a latency-critical loop
// that cannot afford the device-wide synchronisation an allocation or free implies.  They also
// cannot create a feplb context there, because feplb_create allocates its scratch.  For them the
// scratch of the permutation (per-CTA histograms and the segment offsets) lives in a fixed-size
// array that is part of the library image: every GPU that loads libfeplb holds these ~2 MiB
// until the process exits, and no call here allocates or frees anything.
//
// The array is shared by every call on a device and keeps the previous call's contents.  The
// kernels overwrite the parts they read (histograms, offsets) before reading them, so nothing
// needs clearing between calls -- but two calls whose GPU work overlaps (different streams, or
// different host threads) would race on it.  Serialise them.
#include <cuda_runtime.h>

#include <mutex>

#include "feplb.h"
#include "feplb_internal.h"

namespace {

// Layout: [0, kMaxHist) per-CTA histograms (ceil(S/1024) x E ints), then E+1 segment offsets,
// then one spare status word used when the caller passes none.
constexpr size_t kMaxHist = FEPLB_NOALLOC_MAX_HIST_INTS;
constexpr size_t kScratchInts = kMaxHist + FEPLB_MAX_EXPERTS + 1 + 31;

static __device__ __align__(256) int32_t g_dispatch_scratch[kScratchInts];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
int32_t* g_scratch_addr[kMaxDevices] = {nullptr};
int g_num_sms[kMaxDevices] = {0};

// Device address of the array on the current device.  In host code the symbol's name is only a
// handle, never an address a kernel could use, so it is resolved through the runtime once per
// device (with that device current) and cached.
int scratch_for_current_device(int32_t** out, int* num_sms) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FEPLB_E_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    int sms = 0;
    if (cudaGetSymbolAddress(&p, g_dispatch_scratch) != cudaSuccess || !p ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
      cudaGetLastError();
      return FEPLB_E_CUDA;
    }
    g_num_sms[dev] = sms;
    g_scratch_addr[dev] = static_cast<int32_t*>(p);
  }
  *out = g_scratch_addr[dev];
  *num_sms = g_num_sms[dev];
  return FEPLB_OK;
}

}  // namespace

extern "C" int feplb_dispatch_noalloc(const feplb_config* cfg, const void* x, const int32_t* topk_ids,
                                      const int32_t* counts, void* x_perm, int32_t* slot_to_row,
                                      int32_t* row_to_token, uint32_t* status, void* stream) {
  int rc = feplb_validate_config(cfg);
  if (rc != FEPLB_OK) return rc;
  const int64_t S = (int64_t)cfg->T * cfg->K;
  const int64_t nb = (S + FEPLB_SLOTS_PER_BLOCK - 1) / FEPLB_SLOTS_PER_BLOCK;
  if (nb * cfg->E > (int64_t)kMaxHist) return FEPLB_E_NOMEM;   // beyond the built-in scratch: use feplb_dispatch
  if (!counts || !row_to_token) return FEPLB_E_INVALID;
  if (cfg->T > 0) {
    if (!x || !topk_ids || !x_perm || !slot_to_row) return FEPLB_E_INVALID;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(x_perm)) & 15u) return FEPLB_E_INVALID;
  }
  int32_t* scratch = nullptr;
  int num_sms = 0;
  if ((rc = scratch_for_current_device(&scratch, &num_sms)) != FEPLB_OK) return rc;
  int32_t* block_hist = scratch;
  int32_t* pad_off = scratch + kMaxHist;
  uint32_t* st_word = status ? status : reinterpret_cast<uint32_t*>(scratch + kMaxHist + FEPLB_MAX_EXPERTS + 1);
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t s_cap = S + (int64_t)cfg->E * (cfg->row_align - 1);
  int64_t launches = 0;
  if (!status && cudaMemsetAsync(st_word, 0, sizeof(uint32_t), st) != cudaSuccess) return FEPLB_E_CUDA;
  if (feplb_launch_permute(topk_ids, S, cfg->K, cfg->E, cfg->row_align, counts, block_hist, pad_off, slot_to_row,
                           row_to_token, s_cap, st_word, st, &launches) != cudaSuccess)
    return FEPLB_E_CUDA;
  if (feplb_launch_gather(x, topk_ids, block_hist, slot_to_row, counts, pad_off, x_perm, cfg->T, cfg->K, cfg->E, cfg->d,
                          cfg->row_align, s_cap, num_sms, st, &launches, row_to_token, true) != cudaSuccess)
    return FEPLB_E_CUDA;
  return FEPLB_OK;
}
