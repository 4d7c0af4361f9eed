// Internal declarations shared by the translation units of libfeplb (not part of the ABI).
#ifndef FEPLB_INTERNAL_H_
#define FEPLB_INTERNAL_H_

#include <cstddef>
#include <cstdint>

#include "feplb.h"

#define FEPLB_MAX_EXPERTS 1024
#define FEPLB_MAX_GROUPS 1024
#define FEPLB_SLOTS_PER_BLOCK 1024   // slots ranked by one CTA of the permutation kernels
#define FEPLB_TILE_M 128             // rows of one GEMM tile
#ifndef FEPLB_NOALLOC_MAX_HIST_INTS
#error "feplb.h must define FEPLB_NOALLOC_MAX_HIST_INTS"
#endif

// bits of the device status word
#define FEPLB_ST_RANGE 1u      // expert id outside [0, E)
#define FEPLB_ST_COUNTS 2u     // counts passed to dispatch disagree with the ids
#define FEPLB_ST_WAIT 4u       // a bounded mbarrier wait gave up inside the GEMM
#define FEPLB_ST_GROUP 8u      // a group entry was malformed (expert or rows out of range)
#define FEPLB_ST_PLAN 16u      // the GEMM's bounded wait for the planner's dynamic group table gave up
#define FEPLB_WM_AUTO_ROWS_PER_EXPERT 768   // the weights-on-M form is the default below this many rows per expert
#define FEPLB_WM_MAX_ENTRIES 1024    // group entries (static + dynamic table) one weights-on-M launch can hold

int feplb_validate_config(const feplb_config* c);

#ifdef __CUDACC__
#include <cuda_runtime.h>

// Kernel launchers (each enqueues on `st` and returns the cudaError_t of the launch).
// n_launch is incremented by the number of kernels enqueued.
cudaError_t feplb_launch_block_hist(const int32_t* ids, int64_t S, int E, int R, int32_t* block_hist,
                                    int32_t* counts, int32_t* rank_load, uint32_t* status,
                                    cudaStream_t st, int64_t* n_launch);
cudaError_t feplb_launch_permute(const int32_t* ids, int64_t S, int K, int E, int A, const int32_t* counts,
                                 int32_t* block_hist, int32_t* pad_off, int32_t* slot_to_row,
                                 int32_t* row_to_token, int64_t s_cap, uint32_t* status,
                                 cudaStream_t st, int64_t* n_launch);
// Must follow feplb_launch_permute or feplb_launch_route_fused on the same stream: turns the ranks those
// left in slot_to_row into rows (block_base = the scanned per-CTA histograms), fills row_to_token and
// copies the rows of x.
cudaError_t feplb_launch_gather(const void* x, const int32_t* ids, const int32_t* block_base, int32_t* slot_to_row,
                                const int32_t* counts, const int32_t* pad_off, void* x_perm, int T, int K, int E, int d,
                                int A, int64_t s_cap, int num_sms, cudaStream_t st, int64_t* n_launch,
                                int32_t* row_to_token, bool programmatic);
// Whole-layer path: histogram (+ ranks inside each CTA's slots) + one scan kernel that emits counts, rank
// loads, offsets, the home group table and the -1 tail of row_to_token.
cudaError_t feplb_launch_route_fused(const int32_t* ids, int64_t S, int E, int R, int A, int dyn,
                                     const uint8_t* mask_in, int32_t* block_hist, int32_t* counts,
                                     int32_t* rank_load, int32_t* pad_off, feplb_group* groups, uint8_t* mask_out,
                                     int32_t* slot_to_row, int32_t* row_to_token, int64_t s_cap, uint32_t* status,
                                     unsigned long long* counts_host_tagged, int32_t seq, unsigned long long* t_counts,
                                     cudaStream_t st, int64_t* n_launch);
cudaError_t feplb_launch_upload_groups(const feplb_group* src_host_mapped, feplb_group* dst, int n, cudaStream_t st);
cudaError_t feplb_launch_home_groups(const int32_t* counts, const uint8_t* mask_in, int E, int R, int A, int dyn,
                                     feplb_group* groups, uint8_t* mask_out, cudaStream_t st, int64_t* n_launch);
cudaError_t feplb_launch_combine(const void* y_perm, const int32_t* slot_to_row, const float* gates, void* out,
                                 int T, int K, int d, int num_sms, cudaStream_t st, int64_t* n_launch);

cudaError_t feplb_launch_route_topk(const float* logits, int T, int E, int K, int32_t* ids, float* gates,
                                    int num_sms, cudaStream_t st, int64_t* n_launch);

struct feplb_gemm_args {
  const void* x_perm; const void* w1; const void* w3; const void* w2;
  void* h; void* y;
  const feplb_group* groups; int n_groups; int which;
  int E, d, f; int64_t s_cap;
  uint32_t* status;
  int num_sms;
  int pair;   // 1: clusters of two CTAs on 256-row tiles (cta_group::2); 0: one CTA per 128-row tile
  // receive buffer of migrated experts' weights ([n_recv_slots, f, d] x2 and [n_recv_slots, d, f]); may be null
  const void* recv_w1; const void* recv_w3; const void* recv_w2; int n_recv_slots;
  const void* recv_x = nullptr;   // optional [s_cap, d]: rows of pieces that run from a receive slot are read here (pass 1)
  void* ab_out;   // optional [s_cap, 2f]: pass 1 also saves the pre-activations a | b (for the backward pass)
};
// Returns FEPLB_OK or a feplb_status; text of a failure goes to err (size errn).
// One thread waits (bounded by limit_ns) on an mbarrier nobody completes; *gave_up = 1 and FEPLB_ST_WAIT expected.
cudaError_t feplb_launch_wait_selftest(uint32_t* status, unsigned long long limit_ns, int* gave_up, cudaStream_t st);
// A launch per pass walks a.groups (filtered by a.which) and then, if dyn.seq != 0, the planner's dynamic
// table, which it picks up on the device once the host-side ready word carries (seq << 32) | number of
// groups; the CTA that wins `claim` copies it to table_dev (feplb_dyn.cuh).
struct feplb_wm_dyn {
  // the table travels as 32-byte entries {expert, row_start, rows, exec_rank, is_dynamic, seq, 0, 0}
  void* table_dev = nullptr;                         // device copy of the table, written by the claiming CTA
  const void* table_host = nullptr;                  // device address of the planner's table in mapped host memory
  unsigned long long* ready_dev = nullptr;           // set by the claiming CTA after table_dev
  const unsigned long long* ready_host = nullptr;    // device address of the word the planner thread sets after table_host
  uint32_t* claim = nullptr;                         // device word the CTAs race for
  uint32_t seq = 0;                                  // 0: no dynamic table
  int max_groups = 0;                                // capacity of the tables
  unsigned long long* stamps = nullptr;              // optional, 8 words: globaltimer marks of the two launches
  unsigned long long wait_limit_ns = 0;              // bound of the wait for the table (0: the library's default)
};
// Tokens-on-M forms (feplb_gemm.cu): single CTA per 128-row tile or, with a.pair, clusters of two on 256-row tiles.
int feplb_launch_expert_ffn(const feplb_gemm_args& a, cudaStream_t st, int64_t* n_launch, char* err, size_t errn,
                            const feplb_wm_dyn* dyn = nullptr);
// Weights-on-M form (feplb_gemm_wm.cu).
bool feplb_wm_supported(int E, int d, int f, int n_entries_max);
int feplb_launch_expert_ffn_wm(const feplb_gemm_args& a, const feplb_wm_dyn& dyn, cudaStream_t st, int64_t* n_launch,
                               char* err, size_t errn);
// ---- backward pass ---------------------------------------------------------------------------
struct feplb_bwd_args {
  const void* x_perm; const void* ab_saved; void* h; void* d_y_perm;   // padding rows of h, d_y_perm, d_ab get zeros
  const void* w1t; const void* w3t; const void* w2t;        // [E,d,f], [E,d,f], [E,f,d]
  const feplb_group* groups; int n_groups; int which;
  const feplb_group* expert_table;                          // E entries {e, first row, rows}: the K ranges of the weight gradients
  void* d_ab; void* d_x_perm;                               // [s_cap, 2f], [s_cap, d]
  float* dw1; float* dw3; float* dw2; int accumulate;       // fp32 [E,f,d], [E,f,d], [E,d,f]; dw1 == nullptr: skip
  int E, d, f; int64_t s_cap;
  uint32_t* status; int num_sms;
  int pair_dgrad, pair_wgrad;                               // 1: cta_group::2 form (256 x 256 tiles per cluster of two CTAs)
};
cudaError_t feplb_launch_transpose_weights(const void* w1, const void* w3, const void* w2, void* w1t, void* w3t, void* w2t,
                                           int E, int d, int f, cudaStream_t st, int64_t* n_launch);
cudaError_t feplb_launch_combine_bwd(const void* d_out, const void* y_perm, const int32_t* slot_to_row, const float* gates,
                                     void* d_y_perm, float* d_gates, int T, int K, int d, int num_sms, cudaStream_t st,
                                     int64_t* n_launch);
int feplb_launch_expert_ffn_bwd(const feplb_bwd_args& a, cudaStream_t st, int64_t* n_launch, char* err, size_t errn);
#endif

#endif  // FEPLB_INTERNAL_H_
