/*
 * feplb.h -- C ABI of libfeplb: the per-micro-batch MoE-layer hot path of FEPLB on one
 * NVIDIA B200 (sm_100a), with the expert-parallel layout modelled as R virtual ranks.
 *
 * Path (paper Section 2.3, per-micro-batch timeline):
 *   router output (given)  ->  feplb_route_hist   per-expert token counts        (Section 2.2)
 *                          ->  feplb_plan         greedy rebalancing plan (host) (Section 2.3)
 *                          ->  feplb_dispatch     permutation into expert-contiguous rows (2.2)
 *                          ->  feplb_expert_ffn   static, then dynamic grouped SwiGLU GEMMs (2.3)
 *                          ->  feplb_combine      gate-weighted return of the results    (2.3)
 *   feplb_moe_forward runs the whole path and overlaps the host planner with the static-expert
 *   GEMM, as the paper's timeline does.
 *
 * Notation: T tokens, K experts per token, E experts, R ranks, L = E/R experts per rank in
 * contiguous blocks (home(e) = e / L), S = T*K slots with slot s = t*K + k, d hidden size,
 * f expert width, A = row_align, S_cap = feplb_s_pad(cfg) rows of the permuted buffers.
 *
 * Conventions
 *   - Every function returns 0 (FEPLB_OK) or a negative feplb_status; nothing throws.
 *   - "dev" pointers are device global memory on the context's device, 16-byte aligned, owned
 *     by the caller; "host" pointers are ordinary host memory.  The library keeps no pointer
 *     after a call returns, except where stated (feplb_plan_async).
 *   - Device work is enqueued on the cudaStream_t passed as `stream` (as void*) and is
 *     asynchronous unless stated.  Calls on one context must not overlap on the GPU: they share
 *     the context's scratch.
 *   - bf16 tensors are row-major.  Expert weights are stored output-major:
 *     w1, w3 [E, f, d] and w2 [E, d, f] (row n of w1[e] = the d coefficients of hidden unit n).
 *   - Out-of-range expert ids and device-side waits that gave up are reported through the
 *     context's status word: see feplb_check_status.  Kernels never trap.
 *   - There is no CPU fallback: device entry points need a CUDA device of compute capability
 *     10.0 and fail with FEPLB_E_CUDA otherwise.
 */
#ifndef FEPLB_H_
#define FEPLB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FEPLB_OK = 0,
  FEPLB_E_INVALID = -1, /* bad argument or unsupported shape */
  FEPLB_E_RANGE = -2,   /* an expert id outside [0, E) was seen on the device */
  FEPLB_E_CUDA = -3,    /* a CUDA runtime/driver call failed; text in feplb_last_error */
  FEPLB_E_NOMEM = -4,   /* an allocation failed, or a caller-sized array is too small */
  FEPLB_E_TIMEOUT = -5, /* a bounded host wait expired, or the GEMM's bounded wait for the plan did */
  FEPLB_E_STATE = -6,   /* call order violated (e.g. plan_wait without plan_async) */
  FEPLB_E_DEVICE = -7   /* a bounded device-side wait gave up, or counts disagree with ids */
} feplb_status;

enum { FEPLB_POLICY_LITERAL = 0, FEPLB_POLICY_FIRST_FIT = 1 };
enum { FEPLB_MASK_GIVEN = 0, FEPLB_MASK_REACTIVE = 1 };
enum { FEPLB_FFN_ALL = 0, FEPLB_FFN_STATIC = 1, FEPLB_FFN_DYNAMIC = 2 };
enum { FEPLB_FORM_AUTO = -1, FEPLB_FORM_SINGLE = 0, FEPLB_FORM_PAIR = 1, FEPLB_FORM_WEIGHT_M = 2 };

/* Layer geometry and balancer parameters.
 * Requirements: E % R == 0; d % 128 == 0; f % 64 == 0; 1 <= K <= 32; E <= 1024;
 * row_align in {1, 128}; split_granule >= 1. */
typedef struct {
  int32_t T, K, E, R, d, f;
  int32_t dyn;              /* dynamic experts per rank (Section 2.3), used by FEPLB_MASK_REACTIVE */
  int32_t max_num_dyn;      /* received experts (pieces) per rank: the receive buffer holds
                               max_num_dyn expert weights (Section 2.3, memory paragraph) */
  int32_t tau;              /* minimum rows for a migration (Section 2.3, threshold tau) */
  int32_t ranks_per_domain; /* ranks per NVLink domain, 0 = R (Section 2.2: rebalance only inside) */
  int32_t policy;           /* FEPLB_POLICY_*: stop at, or skip, a busiest expert that does not fit */
  int32_t split;            /* 0 = whole experts (the paper); 1 = cut hot experts (extension) */
  int32_t split_granule;    /* rows; pieces of a cut expert are multiples of it */
  int32_t row_align;        /* A: expert segments of the permuted buffers start at multiples of A */
  int32_t mask_policy;      /* FEPLB_MASK_*: who chooses the dynamic experts in feplb_moe_forward */
  int32_t phase2_copy;      /* 1: feplb_moe_forward really copies, for every migrated piece, the expert's
                               weights into a receive buffer of R*max_num_dyn slots and the piece's rows
                               into a receive region (Section 2.2, Phase 2: tokens and weights; Section
                               2.3, memory paragraph) with device-to-device transfers that overlap the
                               static-expert GEMM, and the dynamic GEMM reads both from there.
                               0 (default): a migration only relabels the executing rank. */
} feplb_config;

/* One copy of the plan: `rows` rows of `expert` leave home rank `src` for rank `dst`. */
typedef struct { int32_t expert, src, dst, rows; } feplb_move;

/* One segment of the grouped GEMM: rows [row_start, row_start + rows) of the permuted buffers
 * belong to `expert` and are executed on virtual rank `exec_rank`.  is_dynamic: 0 = static expert,
 * 1 = dynamic expert computed with its home weights, 2 + s = dynamic expert whose weights are read
 * from slot s of the context's receive buffer and whose rows are read from the context's receive
 * region of rows, at the same row numbers (phase2_copy). */
typedef struct { int32_t expert, row_start, rows, exec_rank, is_dynamic; } feplb_group;

/* Caller-sized plan.  cap_moves >= R*max_num_dyn and cap_groups >= E + R*max_num_dyn always
 * suffice; load_before / load_after have R entries.  All host memory, owned by the caller. */
typedef struct {
  int32_t n_moves, n_groups;
  int32_t cap_moves, cap_groups;
  feplb_move* moves;
  feplb_group* groups;
  int64_t* load_before;
  int64_t* load_after;
} feplb_plan_out;

/* Host and device timestamps of the last feplb_moe_forward, in microseconds.  Host times count
 * from the call's entry; device times are CUDA-event intervals on the caller's stream. */
typedef struct {
  double host_enqueue_static_done_us; /* host: static-expert GEMM enqueued */
  double host_counts_ready_us;        /* host planner thread: counts arrived */
  double host_plan_done_us;           /* host planner thread: plan computed */
  double host_upload_enqueued_us;     /* host planner thread: group-table upload enqueued */
  double host_join_us;                /* host: caller joined the planner */
  double host_return_us;              /* host: everything enqueued */
  double plan_us;                     /* host: time inside the planner's greedy */
  double dev_hist_us, dev_dispatch_us, dev_static_ffn_us, dev_dynamic_ffn_us, dev_combine_us;
  double dev_counts_to_static_start_us; /* device: counts copied -> static GEMM starts */
  double dev_counts_to_static_end_us;   /* device: counts copied -> static GEMM ends */
  double dev_total_us;
  double dev_counts_to_copies_done_us;  /* device: counts copied -> Phase-2 weight copies landed (0 if none) */
  double phase2_copy_bytes;             /* bytes moved by those copies */
  /* Merged launches only (one launch per pass walks the static, then the dynamic groups); the
   * marks are taken inside the kernels from the GPU's global timer.  There dev_static_ffn_us is the
   * whole expert FFN, dev_dynamic_ffn_us is 0, dev_counts_to_static_start_us ends at the first CTA's
   * start and dev_counts_to_static_end_us at the first moment a CTA ran out of static work. */
  double dev_ffn_pass1_us, dev_ffn_pass2_us; /* device: first CTA's start -> last CTA's end of each pass */
  double dev_plan_wait_us;              /* device: longest time a CTA spent waiting for the dynamic table */
  double ffn_launches;                  /* GEMM launches of the forward: 4 (static, dynamic x 2 passes) or 2 */
} feplb_timeline;

typedef struct feplb_ctx feplb_ctx;

/* ---- library ------------------------------------------------------------------------------ */

/* Version as major*10000 + minor*100 + patch. */
int feplb_version(void);
/* Static text for a feplb_status. */
const char* feplb_strerror(int status);

/* ---- context ------------------------------------------------------------------------------ */

/* Validates `cfg`, selects the current CUDA device, allocates the context's scratch (block
 * histograms, segment offsets, group tables, pinned staging, status word), creates the copy
 * stream and starts the planner thread.  *out is NULL on failure. */
int feplb_create(const feplb_config* cfg, feplb_ctx** out);
/* Joins the planner thread and frees everything.  NULL is accepted. */
int feplb_destroy(feplb_ctx* ctx);
/* Text of the last error recorded on `ctx` (never NULL; empty if none). */
const char* feplb_last_error(const feplb_ctx* ctx);
/* Synchronises `stream`, reads and clears the device status word.  Returns FEPLB_OK,
 * FEPLB_E_RANGE (bad expert id), FEPLB_E_DEVICE (a device-side wait gave up or counts
 * disagreed with ids) or FEPLB_E_CUDA. */
int feplb_check_status(feplb_ctx* ctx, void* stream);
/* Rows the caller must give x_perm, h_scratch, y_perm and row_to_token:
 * S + E*(A-1), an upper bound of sum_e round_up(counts[e], A); 0 if cfg is invalid. */
size_t feplb_s_pad(const feplb_config* cfg);

/* ---- host-only steps (no GPU needed) ------------------------------------------------------ */

/* Static/dynamic partition (Section 2.3, parameter dyn): marks the `dyn` highest-scoring
 * experts of each rank's block in mask_out[E] (host), ties to the lower expert id.  The paper
 * does not say which experts are dynamic; scoring by this micro-batch's counts is this
 * library's reading. */
int feplb_select_dynamic(const int64_t* score, int32_t E, int32_t R, int32_t dyn, uint8_t* mask_out);

/* The greedy load balancer of Section 2.3: repeatedly moves the busiest dynamic expert of the
 * most loaded rank to the least loaded rank of the same domain, subject to tau, to the receive
 * capacity max_num_dyn, and to the move lowering the larger of the two loads; deterministic
 * (ties to the lower rank / expert id).  counts[E] and dyn_mask[E] are host arrays.  Fills
 * out->moves (ordered), out->groups (expert order; per expert the moved pieces in move order
 * from the front of its segment, then the home remainder; zero-row groups omitted) and the
 * per-rank loads.  Returns FEPLB_E_NOMEM if a capacity is too small.  Pure function. */
int feplb_plan(const feplb_config* cfg, const int32_t* counts, const uint8_t* dyn_mask, feplb_plan_out* out);

/* Macro level (Section 2.3: a Router Predictor re-places experts from historical routing
 * statistics at checkpoint time; the paper gives no algorithm).  feplb_ema_update keeps the
 * statistics: ema[e] <- decay*ema[e] + (1-decay)*counts[e] (host arrays of E entries).
 * feplb_place_experts assigns experts to ranks by the capacity-constrained longest-processing-time
 * greedy: experts by descending load (ties to the lower id), each to the least loaded rank that
 * still has room for one of its E/R experts (ties to the lower rank).  new_index[e] (host, E
 * entries) is the position expert e moves to; its new home rank is new_index[e] / (E/R).  The
 * caller permutes the weights and maps router ids through new_index. */
int feplb_ema_update(double* ema, const int32_t* counts, int32_t E, double decay);
int feplb_place_experts(const double* load, int32_t E, int32_t R, int32_t* new_index);

/* Expert parallelism over R real ranks (Section 2.2, Phases 1 and 2; Section 2.3: every device
 * derives the same plan by itself from the counts all devices know after Phase 1).  Host logic
 * only: the row exchange and the peer copies themselves are the caller's (no multi-GPU data plane
 * is part of this library yet).  Rank s holds its own tokens; counts_by_src[s*E + e] is the number
 * of its (token, k) slots routed to expert e -- the R x E matrix every rank has after one
 * all-gather of its row.  From it every rank computes, identically:
 *   - counts[e] = sum_s counts_by_src[s][e] and the plan of feplb_plan on them (written to *plan);
 *     the rows of expert e are ordered by source rank, then by slot, which is the order
 *     feplb_dispatch gives when the ranks' tokens are numbered one rank after the other;
 *   - Phase 1, dispatch all-to-all-v: rank s sends counts_by_src[s][e] rows to home(e);
 *   - Phase 2: for move i (expert, src = home, dst, rows) the first not yet moved `rows` rows of
 *     the expert's segment and the expert's three weight matrices go from src to slot
 *     dst*max_num_dyn + (number of earlier moves into dst) of dst's receive buffer;
 *   - Combine: every executed row returns from the rank that ran it straight to its source rank.
 * Outputs for `rank` (host arrays of R entries each, any may be NULL): rows it sends to / receives
 * from every rank in Phase 1, in Phase 2 and in the combine; copies[0..*n_copies) lists ALL weight
 * copies in move order (cap_copies >= R*max_num_dyn always suffices; FEPLB_E_NOMEM otherwise). */
typedef struct { int32_t expert, src, dst, slot, rows; int64_t weight_bytes; } feplb_weight_copy;
int feplb_ep_schedule(const feplb_config* cfg, const int32_t* counts_by_src, const uint8_t* dyn_mask, int32_t rank,
                      feplb_plan_out* plan, int64_t* p1_send, int64_t* p1_recv, int64_t* p2_send, int64_t* p2_recv,
                      int64_t* comb_send, int64_t* comb_recv, feplb_weight_copy* copies, int32_t cap_copies,
                      int32_t* n_copies);

/* ---- device steps ------------------------------------------------------------------------- */

/* Step 0, optional (Section 2.3, router; Section 3.1, top-k routing without auxiliary loss):
 * top-k gating from router logits.  Per token the K largest of its E logits in
 * descending order, ties to the lower expert id; gates = softmax over the K selected logits
 * (fp32).  logits dev float [T,E] (finite values) -> topk_ids dev int32 [T,K], gates dev float [T,K]. */
int feplb_route_topk(feplb_ctx* ctx, const float* logits, int32_t* topk_ids, float* gates, void* stream);

/* Step 1 (Section 2.2: per-expert token counts after Phase 1).
 * topk_ids dev int32 [T,K] -> counts dev int32 [E], rank_load dev int32 [R] (both overwritten).
 * Ids outside [0,E) are skipped and raise FEPLB_E_RANGE in the status word. */
int feplb_route_hist(feplb_ctx* ctx, const int32_t* topk_ids, int32_t* counts, int32_t* rank_load, void* stream);

/* Step 3 (Section 2.2, Phase 1: rows are brought into expert order for the grouped GEMM) = stable counting sort of the
 * slots by expert id.  Slot s goes to row pad_off[e] + (earlier slots of e), with
 * pad_off[e] = sum_{e'<e} round_up(counts[e'], A).
 *   x dev bf16 [T,d], topk_ids dev [T,K], counts dev [E] (as written by feplb_route_hist)
 *   -> x_perm dev bf16 [S_cap,d]   (row copies; padding rows inside segments zero-filled)
 *      slot_to_row dev int32 [T,K], row_to_token dev int32 [S_cap] (-1 where no token). */
int feplb_dispatch(feplb_ctx* ctx, const void* x, const int32_t* topk_ids, const int32_t* counts,
                   void* x_perm, int32_t* slot_to_row, int32_t* row_to_token, void* stream);

/* Largest ceil(T*K/1024) * E that feplb_dispatch_noalloc accepts (ints of built-in scratch). */
#define FEPLB_NOALLOC_MAX_HIST_INTS 524288

/* (The paper has no counterpart to this entry point; it exists for deployment reasons only.)
 * feplb_dispatch for callers that cannot allocate device memory where they need a dispatch --
 * e.g. a server whose own pool already owns all free device memory, or a loop that cannot take
 * the device-wide synchronisation of cudaMalloc/cudaFree -- and therefore cannot create a
 * context either.  Same inputs, outputs and results as feplb_dispatch (cfg replaces the
 * context); the permutation's scratch is a ~2 MiB array built into the library image, resident
 * on every GPU that loads the library until the process exits.  This call allocates and frees
 * nothing, on the device or through any library.
 *   - Limit: ceil(T*K/1024) * E <= FEPLB_NOALLOC_MAX_HIST_INTS, else FEPLB_E_NOMEM is returned
 *     and nothing is enqueued (use feplb_dispatch).
 *   - The first call on each device looks the array's device address up once (with that device
 *     current); make that first call before any stream capture begins.
 *   - All calls on a device share the array, which keeps the previous call's contents (the
 *     kernels overwrite what they read before reading it).  Calls whose GPU work overlaps --
 *     other streams or threads -- race on it: serialise them.
 *   - status: dev uint32, zeroed by the caller, receives error bits (1 = expert id out of range,
 *     2 = counts disagree with topk_ids).  With NULL those errors cannot be detected at all (not
 *     merely ignored): the bits go to a spare word of the shared scratch that nothing reads.  In
 *     both cases the kernels stay inside the caller's buffers: an offending slot gets
 *     slot_to_row = -1 and its row is not written. */
int feplb_dispatch_noalloc(const feplb_config* cfg, const void* x, const int32_t* topk_ids,
                           const int32_t* counts, void* x_perm, int32_t* slot_to_row,
                           int32_t* row_to_token, uint32_t* status, void* stream);

/* Writes the E-entry group table {e, pad_off[e], counts[e], home(e), dyn_mask[e]} to
 * groups_out (dev), from device-resident counts and mask, without involving the host: the
 * table the static-expert GEMM runs on while the planner works (Section 2.3 timeline).
 * With FEPLB_MASK_REACTIVE pass dyn_mask = NULL: the mask is derived on the device from counts
 * (same rule as feplb_select_dynamic) and also written to dyn_mask_out (dev uint8 [E], may be NULL). */
int feplb_home_groups(feplb_ctx* ctx, const int32_t* counts, const uint8_t* dyn_mask,
                      feplb_group* groups_out, uint8_t* dyn_mask_out, void* stream);

/* Expert weights enter the library output-major (w1, w3 [E,f,d]; w2 [E,d,f]) -- the only layout the
 * GEMM entry points accept, because both operands of every contraction are then contiguous along
 * the contracted dimension.  A caller that holds them input-major, as the operator is usually
 * written (y = (silu(x W1) * (x W3)) W2 with W1, W3 [E,d,f] and W2 [E,f,d]), converts them once per
 * weight update with this call: w1_in, w3_in dev bf16 [E,d,f], w2_in dev bf16 [E,f,d]
 * -> w1, w3 dev bf16 [E,f,d], w2 dev bf16 [E,d,f] (distinct buffers).  feplb_transpose_weights below
 * is the opposite direction (it makes the copies the backward pass reads). */
int feplb_pack_weights(feplb_ctx* ctx, const void* w1_in, const void* w3_in, const void* w2_in,
                       void* w1, void* w3, void* w2, void* stream);

/* Steps 4-5 (Section 2.3: static-expert, then dynamic-expert grouped GEMM).  For every group g
 * in groups[0..n_groups) selected by `which` (FEPLB_FFN_ALL / _STATIC: is_dynamic == 0 /
 * _DYNAMIC: is_dynamic != 0) and every row i of it:
 *   h = silu(x_perm[i] W1[e]) * (x_perm[i] W3[e])   (bf16 x bf16 -> fp32, h rounded to bf16)
 *   y_perm[i] = h W2[e]                              (fp32 accumulate, rounded to bf16)
 * Rows outside the selected groups are not written.  groups is a dev array (n_groups <= 1024);
 * zero-row groups are allowed.  h_scratch dev bf16 [S_cap,f], y_perm dev bf16 [S_cap,d]. */
int feplb_expert_ffn(feplb_ctx* ctx, const void* x_perm, const void* w1, const void* w3, const void* w2,
                     const feplb_group* groups, int32_t n_groups, int32_t which,
                     void* h_scratch, void* y_perm, void* stream);

/* Step 6 (Section 2.3: Combine): out[t,:] = sum_k gates[t,k] * y_perm[slot_to_row[t,k],:],
 * k ascending, fp32 accumulate, rounded to bf16.  gates dev float [T,K], out dev bf16 [T,d]. */
int feplb_combine(feplb_ctx* ctx, const void* y_perm, const int32_t* slot_to_row, const float* gates,
                  void* out, void* stream);

/* ---- backward pass -------------------------------------------------------------------------- *
 * The paper reports forward/backward layer times (Table 2) without describing the backward
 * pass; these entry points compute the derivative of the forward definition
 *   out[t] = sum_k gates[t,k] * ((silu(x W1[e]) * (x W3[e])) W2[e]),  e = topk_ids[t,k]
 * over the same expert-contiguous rows and groups.  bf16 operands, fp32 accumulation; gradients
 * of activations are bf16, of gates and weights fp32. */

/* While `ab` (dev bf16 [S_cap, 2f], caller-owned) is set, pass 1 of every feplb_expert_ffn /
 * feplb_moe_forward on this context also stores the pre-activations a = x W1[e] (columns [0,f))
 * and b = x W3[e] (columns [f,2f)) of every row, which the backward pass needs.  NULL turns it off. */
int feplb_set_preact_buffer(feplb_ctx* ctx, void* ab);
/* Transposed copies of the expert weights, needed by the activation gradients (their contractions
 * run over the weights' slow dimension): w1t, w3t dev bf16 [E, d, f]; w2t dev bf16 [E, f, d]. */
int feplb_transpose_weights(feplb_ctx* ctx, const void* w1, const void* w3, const void* w2,
                            void* w1t, void* w3t, void* w2t, void* stream);
/* Backward of feplb_combine: for every slot (t,k) with row r = slot_to_row[t,k]
 *   d_y_perm[r,:] = gates[t,k] * d_out[t,:]   (bf16)      d_gates[t,k] = <d_out[t,:], y_perm[r,:]>   (fp32)
 * d_out dev bf16 [T,d]; y_perm as left by the forward pass; d_y_perm dev bf16 [S_cap,d]; d_gates dev float [T,K]. */
int feplb_combine_bwd(feplb_ctx* ctx, const void* d_out, const void* y_perm, const int32_t* slot_to_row,
                      const float* gates, void* d_y_perm, float* d_gates, void* stream);
/* Backward of feplb_expert_ffn over the selected groups (same table and selector as the forward):
 *   dH = d_y_perm W2[e];  dA = dH * b * silu'(a);  dB = dH * silu(a)      -> d_ab [S_cap, 2f] (scratch, bf16)
 *   d_x_perm = dA W1[e]^T + dB W3[e]^T                                       -> dev bf16 [S_cap, d]
 * and, if dw1/dw3/dw2 are given (dev float [E,f,d], [E,f,d], [E,d,f]), the weight gradients of ALL
 * experts listed in expert_table (dev feplb_group[E], e.g. from feplb_home_groups: first row and
 * row count of each expert's segment), accumulated over each expert's rows in fp32:
 *   dW2[e] = d_y_e^T H_e,  dW1[e] = dA_e^T X_e,  dW3[e] = dB_e^T X_e   (overwritten, or added to if accumulate != 0;
 *   experts without rows get zeros / stay unchanged).
 * Weight gradients need cfg.row_align = 128: the contraction runs over whole 64-row blocks of an
 * expert's segment, read in place, so the call first writes zeros to the padding rows (from the
 * expert's row count up to the next multiple of 128) of h, d_y_perm and d_ab; x_perm's are zero
 * already (feplb_dispatch).  ab_saved: the buffer of feplb_set_preact_buffer; h: the forward's h_scratch. */
int feplb_expert_ffn_bwd(feplb_ctx* ctx, const void* x_perm, const void* ab_saved, void* h,
                         void* d_y_perm, const void* w1t, const void* w3t, const void* w2t,
                         const feplb_group* groups, int32_t n_groups, int32_t which,
                         const feplb_group* expert_table, void* d_ab,
                         void* d_x_perm, float* dw1, float* dw3, float* dw2, int32_t accumulate,
                         void* stream);
/* Backward of feplb_dispatch: d_x[t,:] = sum_k d_x_perm[slot_to_row[t,k],:] (fp32 sum, bf16 out). */
int feplb_dispatch_bwd(feplb_ctx* ctx, const void* d_x_perm, const int32_t* slot_to_row, void* d_x, void* stream);
/* The three steps above for the micro-batch whose feplb_moe_forward ran last on this context (its
 * expert table is reused): d_out -> d_x [T,d], d_gates [T,K], and the weight gradients (or NULLs). */
int feplb_moe_backward(feplb_ctx* ctx, const void* d_out, const float* gates, const void* w1t, const void* w3t,
                       const void* w2t, const void* x_perm, const void* ab_saved, void* h,
                       const void* y_perm, const int32_t* slot_to_row,
                       void* d_y_perm, void* d_ab, void* d_x_perm, void* d_x, float* d_gates,
                       float* dw1, float* dw3, float* dw2, int32_t accumulate, void* stream);

/* ---- planner thread (Section 2.3: CPU balancer on a dedicated thread) ---------------------- */

/* Enqueues on `stream` a copy of counts (dev [E]) to pinned memory and wakes the planner
 * thread, which waits for the copy (bounded), chooses the mask (dyn_mask_host, host [E], must
 * stay valid until feplb_plan_wait; NULL with FEPLB_MASK_REACTIVE), runs feplb_plan, and uploads
 * the dynamic groups on the context's copy stream. */
int feplb_plan_async(feplb_ctx* ctx, const int32_t* counts, const uint8_t* dyn_mask_host, void* stream);
/* Waits up to timeout_ms for the planner.  On success copies the plan to *plan_copy (may be
 * NULL), returns the device table of dynamic groups and its length, and makes `stream` wait
 * for the upload.  FEPLB_E_TIMEOUT on expiry (the job stays pending), FEPLB_E_STATE if no job. */
int feplb_plan_wait(feplb_ctx* ctx, int32_t timeout_ms, feplb_plan_out* plan_copy,
                    const feplb_group** dyn_groups_dev, int32_t* n_dyn_groups, void* stream);

/* ---- whole layer -------------------------------------------------------------------------- */

/* One forward pass of the layer on `stream`: route_hist -> (planner thread || dispatch, static
 * FFN) -> dynamic FFN -> combine.  Inputs x, topk_ids, gates, w1, w3, w2 (dev).  Outputs and
 * scratch (dev, caller-owned): counts [E], rank_load [R], x_perm [S_cap,d], h_scratch [S_cap,f],
 * y_perm [S_cap,d], slot_to_row [T,K], row_to_token [S_cap], out [T,d].  dyn_mask_host: host [E]
 * or NULL with FEPLB_MASK_REACTIVE.  plan_copy (host, may be NULL) receives the plan.  Blocks the
 * calling thread only until the planner has enqueued its upload (bounded by 2 s). */
int feplb_moe_forward(feplb_ctx* ctx, const void* x, const int32_t* topk_ids, const float* gates,
                      const void* w1, const void* w3, const void* w2, const uint8_t* dyn_mask_host,
                      int32_t* counts, int32_t* rank_load, void* x_perm, void* h_scratch, void* y_perm,
                      int32_t* slot_to_row, int32_t* row_to_token, void* out,
                      feplb_plan_out* plan_copy, void* stream);

/* Same pass with HOST inputs and output: copies x, topk_ids, gates (host, ideally pinned) to
 * the device buffers x_dev, ids_dev, gates_dev, runs feplb_moe_forward, copies out_dev to
 * out_host, all on `stream`; returns after the stream has drained.  Weights stay resident. */
int feplb_moe_forward_host(feplb_ctx* ctx, const void* x_host, const int32_t* topk_ids_host,
                           const float* gates_host, void* x_dev, int32_t* ids_dev, float* gates_dev,
                           const void* w1, const void* w3, const void* w2, const uint8_t* dyn_mask_host,
                           int32_t* counts, int32_t* rank_load, void* x_perm, void* h_scratch, void* y_perm,
                           int32_t* slot_to_row, int32_t* row_to_token, void* out_dev, void* out_host,
                           feplb_plan_out* plan_copy, void* stream);

/* Pipelined form of feplb_moe_forward_host for back-to-back micro-batches.  `slot`
 * (0 .. FEPLB_HOST_SLOTS-1) names one of the caller-owned staging sets (x_dev, ids_dev, gates_dev,
 * out_dev and the host buffers must differ between slots in use; the other buffers are shared;
 * two slots suffice to overlap copies with kernels, more keep the host from waiting on a result
 * copy that is still in flight before it can launch the next forward).  The call copies the inputs
 * on the context's input stream, runs the forward on `stream` once they have arrived, copies the
 * result to out_host on the context's output stream, and returns without waiting for any of it
 * (it still blocks briefly for the planner, like feplb_moe_forward).  So the copies of micro-batch
 * i+1 overlap the kernels of micro-batch i.  Before reusing a slot's host buffers, or reading
 * out_host, call feplb_host_wait(ctx, slot). */
#define FEPLB_HOST_SLOTS 4
int feplb_moe_forward_host_async(feplb_ctx* ctx, int32_t slot, const void* x_host, const int32_t* topk_ids_host,
                                 const float* gates_host, void* x_dev, int32_t* ids_dev, float* gates_dev,
                                 const void* w1, const void* w3, const void* w2, const uint8_t* dyn_mask_host,
                                 int32_t* counts, int32_t* rank_load, void* x_perm, void* h_scratch, void* y_perm,
                                 int32_t* slot_to_row, int32_t* row_to_token, void* out_dev, void* out_host,
                                 feplb_plan_out* plan_copy, void* stream);
/* Optional prefetch for feplb_moe_forward_host_async: starts the copies of a micro-batch's inputs
 * (host, pinned) into the staging set of `slot` on the context's input stream, after the forward
 * that last read that staging set, and returns at once.  The next feplb_moe_forward_host_async
 * on this slot then uses what was staged and ignores its three host input pointers.  Called
 * for micro-batch i+1 before the forward of micro-batch i, it lets the input copies run under
 * a whole forward instead of only under its tail.  The host buffers must stay untouched until that
 * forward's feplb_host_wait. */
int feplb_host_stage_inputs(feplb_ctx* ctx, int32_t slot, const void* x_host, const int32_t* topk_ids_host,
                            const float* gates_host, void* x_dev, int32_t* ids_dev, float* gates_dev);
/* Blocks until the result of the last feplb_moe_forward_host_async on `slot` is in its out_host. */
int feplb_host_wait(feplb_ctx* ctx, int32_t slot);

/* Turns CUDA-event timing of the stages of feplb_moe_forward on (1) or off (0, default). */
int feplb_set_timeline(feplb_ctx* ctx, int32_t enable);
/* Waits for the last forward's stage events and fills *out (device fields are 0 when timing was
 * off during that forward). */
int feplb_get_timeline(feplb_ctx* ctx, feplb_timeline* out);
/* Sums of every field over the forwards run with timing on since the last reset, and their
 * number.  The stage events of up to 16 forwards stay outstanding, so timing does not make the
 * host wait for the GPU between forwards; this call waits for the outstanding ones. */
int feplb_timeline_totals(feplb_ctx* ctx, feplb_timeline* sum, int64_t* n_forwards, int32_t reset);
/* Bound (milliseconds, default 2000) of the planner thread's wait for the counts.  When it expires
 * the pending plan fails with FEPLB_E_TIMEOUT (returned by feplb_plan_wait / feplb_moe_forward) and
 * the context stays usable.  Not allowed while a plan is pending. */
int feplb_set_planner_timeout(feplb_ctx* ctx, int32_t timeout_ms);
/* Which form of the grouped-GEMM kernel the context uses.  forward_form: FEPLB_FORM_AUTO (default:
 * chosen from the geometry and, per group table, from the rows per group), FEPLB_FORM_SINGLE (one
 * CTA per 128-row tile), FEPLB_FORM_PAIR (clusters of two CTAs on 256-row tiles) or
 * FEPLB_FORM_WEIGHT_M (weight tiles on the M side, up to 256 rows of a group on the N side; needs
 * f % 128 == 0, d % 256 == 0 and 2*E + R*max_num_dyn <= 1024, else FEPLB_E_INVALID) for every
 * forward launch.
 * backward_pair: -1 (default: chosen from the geometry) or a mask, bit 0 = activation-gradient
 * GEMMs in the pair form, bit 1 = weight-gradient GEMMs in the pair form.  Results do not depend
 * on the form beyond fp32 summation order.  Not allowed while a plan is pending. */
int feplb_set_gemm_form(feplb_ctx* ctx, int32_t forward_form, int32_t backward_pair);
/* How feplb_moe_forward launches the expert GEMMs.  merged = 1: one launch per pass runs the static
 * groups (Section 2.3: while the CPU balancer works) and then the dynamic groups, whose table it
 * picks up on the device with a bounded wait on a word the planner thread writes into mapped host
 * memory -- two launches per forward, everything enqueued before the planner is joined, the
 * static-first order kept inside each launch.  merged = 0: static and dynamic groups in launches of
 * their own (four per forward), the dynamic ones enqueued after the planner has been joined and
 * each table in the form that suits it.  -1 (default): merged while a forward's groups are small
 * (below ~768 rows per expert).  With cfg.phase2_copy the four-launch order is always used.
 * merged = 1 needs 2*E + R*max_num_dyn <= 1024.  Not allowed while a plan is pending. */
int feplb_set_launch_merging(feplb_ctx* ctx, int32_t merged);
/* Test and tuning aid for the merged launches of feplb_moe_forward.  planner_delay_us: the
 * planner thread sleeps that long before it publishes its table (0 = off), so that the GEMM's
 * device-side wait for the table really is entered.  device_wait_limit_us: bound of that wait
 * (0 = the default, 400 ms); when it expires the kernels skip the dynamic groups, raise a status
 * bit that feplb_check_status reports as FEPLB_E_TIMEOUT, and return normally.  Not allowed while
 * a plan is pending. */
int feplb_set_planner_timing(feplb_ctx* ctx, int32_t planner_delay_us, int32_t device_wait_limit_us);
/* Self-test of the device-side bounded waits: launches one thread that waits, with the routine
 * the GEMM kernels use, on an mbarrier nothing ever completes, limited to limit_us microseconds.
 * Returns FEPLB_OK if the wait gave up, raised the status bit and the kernel returned normally;
 * FEPLB_E_STATE otherwise.  The status word is clear afterwards.  Synchronises `stream`. */
int feplb_selftest_bounded_wait(feplb_ctx* ctx, int32_t limit_us, void* stream);
/* Number of kernels this library has launched on `ctx` since creation. */
int64_t feplb_launch_count(const feplb_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* FEPLB_H_ */
