// C ABI of libfeplb: context, argument checks, the planner thread (paper Section 2.3: the CPU
// load balancer runs on a dedicated thread, triggered by router completion, while the GPU
// computes the static experts) and the per-micro-batch orchestration.
#include <cuda_runtime.h>

#include <atomic>
#include <chrono>
#include <climits>
#include <condition_variable>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "feplb.h"
#include "feplb_internal.h"

namespace {
using clk = std::chrono::steady_clock;
inline double us_since(clk::time_point t0) {
  return std::chrono::duration<double, std::micro>(clk::now() - t0).count();
}
enum JobState { JOB_IDLE = 0, JOB_PENDING = 1, JOB_RUNNING = 2, JOB_DONE = 3 };
enum { EV_T0 = 0, EV_HIST, EV_DISPATCH, EV_STATIC0, EV_STATIC1, EV_DYN0, EV_DYN1, EV_COMBINE, EV_COUNTS, EV_COPIES, EV_STAMPS, EV_N };
constexpr int kEvRing = 16;   // forwards whose stage events may be outstanding
constexpr int kStampWords = 16;   // [0..3] pass 1, [4..7] pass 2 (see WmParams::stamps), [8] counts left the device
}  // namespace

struct feplb_ctx {
  feplb_config cfg;
  int device = 0, num_sms = 0;
  size_t s_cap = 0;
  int nb = 0;   // CTAs of the permutation kernels
  char err[512] = {0};
  int64_t launches = 0;
  int gemm_pair_default = 0;   // GEMM form for launches whose group sizes the host does not know
  int gemm_pair_forced = -1;   // feplb_set_gemm_form: 0/1 forces one form everywhere, -1 = chosen per table
  int bwd_pair = 0;            // backward GEMMs in the pair form: bit 0 activation gradients, bit 1 weight gradients
  int gemm_pair_auto = 0, bwd_pair_auto = 0;   // the choices feplb_create derived from the geometry
  bool wm_ok = false;          // the weights-on-M form supports this geometry
  bool wm = false;             // ... and is the form in use (feplb_create's choice or feplb_set_gemm_form)
  bool wm_auto = false;
  bool merged_ok = false;      // both group tables of a forward fit one launch (static, then dynamic groups)
  bool merged = false;         // ... and feplb_moe_forward runs that way: two GEMM launches instead of four
  bool merged_auto = false;
  bool merged_pair = false;    // form of the merged launches when none is forced
  int32_t planner_delay_us = 0;        // test aid: the planner sleeps before it publishes its table
  int32_t device_wait_limit_us = 0;    // bound of the GEMM's wait for the table (0: default)
  // weights-on-M form: the words through which a running GEMM launch learns that the dynamic table exists
  int32_t* h_dyn_tab32 = nullptr;                    // pinned + mapped: the dynamic table as 32-byte entries tagged with the sequence number
  int32_t* h_dyn_tab32_dev = nullptr;                // its device address
  int32_t* d_dyn_tab32 = nullptr;                    // device copy, made by the GEMM's claiming CTA
  unsigned long long* d_dyn_ready = nullptr;         // device words: [0] ready, [1] claim
  unsigned long long* h_dyn_ready = nullptr;         // pinned + mapped word, set by the planner thread
  unsigned long long* h_dyn_ready_dev = nullptr;     // its device address
  unsigned long long* d_stamps = nullptr;            // [kEvRing][kStampWords] globaltimer marks of the kernels
  unsigned long long* h_stamps = nullptr;            // pinned copy, filled at the end of a timed forward
  bool job_wm = false;

  // device scratch
  int32_t* d_block_hist = nullptr;
  int32_t* d_pad_off = nullptr;
  uint32_t* d_status = nullptr;
  feplb_group* d_home_groups = nullptr;
  feplb_group* d_dyn_groups = nullptr;
  uint8_t* d_mask = nullptr;
  // Phase-2 receive buffer: R*max_num_dyn slots of one expert's weights each (phase2_copy)
  void* d_recv_w1 = nullptr;
  void* d_recv_w3 = nullptr;
  void* d_recv_w2 = nullptr;
  int n_recv_slots = 0;
  void* d_recv_x = nullptr;    // Phase-2 receive region of the migrated pieces' rows: [s_cap, d], same row numbers as x_perm
  cudaEvent_t ev_gather = nullptr;          // the permuted rows of the current forward are written
  std::atomic<int32_t> gather_seq{0};       // ... recorded for the forward with this sequence number
  const void* job_x_perm = nullptr;
  void* d_preact = nullptr;   // caller-owned [s_cap, 2f]: pass 1 saves a | b there when set (training)
  // pinned staging
  int32_t* h_counts = nullptr;
  feplb_group* h_dyn_groups = nullptr;          // pinned and mapped: the upload kernel reads it through h_dyn_groups_dev
  feplb_group* h_dyn_groups_dev = nullptr;
  uint32_t* h_status = nullptr;
  uint8_t* h_mask = nullptr;
  unsigned long long* h_counts_tagged = nullptr;   // pinned, written by the scan kernel: (sequence number << 32) | count
  int32_t flag_seq = 0;
  int32_t job_flag_seq = 0;          // 0: the job waits on ev_counts instead
  int32_t planner_timeout_ms = 2000; // bound of the planner's wait for the counts

  cudaStream_t copy_stream = nullptr;
  // pipelined host-buffer path: input and output copy streams and per-slot events
  cudaStream_t in_stream = nullptr, out_stream = nullptr;
  cudaEvent_t ev_in[FEPLB_HOST_SLOTS] = {}, ev_done[FEPLB_HOST_SLOTS] = {}, ev_out[FEPLB_HOST_SLOTS] = {};
  bool slot_used[FEPLB_HOST_SLOTS] = {};
  bool slot_staged[FEPLB_HOST_SLOTS] = {};     // inputs already on their way (feplb_host_stage_inputs)
  cudaEvent_t ev_counts = nullptr, ev_plan = nullptr;
  cudaEvent_t evr[kEvRing][EV_N] = {{nullptr}};
  cudaEvent_t* ev = evr[0];        // event set of the current forward
  bool ev_used[kEvRing] = {false};
  feplb_timeline ev_host[kEvRing]; // host fields of the forward that used the set
  int ev_slot = 0;
  bool timeline_on = false, timeline_valid = false;
  feplb_timeline tl;               // host fields of the current forward
  feplb_timeline tl_sum;           // totals over harvested forwards
  feplb_timeline tl_last;          // last harvested forward
  int64_t tl_n = 0;
  clk::time_point t0;

  // planner thread
  std::thread th;
  std::mutex mu;
  std::condition_variable cv;
  bool quit = false;
  int job = JOB_IDLE;
  const uint8_t* job_mask = nullptr;
  const void* job_w1 = nullptr;   // weights of the current forward (sources of the Phase-2 copies)
  const void* job_w3 = nullptr;
  const void* job_w2 = nullptr;
  double copy_bytes = 0;
  int job_rc = FEPLB_OK;
  int n_dyn_groups = 0;
  int dyn_pair = 0;   // GEMM form chosen by the planner for the dynamic groups (it knows their sizes)
  // plan storage owned by the context
  std::vector<feplb_move> moves;
  std::vector<feplb_group> groups;
  std::vector<int64_t> load_before, load_after;
  std::vector<uint8_t> mask;
  feplb_plan_out plan;
};

namespace {

int fail(feplb_ctx* c, int code, const char* fmt, ...) {
  if (c) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(c->err, sizeof(c->err), fmt, ap);
    va_end(ap);
  }
  return code;
}
#define CUDA_TRY(ctx, call)                                                                      \
  do {                                                                                           \
    cudaError_t e_ = (call);                                                                     \
    if (e_ != cudaSuccess) return fail(ctx, FEPLB_E_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The planner thread: waits for the counts, derives mask and plan, uploads the dynamic groups.
void planner_main(feplb_ctx* c) {
  cudaSetDevice(c->device);
  for (;;) {
    {
      std::unique_lock<std::mutex> lk(c->mu);
      c->cv.wait(lk, [&] { return c->quit || c->job == JOB_PENDING; });
      if (c->quit) return;
      c->job = JOB_RUNNING;
    }
    int rc = FEPLB_OK;
    // bounded wait for the counts: either the scan kernel writes them straight into pinned host
    // memory, each tagged with the forward's sequence number (whole-layer path), or a copy was enqueued and its event is
    // polled (stand-alone feplb_plan_async); no blocking driver call either way
    const auto w0 = clk::now();
    for (uint32_t spin = 0;; ++spin) {
      if (c->job_flag_seq) {
        int e = 0;
        for (; e < c->cfg.E; ++e) {
          const unsigned long long v = *(volatile unsigned long long*)(c->h_counts_tagged + e);
          if ((int32_t)(v >> 32) != c->job_flag_seq) break;
          c->h_counts[e] = (int32_t)(uint32_t)v;
        }
        if (e == c->cfg.E) break;
      } else {
        cudaError_t q = cudaEventQuery(c->ev_counts);
        if (q == cudaSuccess) break;
        if (q != cudaErrorNotReady) { rc = FEPLB_E_CUDA; break; }
      }
      if ((spin & 1023u) == 1023u && std::chrono::duration<double>(clk::now() - w0).count() > 1e-3 * c->planner_timeout_ms) { rc = FEPLB_E_TIMEOUT; break; }
#if defined(__x86_64__) || defined(__i386__)
      __builtin_ia32_pause();     // a polite spin: the sibling hyper-thread (another rank's host thread) keeps its issue slots
#endif
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    c->tl.host_counts_ready_us = us_since(c->t0);
    if (rc == FEPLB_OK) {
      const feplb_config& cfg = c->cfg;
      const uint8_t* mask = c->job_mask;
      if (!mask) {
        std::vector<int64_t> score(cfg.E);
        for (int e = 0; e < cfg.E; ++e) score[e] = c->h_counts[e];
        feplb_select_dynamic(score.data(), cfg.E, cfg.R, cfg.dyn, c->mask.data());
        mask = c->mask.data();
      } else {
        memcpy(c->mask.data(), mask, cfg.E);
      }
      const auto p0 = clk::now();
      rc = feplb_plan(&cfg, c->h_counts, mask, &c->plan);
      c->tl.plan_us = us_since(p0);
      c->tl.host_plan_done_us = us_since(c->t0);
      if (rc == FEPLB_OK) {
        int n = 0;
        for (int i = 0; i < c->plan.n_groups; ++i)
          if (c->plan.groups[i].is_dynamic) c->h_dyn_groups[n++] = c->plan.groups[i];
        c->n_dyn_groups = n;
        cudaError_t ce = cudaSuccess;
        c->copy_bytes = 0;
        if (cfg.phase2_copy && c->job_w1) {
          // Phase 2 (Section 2.2): the weights of every migrated expert travel to the receiving
          // rank's buffer on the copy engines while the SMs compute the static experts.  Move i
          // takes the next free slot of its destination rank; the piece's group then reads slot s.
          const int L = cfg.E / cfg.R;
          const size_t per = (size_t)cfg.d * cfg.f * 2;
          std::vector<int> next_slot(cfg.R, 0), move_slot(c->plan.n_moves, 0);
          for (int i = 0; i < c->plan.n_moves && ce == cudaSuccess; ++i) {
            const feplb_move& m = c->plan.moves[i];
            const int s = m.dst * cfg.max_num_dyn + next_slot[m.dst]++;
            move_slot[i] = s;
            const char* src[3] = {(const char*)c->job_w1, (const char*)c->job_w3, (const char*)c->job_w2};
            char* dst[3] = {(char*)c->d_recv_w1, (char*)c->d_recv_w3, (char*)c->d_recv_w2};
            for (int k = 0; k < 3 && ce == cudaSuccess; ++k)
              ce = cudaMemcpyAsync(dst[k] + per * s, src[k] + per * m.expert, per, cudaMemcpyDeviceToDevice, c->copy_stream);
            c->copy_bytes += 3.0 * per;
          }
          std::vector<int> next_move(cfg.E, 0);   // per expert: moves consumed so far, in move order
          for (int g = 0; g < n; ++g) {
            feplb_group& gr = c->h_dyn_groups[g];
            if (gr.exec_rank == gr.expert / L) continue;      // home remainder: home weights
            int i = next_move[gr.expert];
            while (i < c->plan.n_moves && c->plan.moves[i].expert != gr.expert) ++i;
            next_move[gr.expert] = i + 1;
            if (i < c->plan.n_moves) gr.is_dynamic = 2 + move_slot[i];
          }
          // ... and so do the rows of the moved pieces (Section 2.2: Phase 2 redistributes tokens and
          // weights): each piece's rows go to the same row numbers of the receive region, once the
          // gather kernel of this forward has written them (the event is recorded by the calling thread,
          // which then publishes the forward's sequence number)
          if (ce == cudaSuccess && c->plan.n_moves > 0 && c->job_x_perm) {
            const auto g0 = clk::now();
            while (c->gather_seq.load(std::memory_order_acquire) != c->job_flag_seq &&
                   std::chrono::duration<double>(clk::now() - g0).count() < 1e-3 * c->planner_timeout_ms) {
#if defined(__x86_64__) || defined(__i386__)
              __builtin_ia32_pause();
#endif
            }
            if (c->gather_seq.load(std::memory_order_acquire) != c->job_flag_seq) ce = cudaErrorNotReady;
            if (ce == cudaSuccess) ce = cudaStreamWaitEvent(c->copy_stream, c->ev_gather, 0);
            const size_t row_bytes = (size_t)cfg.d * 2;
            for (int g = 0; g < n && ce == cudaSuccess; ++g) {
              const feplb_group& gr = c->h_dyn_groups[g];
              if (gr.is_dynamic < 2 || gr.rows <= 0) continue;
              ce = cudaMemcpyAsync((char*)c->d_recv_x + row_bytes * gr.row_start, (const char*)c->job_x_perm + row_bytes * gr.row_start,
                                   row_bytes * gr.rows, cudaMemcpyDeviceToDevice, c->copy_stream);
              c->copy_bytes += (double)row_bytes * gr.rows;
            }
          }
          if (ce == cudaSuccess && c->copy_bytes > 0) ce = cudaEventRecord(c->ev[EV_COPIES], c->copy_stream);
          if (ce != cudaSuccess) c->copy_bytes = 0;
          c->tl.phase2_copy_bytes = c->copy_bytes;
        }
        if (ce != cudaSuccess) rc = FEPLB_E_CUDA;
        int64_t dyn_rows = 0;
        for (int i = 0; i < n; ++i) dyn_rows += c->h_dyn_groups[i].rows;
        c->dyn_pair = c->gemm_pair_forced >= 0 ? c->gemm_pair_forced == FEPLB_FORM_PAIR : (n > 0 && dyn_rows >= (int64_t)512 * n);
        cudaError_t e = cudaSuccess;
        if (c->job_wm) {
          // A GEMM launch may already be running and waiting for this table (the merged launches
          // are never combined with Phase-2 copies): publish it from here, with a plain store into
          // mapped host memory, so that the waiting kernel depends on this thread alone.  The first
          // CTA that sees the word brings the table into device memory for the others; there is no
          // upload kernel on this path (it could not be relied on to run beside a kernel that holds
          // every SM, and a late one would overwrite the next forward's table).
          if (c->planner_delay_us > 0) std::this_thread::sleep_for(std::chrono::microseconds(c->planner_delay_us));
          const unsigned long long word = ((unsigned long long)(uint32_t)c->job_flag_seq << 32) | (uint32_t)n;
          for (int i = 0; i < n; ++i) {
            const feplb_group& gr = c->h_dyn_groups[i];
            volatile int32_t* t = c->h_dyn_tab32 + 8 * i;
            t[0] = gr.expert; t[1] = gr.row_start; t[2] = gr.rows; t[3] = gr.exec_rank;
            t[4] = gr.is_dynamic; t[5] = c->job_flag_seq; t[6] = 0; t[7] = 0;
          }
          std::atomic_thread_fence(std::memory_order_release);
          *(volatile unsigned long long*)c->h_dyn_ready = word;
          c->tl.host_upload_enqueued_us = us_since(c->t0);
        } else {
          if (n) e = feplb_launch_upload_groups(c->h_dyn_groups_dev, c->d_dyn_groups, n, c->copy_stream);
          if (e == cudaSuccess) e = cudaEventRecord(c->ev_plan, c->copy_stream);
          c->tl.host_upload_enqueued_us = us_since(c->t0);
        }
        if (e != cudaSuccess) rc = FEPLB_E_CUDA;
      }
    }
    if (rc != FEPLB_OK && c->job_wm && c->job_flag_seq) {
      // the launches of this forward must not wait for a table that will not come: an empty one
      std::atomic_thread_fence(std::memory_order_release);
      *(volatile unsigned long long*)c->h_dyn_ready = (unsigned long long)(uint32_t)c->job_flag_seq << 32;
    }
    {
      std::lock_guard<std::mutex> lk(c->mu);
      c->job_rc = rc;
      c->job = JOB_DONE;
    }
    c->cv.notify_all();
  }
}

int check_dev_ptrs(feplb_ctx* c, std::initializer_list<const void*> ptrs) {
  for (const void* p : ptrs)
    if (!p || !aligned16(p)) return fail(c, FEPLB_E_INVALID, "null or unaligned device pointer");
  return FEPLB_OK;
}

}  // namespace

extern "C" int feplb_version(void) { return 100; }

extern "C" const char* feplb_strerror(int s) {
  switch (s) {
    case FEPLB_OK: return "ok";
    case FEPLB_E_INVALID: return "invalid argument";
    case FEPLB_E_RANGE: return "expert id out of range";
    case FEPLB_E_CUDA: return "CUDA error";
    case FEPLB_E_NOMEM: return "out of memory or capacity too small";
    case FEPLB_E_TIMEOUT: return "timed out";
    case FEPLB_E_STATE: return "invalid call order";
    case FEPLB_E_DEVICE: return "device-side check failed";
    default: return "unknown status";
  }
}

extern "C" int feplb_create(const feplb_config* cfg, feplb_ctx** out) {
  if (!out) return FEPLB_E_INVALID;
  *out = nullptr;
  int rc = feplb_validate_config(cfg);
  if (rc != FEPLB_OK) return rc;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FEPLB_E_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return FEPLB_E_CUDA;
  if (prop.major != 10) return FEPLB_E_CUDA;   // sm_100a code only
  feplb_ctx* c = new (std::nothrow) feplb_ctx();
  if (!c) return FEPLB_E_NOMEM;
  c->cfg = *cfg;
  c->device = dev;
  c->num_sms = prop.multiProcessorCount;
  c->s_cap = feplb_s_pad(cfg);
  // 256-row pair tiles pay off when an expert's segment is several tiles long on average
  c->gemm_pair_auto = c->gemm_pair_default = (int64_t)cfg->T * cfg->K >= (int64_t)2048 * cfg->E;
  // a merged launch runs static and dynamic groups in one form: the two-CTA form from 256 rows per expert
  c->merged_pair = (int64_t)cfg->T * cfg->K >= (int64_t)256 * cfg->E;
  // backward GEMMs: the pair form pays once an expert's segment spans several 256-row tiles
  // (measured: -7.5 % backward time at 1024 rows per expert, slower at 384)
  c->bwd_pair_auto = c->bwd_pair = (int64_t)cfg->T * cfg->K >= (int64_t)512 * cfg->E ? 3 : 0;
  const int64_t S = (int64_t)cfg->T * cfg->K;
  c->nb = (int)((S + FEPLB_SLOTS_PER_BLOCK - 1) / FEPLB_SLOTS_PER_BLOCK);
  const int cap_moves = cfg->R * cfg->max_num_dyn;
  const int cap_groups = cfg->E + cap_moves;
  // Weights-on-M form: pays while groups are a few hundred rows (less padding, an expert's weights cross
  // the L2 port once per 256 rows); from ~1000 rows per expert the two-CTA form keeps its lead because
  // it can overlap every tile's epilogue with the next tile's MMAs.
  c->wm_ok = feplb_wm_supported(cfg->E, cfg->d, cfg->f, cfg->E + cap_groups);
  c->wm_auto = c->wm = false;      // measured a few percent behind the tokens-on-M forms at every benchmarked size: on request only
  // One launch per pass over the static and then the dynamic groups (the table of the latter is
  // picked up on the device): saves two launch ramps and two partly filled last waves per forward,
  // which matters while a forward's GEMMs take a few hundred microseconds; one form serves both
  // tables then, so it stays off where the dynamic groups want the two-CTA form and the static ones
  // do not (from ~1000 rows per expert).
  c->merged_ok = cfg->E + cap_groups <= FEPLB_MAX_GROUPS;
  c->merged_auto = c->merged = c->merged_ok && S < (int64_t)FEPLB_WM_AUTO_ROWS_PER_EXPERT * cfg->E;
  bool ok = true;
  ok = ok && cudaMalloc(&c->d_dyn_ready, 2 * sizeof(unsigned long long)) == cudaSuccess &&     // [0] ready word, [1] claim word
       cudaMemset(c->d_dyn_ready, 0, 2 * sizeof(unsigned long long)) == cudaSuccess;
  ok = ok && cudaHostAlloc(&c->h_dyn_ready, sizeof(unsigned long long), cudaHostAllocMapped) == cudaSuccess &&
       cudaHostGetDevicePointer(&c->h_dyn_ready_dev, c->h_dyn_ready, 0) == cudaSuccess;
  if (ok) *c->h_dyn_ready = 0;
  ok = ok && cudaHostAlloc(&c->h_dyn_tab32, 32 * (size_t)(cap_groups > 0 ? cap_groups : 1), cudaHostAllocMapped) == cudaSuccess &&
       cudaHostGetDevicePointer(&c->h_dyn_tab32_dev, c->h_dyn_tab32, 0) == cudaSuccess;
  if (ok) memset(c->h_dyn_tab32, 0, 32 * (size_t)(cap_groups > 0 ? cap_groups : 1));
  ok = ok && cudaMalloc(&c->d_dyn_tab32, 32 * (size_t)(cap_groups > 0 ? cap_groups : 1)) == cudaSuccess &&
       cudaMemset(c->d_dyn_tab32, 0, 32 * (size_t)(cap_groups > 0 ? cap_groups : 1)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_stamps, sizeof(unsigned long long) * kEvRing * kStampWords) == cudaSuccess;
  ok = ok && cudaMallocHost(&c->h_stamps, sizeof(unsigned long long) * kEvRing * kStampWords) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_block_hist, sizeof(int32_t) * (size_t)(c->nb > 0 ? c->nb : 1) * cfg->E) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_pad_off, sizeof(int32_t) * (cfg->E + 1)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_status, sizeof(uint32_t)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_home_groups, sizeof(feplb_group) * cfg->E) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_dyn_groups, (sizeof(feplb_group) * cap_groups + 15) / 16 * 16) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_mask, cfg->E) == cudaSuccess;
  if (cfg->phase2_copy && (int64_t)cfg->R * cfg->max_num_dyn > 30000) ok = false;   // slot ids travel in 15 bits
  if (ok && cfg->phase2_copy) {
    c->n_recv_slots = cfg->R * cfg->max_num_dyn;
    const size_t per = (size_t)cfg->d * cfg->f * 2, n = (size_t)(c->n_recv_slots > 0 ? c->n_recv_slots : 1);
    ok = ok && cudaMalloc(&c->d_recv_w1, per * n) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_recv_w3, per * n) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_recv_w2, per * n) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_recv_x, (size_t)(c->s_cap > 0 ? c->s_cap : 1) * cfg->d * 2) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_gather, cudaEventDisableTiming) == cudaSuccess;
  }
  ok = ok && cudaMallocHost(&c->h_counts, sizeof(int32_t) * cfg->E) == cudaSuccess;
  ok = ok && cudaHostAlloc(&c->h_dyn_groups, (sizeof(feplb_group) * cap_groups + 15) / 16 * 16, cudaHostAllocMapped) == cudaSuccess &&
       cudaHostGetDevicePointer(&c->h_dyn_groups_dev, c->h_dyn_groups, 0) == cudaSuccess;
  ok = ok && cudaMallocHost(&c->h_status, sizeof(uint32_t)) == cudaSuccess;
  ok = ok && cudaMallocHost(&c->h_mask, cfg->E) == cudaSuccess;
  ok = ok && cudaMallocHost(&c->h_counts_tagged, sizeof(unsigned long long) * (cfg->E > 0 ? cfg->E : 1)) == cudaSuccess;
  if (ok) memset(c->h_counts_tagged, 0, sizeof(unsigned long long) * cfg->E);
  ok = ok && cudaMemset(c->d_status, 0, sizeof(uint32_t)) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&c->in_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking) == cudaSuccess;
  for (int i = 0; ok && i < FEPLB_HOST_SLOTS; ++i)
    ok = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreate(&c->ev_counts) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->ev_plan, cudaEventDisableTiming) == cudaSuccess;
  for (int r = 0; ok && r < kEvRing; ++r)
    for (int i = 0; ok && i < EV_N; ++i) ok = cudaEventCreate(&c->evr[r][i]) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    feplb_destroy(c);
    return FEPLB_E_NOMEM;
  }
  c->moves.resize(cap_moves > 0 ? cap_moves : 1);
  c->groups.resize(cap_groups);
  c->load_before.resize(cfg->R);
  c->load_after.resize(cfg->R);
  c->mask.resize(cfg->E);
  c->plan = feplb_plan_out{0, 0, cap_moves, cap_groups, c->moves.data(), c->groups.data(),
                           c->load_before.data(), c->load_after.data()};
  memset(&c->tl, 0, sizeof(c->tl));
  memset(&c->tl_sum, 0, sizeof(c->tl_sum));
  memset(&c->tl_last, 0, sizeof(c->tl_last));
  c->th = std::thread(planner_main, c);
  *out = c;
  return FEPLB_OK;
}

extern "C" int feplb_destroy(feplb_ctx* c) {
  if (!c) return FEPLB_OK;
  if (c->th.joinable()) {
    {
      std::lock_guard<std::mutex> lk(c->mu);
      c->quit = true;
    }
    c->cv.notify_all();
    c->th.join();
  }
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  cudaFree(c->d_block_hist);
  cudaFree(c->d_pad_off);
  cudaFree(c->d_status);
  cudaFree(c->d_home_groups);
  cudaFree(c->d_dyn_groups);
  cudaFree(c->d_mask);
  cudaFree(c->d_recv_w1);
  cudaFree(c->d_recv_w3);
  cudaFree(c->d_recv_w2);
  cudaFree(c->d_recv_x);
  if (c->ev_gather) cudaEventDestroy(c->ev_gather);
  cudaFree(c->d_dyn_ready);
  cudaFree(c->d_dyn_tab32);
  cudaFreeHost(c->h_dyn_tab32);
  cudaFree(c->d_stamps);
  cudaFreeHost(c->h_dyn_ready);
  cudaFreeHost(c->h_stamps);
  cudaFreeHost(c->h_counts);
  cudaFreeHost(c->h_dyn_groups);
  cudaFreeHost(c->h_status);
  cudaFreeHost(c->h_mask);
  cudaFreeHost(c->h_counts_tagged);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->in_stream) cudaStreamDestroy(c->in_stream);
  if (c->out_stream) cudaStreamDestroy(c->out_stream);
  for (int i = 0; i < FEPLB_HOST_SLOTS; ++i) {
    if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
    if (c->ev_done[i]) cudaEventDestroy(c->ev_done[i]);
    if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
  }
  if (c->ev_counts) cudaEventDestroy(c->ev_counts);
  if (c->ev_plan) cudaEventDestroy(c->ev_plan);
  for (int r = 0; r < kEvRing; ++r)
    for (int i = 0; i < EV_N; ++i)
      if (c->evr[r][i]) cudaEventDestroy(c->evr[r][i]);
  cudaGetLastError();
  delete c;
  return FEPLB_OK;
}

extern "C" const char* feplb_last_error(const feplb_ctx* c) { return c ? c->err : ""; }

extern "C" int64_t feplb_launch_count(const feplb_ctx* c) { return c ? c->launches : 0; }

extern "C" int feplb_check_status(feplb_ctx* c, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  CUDA_TRY(c, cudaMemcpyAsync(c->h_status, c->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(c, cudaMemsetAsync(c->d_status, 0, sizeof(uint32_t), st));
  CUDA_TRY(c, cudaStreamSynchronize(st));
  const uint32_t s = *c->h_status;
  if (s & FEPLB_ST_WAIT) return fail(c, FEPLB_E_DEVICE, "a bounded device-side wait gave up (status 0x%x)", s);
  if (s & FEPLB_ST_PLAN)
    return fail(c, FEPLB_E_TIMEOUT, "the expert GEMM gave up waiting for the planner's dynamic group table (status 0x%x)", s);
  if (s & FEPLB_ST_GROUP) return fail(c, FEPLB_E_DEVICE, "malformed group entry (status 0x%x)", s);
  if (s & FEPLB_ST_COUNTS) return fail(c, FEPLB_E_DEVICE, "counts disagree with topk_ids (status 0x%x)", s);
  if (s & FEPLB_ST_RANGE) return fail(c, FEPLB_E_RANGE, "expert id outside [0, E) (status 0x%x)", s);
  return FEPLB_OK;
}

extern "C" int feplb_route_hist(feplb_ctx* c, const int32_t* topk_ids, int32_t* counts, int32_t* rank_load, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (!counts || !rank_load || (!topk_ids && c->cfg.T > 0)) return fail(c, FEPLB_E_INVALID, "route_hist: null pointer");
  const int64_t S = (int64_t)c->cfg.T * c->cfg.K;
  CUDA_TRY(c, feplb_launch_block_hist(topk_ids, S, c->cfg.E, c->cfg.R, c->d_block_hist, counts, rank_load,
                                      c->d_status, (cudaStream_t)stream, &c->launches));
  return FEPLB_OK;
}

static int dispatch_impl(feplb_ctx* c, const void* x, const int32_t* topk_ids, const int32_t* counts, void* x_perm,
                         int32_t* slot_to_row, int32_t* row_to_token, cudaStream_t st) {
  const feplb_config& g = c->cfg;
  const int64_t S = (int64_t)g.T * g.K;
  if (!counts || !row_to_token) return fail(c, FEPLB_E_INVALID, "dispatch: null pointer");
  if (g.T > 0) {
    int rc = check_dev_ptrs(c, {x, x_perm});
    if (rc != FEPLB_OK) return rc;
    if (!topk_ids || !slot_to_row) return fail(c, FEPLB_E_INVALID, "dispatch: null pointer");
  }
  CUDA_TRY(c, feplb_launch_permute(topk_ids, S, g.K, g.E, g.row_align, counts, c->d_block_hist, c->d_pad_off,
                                   slot_to_row, row_to_token, (int64_t)c->s_cap, c->d_status, st, &c->launches));
  CUDA_TRY(c, feplb_launch_gather(x, topk_ids, c->d_block_hist, slot_to_row, counts, c->d_pad_off, x_perm, g.T, g.K, g.E,
                                  g.d, g.row_align, (int64_t)c->s_cap, c->num_sms, st, &c->launches, row_to_token, true));
  return FEPLB_OK;
}

extern "C" int feplb_dispatch(feplb_ctx* c, const void* x, const int32_t* topk_ids, const int32_t* counts,
                              void* x_perm, int32_t* slot_to_row, int32_t* row_to_token, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  return dispatch_impl(c, x, topk_ids, counts, x_perm, slot_to_row, row_to_token, (cudaStream_t)stream);
}

extern "C" int feplb_home_groups(feplb_ctx* c, const int32_t* counts, const uint8_t* dyn_mask,
                                 feplb_group* groups_out, uint8_t* dyn_mask_out, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (!counts || !groups_out) return fail(c, FEPLB_E_INVALID, "home_groups: null pointer");
  if (!dyn_mask && c->cfg.mask_policy != FEPLB_MASK_REACTIVE)
    return fail(c, FEPLB_E_INVALID, "home_groups: dyn_mask is required unless mask_policy is REACTIVE");
  CUDA_TRY(c, feplb_launch_home_groups(counts, dyn_mask, c->cfg.E, c->cfg.R, c->cfg.row_align, c->cfg.dyn,
                                       groups_out, dyn_mask_out, (cudaStream_t)stream, &c->launches));
  return FEPLB_OK;
}

// `dyn` != nullptr: weights-on-M launches that go on to the planner's dynamic table after `groups`.
static int ffn_impl(feplb_ctx* c, const void* x_perm, const void* w1, const void* w3, const void* w2,
                    const feplb_group* groups, int32_t n_groups, int32_t which, void* h, void* y, cudaStream_t st,
                    int pair = -1, const feplb_wm_dyn* dyn = nullptr) {
  if (pair < 0) pair = c->gemm_pair_default;
  if (n_groups < 0 || n_groups > FEPLB_MAX_GROUPS) return fail(c, FEPLB_E_INVALID, "expert_ffn: n_groups out of range");
  if (which != FEPLB_FFN_ALL && which != FEPLB_FFN_STATIC && which != FEPLB_FFN_DYNAMIC)
    return fail(c, FEPLB_E_INVALID, "expert_ffn: bad selector");
  if ((n_groups == 0 && !dyn) || c->s_cap == 0) return FEPLB_OK;
  int rc = check_dev_ptrs(c, {x_perm, w1, w3, w2, h, y});
  if (rc != FEPLB_OK) return rc;
  if (!groups) return fail(c, FEPLB_E_INVALID, "expert_ffn: null group table");
  feplb_gemm_args a;
  a.x_perm = x_perm; a.w1 = w1; a.w3 = w3; a.w2 = w2; a.h = h; a.y = y;
  a.groups = groups; a.n_groups = n_groups; a.which = which;
  a.E = c->cfg.E; a.d = c->cfg.d; a.f = c->cfg.f; a.s_cap = (int64_t)c->s_cap;
  a.status = c->d_status; a.num_sms = c->num_sms; a.pair = pair;
  a.ab_out = c->d_preact;
  a.recv_w1 = c->d_recv_w1; a.recv_w3 = c->d_recv_w3; a.recv_w2 = c->d_recv_w2; a.n_recv_slots = c->n_recv_slots;
  a.recv_x = c->d_recv_x;
  if (c->wm && n_groups + (dyn ? dyn->max_groups : 0) <= FEPLB_WM_MAX_ENTRIES) {
    const feplb_wm_dyn none;
    return feplb_launch_expert_ffn_wm(a, dyn ? *dyn : none, st, &c->launches, c->err, sizeof(c->err));
  }
  return feplb_launch_expert_ffn(a, st, &c->launches, c->err, sizeof(c->err), dyn);
}

extern "C" int feplb_expert_ffn(feplb_ctx* c, const void* x_perm, const void* w1, const void* w3, const void* w2,
                                const feplb_group* groups, int32_t n_groups, int32_t which,
                                void* h_scratch, void* y_perm, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  return ffn_impl(c, x_perm, w1, w3, w2, groups, n_groups, which, h_scratch, y_perm, (cudaStream_t)stream);
}

extern "C" int feplb_combine(feplb_ctx* c, const void* y_perm, const int32_t* slot_to_row, const float* gates,
                             void* out, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (c->cfg.T == 0) return FEPLB_OK;
  int rc = check_dev_ptrs(c, {y_perm, out});
  if (rc != FEPLB_OK) return rc;
  if (!slot_to_row || !gates) return fail(c, FEPLB_E_INVALID, "combine: null pointer");
  CUDA_TRY(c, feplb_launch_combine(y_perm, slot_to_row, gates, out, c->cfg.T, c->cfg.K, c->cfg.d, c->num_sms,
                                   (cudaStream_t)stream, &c->launches));
  return FEPLB_OK;
}

extern "C" int feplb_plan_async(feplb_ctx* c, const int32_t* counts, const uint8_t* dyn_mask_host, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (!counts) return fail(c, FEPLB_E_INVALID, "plan_async: null counts");
  if (!dyn_mask_host && c->cfg.mask_policy != FEPLB_MASK_REACTIVE)
    return fail(c, FEPLB_E_INVALID, "plan_async: dyn_mask_host is required unless mask_policy is REACTIVE");
  {
    std::lock_guard<std::mutex> lk(c->mu);
    if (c->job != JOB_IDLE) return fail(c, FEPLB_E_STATE, "plan_async: a plan is already pending");
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (!c->timeline_valid) c->t0 = clk::now();
  CUDA_TRY(c, cudaMemcpyAsync(c->h_counts, counts, sizeof(int32_t) * c->cfg.E, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(c, cudaEventRecord(c->ev_counts, st));
  {
    std::lock_guard<std::mutex> lk(c->mu);
    c->job_mask = dyn_mask_host;
    c->job_flag_seq = 0;
    c->job_wm = false;
    c->job = JOB_PENDING;
  }
  c->cv.notify_all();
  return FEPLB_OK;
}

// Whole-layer path: the counts of this forward arrive in h_counts with sequence number `seq`.
static int plan_kick_flag(feplb_ctx* c, const uint8_t* dyn_mask_host, int32_t seq, bool wm) {
  {
    std::lock_guard<std::mutex> lk(c->mu);
    if (c->job != JOB_IDLE) return fail(c, FEPLB_E_STATE, "moe_forward: a plan is already pending");
    c->job_mask = dyn_mask_host;
    c->job_wm = wm;
    c->job_flag_seq = seq;
    c->job = JOB_PENDING;
  }
  c->cv.notify_all();
  return FEPLB_OK;
}

// Waits for the planner's job and returns the context to idle; copies the plan out.
static int join_planner(feplb_ctx* c, int32_t timeout_ms, feplb_plan_out* plan_copy) {
  int rc;
  {
    std::unique_lock<std::mutex> lk(c->mu);
    if (c->job == JOB_IDLE) return fail(c, FEPLB_E_STATE, "plan_wait: no plan was requested");
    if (!c->cv.wait_for(lk, std::chrono::milliseconds(timeout_ms < 0 ? 0 : timeout_ms), [&] { return c->job == JOB_DONE; }))
      return fail(c, FEPLB_E_TIMEOUT, "plan_wait: planner did not finish within %d ms", timeout_ms);
    rc = c->job_rc;
    c->job = JOB_IDLE;
  }
  if (rc != FEPLB_OK) return fail(c, rc, "planner failed: %s", feplb_strerror(rc));
  if (plan_copy) {
    if (plan_copy->cap_moves < c->plan.n_moves || plan_copy->cap_groups < c->plan.n_groups ||
        !plan_copy->load_before || !plan_copy->load_after)
      return fail(c, FEPLB_E_NOMEM, "plan_wait: plan_copy too small");
    plan_copy->n_moves = c->plan.n_moves;
    plan_copy->n_groups = c->plan.n_groups;
    if (c->plan.n_moves) memcpy(plan_copy->moves, c->plan.moves, sizeof(feplb_move) * c->plan.n_moves);
    if (c->plan.n_groups) memcpy(plan_copy->groups, c->plan.groups, sizeof(feplb_group) * c->plan.n_groups);
    memcpy(plan_copy->load_before, c->plan.load_before, sizeof(int64_t) * c->cfg.R);
    memcpy(plan_copy->load_after, c->plan.load_after, sizeof(int64_t) * c->cfg.R);
  }
  if (c->n_dyn_groups > 0 && !c->job_wm) ++c->launches;     // the planner thread's table upload kernel
  return FEPLB_OK;
}

extern "C" int feplb_plan_wait(feplb_ctx* c, int32_t timeout_ms, feplb_plan_out* plan_copy,
                               const feplb_group** dyn_groups_dev, int32_t* n_dyn_groups, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  int rc = join_planner(c, timeout_ms, plan_copy);
  if (rc != FEPLB_OK) return rc;
  if (dyn_groups_dev) *dyn_groups_dev = c->d_dyn_groups;
  if (n_dyn_groups) *n_dyn_groups = c->n_dyn_groups;
  CUDA_TRY(c, cudaStreamWaitEvent((cudaStream_t)stream, c->ev_plan, 0));
  return FEPLB_OK;
}

// Reads the stage events of ring slot r (waiting for them if needed) and adds them to the totals.
static int harvest_slot(feplb_ctx* c, int r) {
  if (!c->ev_used[r]) return FEPLB_OK;
  cudaEvent_t* ev = c->evr[r];
  CUDA_TRY(c, cudaEventSynchronize(ev[EV_COMBINE]));
  if (c->ev_host[r].ffn_launches == 2) CUDA_TRY(c, cudaEventSynchronize(ev[EV_STAMPS]));
  float ms = 0;
  auto el = [&](cudaEvent_t a, cudaEvent_t b) { return cudaEventElapsedTime(&ms, a, b) == cudaSuccess ? ms * 1e3 : 0.0; };
  feplb_timeline t = c->ev_host[r];
  t.dev_hist_us = el(ev[EV_T0], ev[EV_HIST]);
  t.dev_dispatch_us = el(ev[EV_HIST], ev[EV_DISPATCH]);
  const bool merged = t.ffn_launches == 2;
  t.dev_static_ffn_us = el(ev[EV_STATIC0], ev[EV_STATIC1]);
  t.dev_dynamic_ffn_us = merged ? 0.0 : el(ev[EV_DYN0], ev[EV_DYN1]);
  t.dev_combine_us = el(ev[merged ? EV_STATIC1 : EV_DYN1], ev[EV_COMBINE]);
  t.dev_counts_to_static_start_us = el(ev[EV_COUNTS], ev[EV_STATIC0]);
  t.dev_counts_to_static_end_us = el(ev[EV_COUNTS], ev[EV_STATIC1]);
  t.dev_total_us = el(ev[EV_T0], ev[EV_COMBINE]);
  t.dev_counts_to_copies_done_us = t.phase2_copy_bytes > 0 ? el(ev[EV_COUNTS], ev[EV_COPIES]) : 0.0;
  if (t.ffn_launches == 2) {
    // weights-on-M form: marks taken inside the kernels (all ones = never written)
    const unsigned long long* sp = c->h_stamps + (size_t)r * kStampWords;
    const unsigned long long none = ~0ull;
    auto span = [&](unsigned long long a, unsigned long long b) { return a != none && b != none && b >= a ? (b - a) * 1e-3 : 0.0; };
    const unsigned long long t_counts = sp[8], p1_start = sp[0], p1_first_dyn = sp[1], p1_end = sp[2] == none ? none : ~sp[2];
    const unsigned long long p2_start = sp[4], p2_end = sp[6] == none ? none : ~sp[6];
    t.dev_ffn_pass1_us = span(p1_start, p1_end);
    t.dev_ffn_pass2_us = span(p2_start, p2_end);
    t.dev_counts_to_static_start_us = span(t_counts, p1_start);
    t.dev_counts_to_static_end_us = span(t_counts, p1_first_dyn != none ? p1_first_dyn : p1_end);
    const unsigned long long w1 = sp[3] == none ? 0 : ~sp[3], w2 = sp[7] == none ? 0 : ~sp[7];
    t.dev_plan_wait_us = (w1 > w2 ? w1 : w2) * 1e-3;
  }
  cudaGetLastError();
  const double* src = reinterpret_cast<const double*>(&t);
  double* dst = reinterpret_cast<double*>(&c->tl_sum);
  for (size_t i = 0; i < sizeof(feplb_timeline) / sizeof(double); ++i) dst[i] += src[i];
  c->tl_last = t;
  c->tl_n += 1;
  c->ev_used[r] = false;
  return FEPLB_OK;
}

extern "C" int feplb_set_timeline(feplb_ctx* c, int32_t enable) {
  if (!c) return FEPLB_E_INVALID;
  c->timeline_on = enable != 0;
  return FEPLB_OK;
}

#define TL_EVENT(i)                                                  \
  do {                                                               \
    if (c->timeline_on) CUDA_TRY(c, cudaEventRecord(c->ev[i], st));  \
  } while (0)

extern "C" int feplb_moe_forward(feplb_ctx* c, const void* x, const int32_t* topk_ids, const float* gates,
                                 const void* w1, const void* w3, const void* w2, const uint8_t* dyn_mask_host,
                                 int32_t* counts, int32_t* rank_load, void* x_perm, void* h_scratch, void* y_perm,
                                 int32_t* slot_to_row, int32_t* row_to_token, void* out,
                                 feplb_plan_out* plan_copy, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  const feplb_config& g = c->cfg;
  if (!dyn_mask_host && g.mask_policy != FEPLB_MASK_REACTIVE)
    return fail(c, FEPLB_E_INVALID, "moe_forward: dyn_mask_host is required unless mask_policy is REACTIVE");
  int rc;
  if (c->timeline_on) {
    c->ev_slot = (c->ev_slot + 1) % kEvRing;
    if ((rc = harvest_slot(c, c->ev_slot)) != FEPLB_OK) return rc;   // long finished unless the ring wrapped quickly
    c->ev = c->evr[c->ev_slot];
  }
  c->t0 = clk::now();
  c->timeline_valid = true;
  c->tl.phase2_copy_bytes = 0;
  c->tl.dev_counts_to_copies_done_us = 0;
  // Weights-on-M form: one launch per pass runs the static groups and then the dynamic ones, whose
  // table it picks up on the device, so everything is enqueued before the planner is joined.
  // Not with Phase-2 weight copies: the dynamic groups would then wait, inside a kernel that holds
  // every SM, for device-to-device copies that the driver may carry out with kernels of its own;
  // that case keeps the four-launch order (the dynamic launches follow the copies in stream order).
  const bool wm = c->merged && !g.phase2_copy;
  c->tl.ffn_launches = wm ? 2 : 4;
  c->tl.dev_ffn_pass1_us = c->tl.dev_ffn_pass2_us = c->tl.dev_plan_wait_us = 0;
  unsigned long long* stamps = nullptr;
  if (wm && c->timeline_on) {
    stamps = c->d_stamps + (size_t)c->ev_slot * kStampWords;
    CUDA_TRY(c, cudaMemsetAsync(stamps, 0xFF, sizeof(unsigned long long) * kStampWords, st));
  }
  TL_EVENT(EV_T0);
  // step 1: counts, rank loads, segment offsets and the home group table in two launches; the
  // planner thread starts as soon as the counts reach the host
  if (!counts || !rank_load || !row_to_token) return fail(c, FEPLB_E_INVALID, "moe_forward: null pointer");
  if (g.T > 0) {
    if ((rc = check_dev_ptrs(c, {x, x_perm})) != FEPLB_OK) return rc;
    if (!topk_ids || !slot_to_row) return fail(c, FEPLB_E_INVALID, "moe_forward: null pointer");
  }
  const int64_t S = (int64_t)g.T * g.K;
  const uint8_t* mask_dev = nullptr;
  if (dyn_mask_host) {
    memcpy(c->h_mask, dyn_mask_host, g.E);
    CUDA_TRY(c, cudaMemcpyAsync(c->d_mask, c->h_mask, g.E, cudaMemcpyHostToDevice, st));
    mask_dev = c->d_mask;
  }
  c->flag_seq = c->flag_seq == INT32_MAX ? 1 : c->flag_seq + 1;
  const int32_t seq = c->flag_seq;
  CUDA_TRY(c, feplb_launch_route_fused(topk_ids, S, g.E, g.R, g.row_align, g.dyn, mask_dev, c->d_block_hist, counts,
                                       rank_load, c->d_pad_off, c->d_home_groups, nullptr, slot_to_row, row_to_token,
                                       (int64_t)c->s_cap, c->d_status, c->h_counts_tagged, seq,
                                       stamps ? stamps + 8 : nullptr, st, &c->launches));
  c->job_w1 = w1; c->job_w3 = w3; c->job_w2 = w2;   // read by the planner thread after it is woken
  c->job_x_perm = x_perm;
  if ((rc = plan_kick_flag(c, dyn_mask_host, seq, wm)) != FEPLB_OK) return rc;
  TL_EVENT(EV_COUNTS);
  TL_EVENT(EV_HIST);
  // step 3: permutation (does not depend on the plan: a migration relabels rows, it does not move
  // them here).  From here on a failure must still join the planner, so errors are carried in rc.
  {
    cudaError_t e = feplb_launch_gather(x, topk_ids, c->d_block_hist, slot_to_row, counts, c->d_pad_off, x_perm, g.T, g.K,
                                        g.E, g.d, g.row_align, (int64_t)c->s_cap, c->num_sms, st, &c->launches,
                                        row_to_token, true);
    if (e == cudaSuccess && g.phase2_copy) {
      // the planner's row copies of Phase 2 wait for the permuted rows
      e = cudaEventRecord(c->ev_gather, st);
      c->gather_seq.store(seq, std::memory_order_release);
    }
    if (e != cudaSuccess) rc = fail(c, FEPLB_E_CUDA, "dispatch launch: %s", cudaGetErrorString(e));
  }
  TL_EVENT(EV_DISPATCH);
  TL_EVENT(EV_STATIC0);
  if (wm) {
    // steps 4 + 5 in two launches: static groups from the table built on the device, then the dynamic
    // groups as soon as the planner has published them (bounded wait inside the kernel)
    feplb_wm_dyn dyn;
    dyn.table_dev = c->d_dyn_tab32; dyn.table_host = c->h_dyn_tab32_dev;
    dyn.ready_dev = c->d_dyn_ready; dyn.ready_host = c->h_dyn_ready_dev;
    dyn.claim = reinterpret_cast<uint32_t*>(c->d_dyn_ready + 1);
    dyn.seq = (uint32_t)seq; dyn.max_groups = c->plan.cap_groups; dyn.stamps = stamps;
    dyn.wait_limit_ns = 1000ull * (unsigned long long)c->device_wait_limit_us;
    if (rc == FEPLB_OK)
      rc = ffn_impl(c, x_perm, w1, w3, w2, c->d_home_groups, g.E, FEPLB_FFN_STATIC, h_scratch, y_perm, st,
                    c->gemm_pair_forced >= 0 ? c->gemm_pair_forced : (int)c->merged_pair, &dyn);
    TL_EVENT(EV_STATIC1);          // both launches lie between EV_STATIC0 and here; no events of their own for the dynamic part
    c->tl.host_enqueue_static_done_us = us_since(c->t0);
    int rc_comb = rc == FEPLB_OK ? feplb_combine(c, y_perm, slot_to_row, gates, out, stream) : FEPLB_OK;
    if (c->timeline_on && rc == FEPLB_OK && rc_comb == FEPLB_OK) {
      cudaError_t e = cudaEventRecord(c->ev[EV_COMBINE], st);
      if (e == cudaSuccess && stamps)      // the kernels' own marks follow the last stage event to the host
        e = cudaMemcpyAsync(c->h_stamps + (size_t)c->ev_slot * kStampWords, stamps, sizeof(unsigned long long) * kStampWords,
                            cudaMemcpyDeviceToHost, st);
      if (e == cudaSuccess) e = cudaEventRecord(c->ev[EV_STAMPS], st);
      if (e != cudaSuccess) rc_comb = fail(c, FEPLB_E_CUDA, "timeline records: %s", cudaGetErrorString(e));
    }
    // join the planner (always, so that the context returns to idle): everything is already enqueued
    int rc_join = join_planner(c, c->planner_timeout_ms + 500, plan_copy);
    c->tl.host_join_us = us_since(c->t0);
    if (rc != FEPLB_OK) return rc;
    if (rc_comb != FEPLB_OK) return rc_comb;
    if (rc_join != FEPLB_OK) return rc_join;
  } else {
    // step 4: static experts on their home ranks, from the group table built on the device
    if (rc == FEPLB_OK)
      rc = ffn_impl(c, x_perm, w1, w3, w2, c->d_home_groups, g.E, FEPLB_FFN_STATIC, h_scratch, y_perm, st);
    TL_EVENT(EV_STATIC1);
    c->tl.host_enqueue_static_done_us = us_since(c->t0);
    // join the planner (always, so that the context returns to idle), then step 5
    const feplb_group* dyn_groups = nullptr;
    int32_t n_dyn = 0;
    int rc_join = feplb_plan_wait(c, c->planner_timeout_ms + 500, plan_copy, &dyn_groups, &n_dyn, stream);
    c->tl.host_join_us = us_since(c->t0);
    if (rc != FEPLB_OK) return rc;
    if (rc_join != FEPLB_OK) return rc_join;
    TL_EVENT(EV_DYN0);
    if ((rc = ffn_impl(c, x_perm, w1, w3, w2, dyn_groups, n_dyn, FEPLB_FFN_ALL, h_scratch, y_perm, st, c->dyn_pair)) != FEPLB_OK) return rc;
    TL_EVENT(EV_DYN1);
    // step 6
    if ((rc = feplb_combine(c, y_perm, slot_to_row, gates, out, stream)) != FEPLB_OK) return rc;
    TL_EVENT(EV_COMBINE);
  }
  c->tl.host_return_us = us_since(c->t0);
  if (c->timeline_on) {
    c->ev_host[c->ev_slot] = c->tl;
    c->ev_used[c->ev_slot] = true;
  }
  return FEPLB_OK;
}

extern "C" int feplb_moe_forward_host(feplb_ctx* c, const void* x_host, const int32_t* topk_ids_host,
                                      const float* gates_host, void* x_dev, int32_t* ids_dev, float* gates_dev,
                                      const void* w1, const void* w3, const void* w2, const uint8_t* dyn_mask_host,
                                      int32_t* counts, int32_t* rank_load, void* x_perm, void* h_scratch, void* y_perm,
                                      int32_t* slot_to_row, int32_t* row_to_token, void* out_dev, void* out_host,
                                      feplb_plan_out* plan_copy, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  const feplb_config& g = c->cfg;
  const size_t nx = (size_t)g.T * g.d * 2, nk = (size_t)g.T * g.K * 4;
  if (g.T > 0) {
    if (!x_host || !topk_ids_host || !gates_host || !out_host || !x_dev || !ids_dev || !gates_dev || !out_dev)
      return fail(c, FEPLB_E_INVALID, "moe_forward_host: null pointer");
    CUDA_TRY(c, cudaMemcpyAsync(ids_dev, topk_ids_host, nk, cudaMemcpyHostToDevice, st));
    CUDA_TRY(c, cudaMemcpyAsync(gates_dev, gates_host, nk, cudaMemcpyHostToDevice, st));
    CUDA_TRY(c, cudaMemcpyAsync(x_dev, x_host, nx, cudaMemcpyHostToDevice, st));
  }
  int rc = feplb_moe_forward(c, x_dev, ids_dev, gates_dev, w1, w3, w2, dyn_mask_host, counts, rank_load, x_perm,
                             h_scratch, y_perm, slot_to_row, row_to_token, out_dev, plan_copy, stream);
  if (rc != FEPLB_OK) return rc;
  if (g.T > 0) CUDA_TRY(c, cudaMemcpyAsync(out_host, out_dev, nx, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(c, cudaStreamSynchronize(st));
  return FEPLB_OK;
}

extern "C" int feplb_host_stage_inputs(feplb_ctx* c, int32_t slot, const void* x_host, const int32_t* topk_ids_host,
                                       const float* gates_host, void* x_dev, int32_t* ids_dev, float* gates_dev) {
  if (!c) return FEPLB_E_INVALID;
  if (slot < 0 || slot >= FEPLB_HOST_SLOTS) return fail(c, FEPLB_E_INVALID, "host_stage_inputs: slot out of range");
  if (c->slot_staged[slot]) return fail(c, FEPLB_E_STATE, "host_stage_inputs: slot %d already holds staged inputs", slot);
  const feplb_config& g = c->cfg;
  const size_t nx = (size_t)g.T * g.d * 2, nk = (size_t)g.T * g.K * 4;
  if (g.T > 0 && (!x_host || !topk_ids_host || !gates_host || !x_dev || !ids_dev || !gates_dev))
    return fail(c, FEPLB_E_INVALID, "host_stage_inputs: null pointer");
  // the slot's device staging was last read by the forward that used this slot before
  if (c->slot_used[slot]) CUDA_TRY(c, cudaStreamWaitEvent(c->in_stream, c->ev_done[slot], 0));
  if (g.T > 0) {
    CUDA_TRY(c, cudaMemcpyAsync(ids_dev, topk_ids_host, nk, cudaMemcpyHostToDevice, c->in_stream));
    CUDA_TRY(c, cudaMemcpyAsync(gates_dev, gates_host, nk, cudaMemcpyHostToDevice, c->in_stream));
    CUDA_TRY(c, cudaMemcpyAsync(x_dev, x_host, nx, cudaMemcpyHostToDevice, c->in_stream));
  }
  CUDA_TRY(c, cudaEventRecord(c->ev_in[slot], c->in_stream));
  c->slot_staged[slot] = true;
  return FEPLB_OK;
}

extern "C" int feplb_moe_forward_host_async(feplb_ctx* c, int32_t slot, const void* x_host, const int32_t* topk_ids_host,
                                            const float* gates_host, void* x_dev, int32_t* ids_dev, float* gates_dev,
                                            const void* w1, const void* w3, const void* w2, const uint8_t* dyn_mask_host,
                                            int32_t* counts, int32_t* rank_load, void* x_perm, void* h_scratch,
                                            void* y_perm, int32_t* slot_to_row, int32_t* row_to_token, void* out_dev,
                                            void* out_host, feplb_plan_out* plan_copy, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (slot < 0 || slot >= FEPLB_HOST_SLOTS) return fail(c, FEPLB_E_INVALID, "moe_forward_host_async: slot out of range");
  cudaStream_t st = (cudaStream_t)stream;
  const feplb_config& g = c->cfg;
  const size_t nx = (size_t)g.T * g.d * 2;
  if (g.T > 0 && (!out_host || !x_dev || !ids_dev || !gates_dev || !out_dev))
    return fail(c, FEPLB_E_INVALID, "moe_forward_host_async: null pointer");
  if (c->slot_staged[slot]) {
    c->slot_staged[slot] = false;        // inputs were started by feplb_host_stage_inputs; ev_in[slot] marks their end
  } else {
    int rc = feplb_host_stage_inputs(c, slot, x_host, topk_ids_host, gates_host, x_dev, ids_dev, gates_dev);
    if (rc != FEPLB_OK) return rc;
    c->slot_staged[slot] = false;
  }
  // compute: after its inputs have arrived and the slot's previous result has left out_dev
  CUDA_TRY(c, cudaStreamWaitEvent(st, c->ev_in[slot], 0));
  if (c->slot_used[slot]) CUDA_TRY(c, cudaStreamWaitEvent(st, c->ev_out[slot], 0));
  int rc = feplb_moe_forward(c, x_dev, ids_dev, gates_dev, w1, w3, w2, dyn_mask_host, counts, rank_load, x_perm,
                             h_scratch, y_perm, slot_to_row, row_to_token, out_dev, plan_copy, stream);
  if (rc != FEPLB_OK) return rc;
  CUDA_TRY(c, cudaEventRecord(c->ev_done[slot], st));
  // output
  CUDA_TRY(c, cudaStreamWaitEvent(c->out_stream, c->ev_done[slot], 0));
  if (g.T > 0) CUDA_TRY(c, cudaMemcpyAsync(out_host, out_dev, nx, cudaMemcpyDeviceToHost, c->out_stream));
  CUDA_TRY(c, cudaEventRecord(c->ev_out[slot], c->out_stream));
  c->slot_used[slot] = true;
  return FEPLB_OK;
}

extern "C" int feplb_host_wait(feplb_ctx* c, int32_t slot) {
  if (!c) return FEPLB_E_INVALID;
  if (slot < 0 || slot >= FEPLB_HOST_SLOTS) return fail(c, FEPLB_E_INVALID, "host_wait: slot out of range");
  if (c->slot_used[slot]) CUDA_TRY(c, cudaEventSynchronize(c->ev_out[slot]));
  return FEPLB_OK;
}

extern "C" int feplb_get_timeline(feplb_ctx* c, feplb_timeline* out) {
  if (!c || !out) return FEPLB_E_INVALID;
  if (!c->timeline_valid) return fail(c, FEPLB_E_STATE, "get_timeline: no forward pass yet");
  if (c->timeline_on || c->tl_n) {
    for (int i = 1; i <= kEvRing; ++i) {   // oldest first, so that tl_last is the newest forward
      int rc = harvest_slot(c, (c->ev_slot + i) % kEvRing);
      if (rc != FEPLB_OK) return rc;
    }
    *out = c->tl_last;
  } else {
    *out = c->tl;   // host fields only
  }
  return FEPLB_OK;
}

extern "C" int feplb_timeline_totals(feplb_ctx* c, feplb_timeline* sum, int64_t* n_forwards, int32_t reset) {
  if (!c || !sum || !n_forwards) return FEPLB_E_INVALID;
  for (int i = 1; i <= kEvRing; ++i) {
    int rc = harvest_slot(c, (c->ev_slot + i) % kEvRing);
    if (rc != FEPLB_OK) return rc;
  }
  *sum = c->tl_sum;
  *n_forwards = c->tl_n;
  if (reset) {
    memset(&c->tl_sum, 0, sizeof(c->tl_sum));
    c->tl_n = 0;
  }
  return FEPLB_OK;
}

extern "C" int feplb_set_planner_timeout(feplb_ctx* c, int32_t timeout_ms) {
  if (!c || timeout_ms < 1) return FEPLB_E_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  if (c->job != JOB_IDLE) return fail(c, FEPLB_E_STATE, "set_planner_timeout: a plan is pending");
  c->planner_timeout_ms = timeout_ms;
  return FEPLB_OK;
}

extern "C" int feplb_set_gemm_form(feplb_ctx* c, int32_t forward_form, int32_t backward_pair) {
  if (!c) return FEPLB_E_INVALID;
  if (forward_form < FEPLB_FORM_AUTO || forward_form > FEPLB_FORM_WEIGHT_M)
    return fail(c, FEPLB_E_INVALID, "set_gemm_form: forward_form must be FEPLB_FORM_AUTO, _SINGLE, _PAIR or _WEIGHT_M");
  if (forward_form == FEPLB_FORM_WEIGHT_M && !c->wm_ok)
    return fail(c, FEPLB_E_INVALID, "set_gemm_form: the weights-on-M form needs f %% 128 == 0, d %% 256 == 0 and "
                                    "2*E + R*max_num_dyn <= %d", FEPLB_WM_MAX_ENTRIES);
  if (backward_pair < -1 || backward_pair > 3)
    return fail(c, FEPLB_E_INVALID, "set_gemm_form: backward_pair must be -1 (auto) or a 2-bit mask");
  std::lock_guard<std::mutex> lk(c->mu);
  if (c->job != JOB_IDLE) return fail(c, FEPLB_E_STATE, "set_gemm_form: a plan is pending");
  c->wm = forward_form == FEPLB_FORM_AUTO ? c->wm_auto : forward_form == FEPLB_FORM_WEIGHT_M;
  c->gemm_pair_forced = forward_form == FEPLB_FORM_SINGLE || forward_form == FEPLB_FORM_PAIR ? forward_form : -1;
  c->gemm_pair_default = c->gemm_pair_forced < 0 ? c->gemm_pair_auto : forward_form;
  c->bwd_pair = backward_pair < 0 ? c->bwd_pair_auto : backward_pair;
  return FEPLB_OK;
}

extern "C" int feplb_set_launch_merging(feplb_ctx* c, int32_t merged) {
  if (!c || merged < -1 || merged > 1) return FEPLB_E_INVALID;
  if (merged == 1 && !c->merged_ok)
    return fail(c, FEPLB_E_INVALID, "set_launch_merging: needs 2*E + R*max_num_dyn <= %d", FEPLB_MAX_GROUPS);
  std::lock_guard<std::mutex> lk(c->mu);
  if (c->job != JOB_IDLE) return fail(c, FEPLB_E_STATE, "set_launch_merging: a plan is pending");
  c->merged = merged < 0 ? c->merged_auto : merged != 0;
  return FEPLB_OK;
}

extern "C" int feplb_set_planner_timing(feplb_ctx* c, int32_t planner_delay_us, int32_t device_wait_limit_us) {
  if (!c || planner_delay_us < 0 || planner_delay_us > 1000000 || device_wait_limit_us < 0) return FEPLB_E_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  if (c->job != JOB_IDLE) return fail(c, FEPLB_E_STATE, "set_planner_timing: a plan is pending");
  c->planner_delay_us = planner_delay_us;
  c->device_wait_limit_us = device_wait_limit_us;
  return FEPLB_OK;
}

extern "C" int feplb_pack_weights(feplb_ctx* c, const void* w1_in, const void* w3_in, const void* w2_in, void* w1, void* w3,
                                  void* w2, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (!w1_in || !w3_in || !w2_in || !w1 || !w3 || !w2) return fail(c, FEPLB_E_INVALID, "pack_weights: null pointer");
  // [E,d,f] -> [E,f,d] and [E,f,d] -> [E,d,f]: the transposition of feplb_transpose_weights with d and f exchanged
  CUDA_TRY(c, feplb_launch_transpose_weights(w1_in, w3_in, w2_in, w1, w3, w2, c->cfg.E, c->cfg.f, c->cfg.d,
                                             (cudaStream_t)stream, &c->launches));
  return FEPLB_OK;
}

extern "C" int feplb_selftest_bounded_wait(feplb_ctx* c, int32_t limit_us, void* stream) {
  if (!c || limit_us < 1 || limit_us > 1000000) return FEPLB_E_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  int rc = feplb_check_status(c, stream);          // start from a clean status word
  if (rc != FEPLB_OK) return rc;
  int* d_flag = reinterpret_cast<int*>(c->d_pad_off);   // scratch word, rewritten by the next dispatch
  CUDA_TRY(c, cudaMemsetAsync(d_flag, 0xFF, sizeof(int), st));
  CUDA_TRY(c, feplb_launch_wait_selftest(c->d_status, 1000ull * limit_us, d_flag, st));
  ++c->launches;
  int gave_up = -1;
  CUDA_TRY(c, cudaMemcpyAsync(&gave_up, d_flag, sizeof(int), cudaMemcpyDeviceToHost, st));
  rc = feplb_check_status(c, stream);              // synchronises; expected: FEPLB_E_DEVICE from the wait
  if (rc == FEPLB_E_DEVICE && gave_up == 1) return FEPLB_OK;
  return fail(c, FEPLB_E_STATE, "bounded-wait self-test: status %d, gave_up %d", rc, gave_up);
}

extern "C" int feplb_route_topk(feplb_ctx* c, const float* logits, int32_t* topk_ids, float* gates, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (c->cfg.K > c->cfg.E) return fail(c, FEPLB_E_INVALID, "route_topk: K > E");
  if (c->cfg.T > 0 && (!logits || !topk_ids || !gates)) return fail(c, FEPLB_E_INVALID, "route_topk: null pointer");
  CUDA_TRY(c, feplb_launch_route_topk(logits, c->cfg.T, c->cfg.E, c->cfg.K, topk_ids, gates, c->num_sms,
                                      (cudaStream_t)stream, &c->launches));
  return FEPLB_OK;
}

// ---- backward pass ---------------------------------------------------------------------------

extern "C" int feplb_set_preact_buffer(feplb_ctx* c, void* ab) {
  if (!c) return FEPLB_E_INVALID;
  if (ab && !aligned16(ab)) return fail(c, FEPLB_E_INVALID, "set_preact_buffer: unaligned pointer");
  c->d_preact = ab;
  return FEPLB_OK;
}

extern "C" int feplb_transpose_weights(feplb_ctx* c, const void* w1, const void* w3, const void* w2, void* w1t, void* w3t,
                                       void* w2t, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (!w1 || !w3 || !w2 || !w1t || !w3t || !w2t) return fail(c, FEPLB_E_INVALID, "transpose_weights: null pointer");
  CUDA_TRY(c, feplb_launch_transpose_weights(w1, w3, w2, w1t, w3t, w2t, c->cfg.E, c->cfg.d, c->cfg.f, (cudaStream_t)stream,
                                             &c->launches));
  return FEPLB_OK;
}

extern "C" int feplb_combine_bwd(feplb_ctx* c, const void* d_out, const void* y_perm, const int32_t* slot_to_row,
                                 const float* gates, void* d_y_perm, float* d_gates, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (c->cfg.T == 0) return FEPLB_OK;
  int rc = check_dev_ptrs(c, {d_out, y_perm, d_y_perm});
  if (rc != FEPLB_OK) return rc;
  if (!slot_to_row || !gates || !d_gates) return fail(c, FEPLB_E_INVALID, "combine_bwd: null pointer");
  CUDA_TRY(c, feplb_launch_combine_bwd(d_out, y_perm, slot_to_row, gates, d_y_perm, d_gates, c->cfg.T, c->cfg.K, c->cfg.d,
                                       c->num_sms, (cudaStream_t)stream, &c->launches));
  return FEPLB_OK;
}

extern "C" int feplb_dispatch_bwd(feplb_ctx* c, const void* d_x_perm, const int32_t* slot_to_row, void* d_x, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (c->cfg.T == 0) return FEPLB_OK;
  int rc = check_dev_ptrs(c, {d_x_perm, d_x});
  if (rc != FEPLB_OK) return rc;
  if (!slot_to_row) return fail(c, FEPLB_E_INVALID, "dispatch_bwd: null pointer");
  CUDA_TRY(c, feplb_launch_combine(d_x_perm, slot_to_row, nullptr, d_x, c->cfg.T, c->cfg.K, c->cfg.d, c->num_sms,
                                   (cudaStream_t)stream, &c->launches));
  return FEPLB_OK;
}

extern "C" int feplb_expert_ffn_bwd(feplb_ctx* c, const void* x_perm, const void* ab_saved, void* h,
                                    void* d_y_perm, const void* w1t, const void* w3t, const void* w2t,
                                    const feplb_group* groups, int32_t n_groups, int32_t which,
                                    const feplb_group* expert_table, void* d_ab,
                                    void* d_x_perm, float* dw1, float* dw3, float* dw2, int32_t accumulate,
                                    void* stream) {
  if (!c) return FEPLB_E_INVALID;
  if (n_groups < 0 || n_groups > FEPLB_MAX_GROUPS) return fail(c, FEPLB_E_INVALID, "expert_ffn_bwd: n_groups out of range");
  if (n_groups == 0 || c->s_cap == 0) return FEPLB_OK;
  int rc = check_dev_ptrs(c, {x_perm, ab_saved, h, d_y_perm, w1t, w3t, w2t, d_ab, d_x_perm});
  if (rc != FEPLB_OK) return rc;
  if (!groups) return fail(c, FEPLB_E_INVALID, "expert_ffn_bwd: null group table");
  const bool want_w = dw1 || dw3 || dw2;
  if (want_w) {
    if (!dw1 || !dw3 || !dw2 || !expert_table)
      return fail(c, FEPLB_E_INVALID, "expert_ffn_bwd: weight gradients need dw1, dw3, dw2 and expert_table");
    if (c->cfg.row_align != 128)
      return fail(c, FEPLB_E_INVALID, "expert_ffn_bwd: weight gradients need row_align = 128 (an expert's rows are the K range)");
  }
  feplb_bwd_args a;
  a.x_perm = x_perm; a.ab_saved = ab_saved; a.h = h; a.d_y_perm = d_y_perm;
  a.w1t = w1t; a.w3t = w3t; a.w2t = w2t;
  a.groups = groups; a.n_groups = n_groups; a.which = which;
  a.expert_table = expert_table;
  a.d_ab = d_ab; a.d_x_perm = d_x_perm;
  a.dw1 = want_w ? dw1 : nullptr; a.dw3 = dw3; a.dw2 = dw2; a.accumulate = accumulate != 0;
  a.E = c->cfg.E; a.d = c->cfg.d; a.f = c->cfg.f; a.s_cap = (int64_t)c->s_cap;
  a.status = c->d_status; a.num_sms = c->num_sms;
  a.pair_dgrad = c->bwd_pair & 1; a.pair_wgrad = (c->bwd_pair >> 1) & 1;
  return feplb_launch_expert_ffn_bwd(a, (cudaStream_t)stream, &c->launches, c->err, sizeof(c->err));
}

extern "C" int feplb_moe_backward(feplb_ctx* c, const void* d_out, const float* gates, const void* w1t, const void* w3t,
                                  const void* w2t, const void* x_perm, const void* ab_saved, void* h,
                                  const void* y_perm, const int32_t* slot_to_row,
                                  void* d_y_perm, void* d_ab, void* d_x_perm, void* d_x, float* d_gates,
                                  float* dw1, float* dw3, float* dw2, int32_t accumulate, void* stream) {
  if (!c) return FEPLB_E_INVALID;
  int rc = feplb_combine_bwd(c, d_out, y_perm, slot_to_row, gates, d_y_perm, d_gates, stream);
  if (rc != FEPLB_OK) return rc;
  // every expert's rows in one table: the home table of the forward pass that ran last on this context
  rc = feplb_expert_ffn_bwd(c, x_perm, ab_saved, h, d_y_perm, w1t, w3t, w2t, c->d_home_groups, c->cfg.E, FEPLB_FFN_ALL,
                            c->d_home_groups, d_ab, d_x_perm, dw1, dw3, dw2, accumulate, stream);
  if (rc != FEPLB_OK) return rc;
  return feplb_dispatch_bwd(c, d_x_perm, slot_to_row, d_x, stream);
}
