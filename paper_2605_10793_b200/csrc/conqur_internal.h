// Internal definitions shared by the host orchestration and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

namespace conqur {

enum : int {
  STATUS_FLAG_NONFINITE = 1,
  STATUS_FLAG_NS_FAILED = 2,
  STATUS_FLAG_TIMEOUT = 4,
};
enum : int { NS_DONE_CONVERGED = 1, NS_DONE_FAILED = 2 };

// Per-problem device state (lives at the head of the workspace).
struct DevState {
  double J;                 // objective sum since the last update (1/sqrt(d) applied)
  long long N;              // rows used since the last update
  long long n_skipped;      // rows skipped since init
  long long step_skipped;   // rows skipped by the step in flight (folded by finalize_step)
  double last_J;
  long long last_N;
  int status_flags;
  int ns_done;              // 0 running, NS_DONE_*
  int ns_steps_used;
  int ns_final_buf;
  int updates;
  int timeout_site;
  float e_max, e_fro;       // residual norms of the last Newton-Schulz check
  float last_orth, last_fro;
  float scale, x0_scale, lam;
  float coef[4];            // gamma + kappa, beta1, beta2, kappa of the step in flight
  float tau;                // shift of the residual: E = X^T X - tau I (1 in exact mode)
  int ns_idx;               // next entry of the polynomial schedule
  int seg_x;                // tensor-core mode: passes of the next-iterate product of the step in flight (1 or 2)
  int seg_e;                // tensor-core mode: passes of the next residual product (1 while the iterate is tiny, else 3)
  // How many lifting steps an update starts with is learnt per problem from the updates before it: the count that
  // keeps the running mean of the steps spent beyond plan + endgame below one; see ns_adapt_lift_plan.
  int lift_init, lift_plan;
  int lift_succ, lift_patience;   // updates in a row that needed no extra step / how many of them before one step fewer is tried
  int lift_trial;                 // updates left of the trial period after such a descent
  float lift_ema;                 // running mean of the extra steps at the current count
  int loop_passes;          // passes of the update graph's loop body in the update in flight
  long long loop_passes_total;   // ... since init (launch accounting)
  int lift_left;            // lifting steps still to run in the update in flight
  int reentries;            // times the endgame ran out in the update in flight
  float growth;             // cumulative growth of the smallest singular values in the update in flight
  double diag_pr, diag_rho, diag_qnum, diag_qden;   // Section-4 diagnostics accumulated since the last update
  unsigned char seg_log[128];   // seg_x | seg_e << 4 of each step of the last update (launch accounting)
};

static_assert(sizeof(DevState) <= 512, "scratch buffers of the test hooks are documented as 512 bytes");

// One entry of the device copy of the polynomial schedule.
struct SchedEntry { float a, b, c, l; int lift, seg_x; };
constexpr int NS_SCHED_MAX = 128;

// Kernel classes for launch counting / optional per-launch timing.
enum : int { K_ROWNORM = 0, K_ROTATE = 1, K_ACCUM = 2, K_NS_RESID = 3, K_NS_POLY = 4, K_NS_NEXT = 5, K_OTHER = 6, K_COUNT = 8 };

// Host-side launch accounting.  Launch counts are always kept; when `enabled`, the contractions are bracketed by
// CUDA events on the launching stream (events are created lazily and reused).
struct Prof {
  struct Rec { int cls; double flops; int ns_k; int nseg; cudaEvent_t e0, e1; };   // nseg 0 / -1: seg_x / seg_e from seg_log
  bool enabled = false;
  long long launches[K_COUNT] = {0};
  long long total = 0;
  double flops[K_COUNT] = {0};
  double ms[K_COUNT] = {0};
  long long timed[K_COUNT] = {0};
  std::vector<Rec> open;                 // records not yet folded into the sums
  std::vector<cudaEvent_t> pool;

  void count(int cls) { ++launches[cls]; ++total; }
  cudaEvent_t get_event() {
    if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
  // Fold the finished records into the sums (call after a stream synchronise).  Newton-Schulz launches whose
  // step index lies past `steps_used` early-exited on the device and are left out.
  void fold(int steps_used, const unsigned char* seg_log = nullptr) {
    for (Rec& r : open) {
      bool ran = true;
      if (r.ns_k >= 0) ran = (r.cls == K_NS_RESID) ? (r.ns_k <= steps_used) : (r.ns_k < steps_used);
      float t = 0.f;
      if (cudaEventElapsedTime(&t, r.e0, r.e1) == cudaSuccess && ran) {
        int passes = r.nseg;
        if (passes <= 0) {
          const int lg = (seg_log && r.ns_k >= 0 && r.ns_k < 128) ? seg_log[r.ns_k] : 0x31;
          passes = (passes == 0) ? (lg & 15) : (lg >> 4);
          if (passes < 1) passes = 1;
        }
        ms[r.cls] += t; flops[r.cls] += r.flops * passes; ++timed[r.cls];
      }
      pool.push_back(r.e0); pool.push_back(r.e1);
    }
    open.clear();
  }
  void reset() {
    for (int i = 0; i < K_COUNT; ++i) { launches[i] = 0; flops[i] = 0; ms[i] = 0; timed[i] = 0; }
    total = 0;
  }
  ~Prof() {
    for (Rec& r : open) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
    for (cudaEvent_t e : pool) cudaEventDestroy(e);
  }
};

}  // namespace conqur
