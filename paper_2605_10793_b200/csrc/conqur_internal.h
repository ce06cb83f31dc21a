// Internal definitions shared by the host orchestration and the kernels.
#pragma once
#include <stddef.h>
#include <stdint.h>

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
  float coef[3];            // gamma, beta1, beta2 of the step in flight
  float pad_[2];
};

}  // namespace conqur
