/*
 * conqur.h -- C ABI of the ConQuR online rotation-calibration hot path (B200, sm_100a).
 *
 * One context holds one orthogonal Procrustes problem of size d (or P independent
 * problems of size d, the per-head case): the current rotation R (d x d), the
 * accumulated cross-covariance M (d x d) and the objective sums J, N.
 *
 * Row-vector convention (the paper's Appendix A, "X_hat = X R"): activations are
 * the ROWS of X (n x d, row-major), the rotation acts on the right.  The paper's
 * Section 3.3 states the same update in column form; with R_here = R_paper^T and
 * M_here = (Z^T X_tilde)^T the two are the same matrices transposed.
 *
 * Memory: every pointer named *_dev is DEVICE memory owned by the caller,
 * including the workspace.  The library allocates no device memory.  Pointers
 * without that suffix are HOST memory.  All matrices are dense row-major.
 *
 * Ordering: conqur_step / conqur_step_batched(_range) / conqur_update only ENQUEUE work on
 * the context's stream and return; X must stay valid until that work has run.
 * The conqur_get_* calls synchronise the stream.  A context is not thread-safe.
 *
 * Errors: every call returns CONQUR_OK (0) or a negative conqur_status.  Errors
 * found on the host change nothing.  Conditions found on the device (non-finite
 * input, Newton-Schulz not converged) are latched in a device status word and
 * returned by the next synchronising call; conqur_get_stats reports and clears it.
 */
#ifndef CONQUR_H_
#define CONQUR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct conqur_ctx conqur_ctx;

typedef enum {
  CONQUR_OK = 0,
  CONQUR_ERR_INVALID_ARG = -1,
  CONQUR_ERR_WORKSPACE_TOO_SMALL = -2,
  CONQUR_ERR_NOT_ORTHOGONAL_INPUT = -3,
  CONQUR_ERR_EMPTY_UPDATE = -4,     /* update with no accumulated tokens */
  CONQUR_ERR_RANK_DEFICIENT = -5,   /* fewer tokens than dimensions and prior_rel == 0 */
  CONQUR_ERR_NS_NOT_CONVERGED = -6, /* previous R kept, M not cleared */
  CONQUR_ERR_NONFINITE_INPUT = -7,  /* a row of X held NaN/Inf (that row was skipped) */
  CONQUR_ERR_TIMEOUT = -8,          /* a bounded device-side wait expired */
  CONQUR_ERR_CUDA = -9,
  CONQUR_ERR_UNSUPPORTED = -10
} conqur_status;

enum { CONQUR_F32 = 0, CONQUR_BF16 = 1 };            /* storage type of X */
enum { CONQUR_EXACT_F32 = 0, CONQUR_TC_BF16 = 1 };   /* arithmetic mode */
enum { CONQUR_QUANT_SYMMETRIC = 0, CONQUR_QUANT_ZEROPOINT = 1 };   /* fake-quantiser applied when quant_bits > 0 */

/*
 * mode CONQUR_EXACT_F32: fp32 CUDA-core contractions throughout (parity anchor).
 * mode CONQUR_TC_BF16:   bf16 operands, fp32 accumulation on the tcgen05 tensor
 *                        cores; fp32 X is rounded to bf16 on the way in; the
 *                        Newton-Schulz iterate is held as a two-term bf16 split hi + lo
 *                        and each of its products takes one to three bf16 passes
 *                        (hi hi, hi lo, lo hi), chosen per step on the device.
 */
typedef struct {
  uint32_t struct_size;     /* = sizeof(conqur_config) */
  int32_t  in_dtype;        /* CONQUR_F32 | CONQUR_BF16 */
  int32_t  mode;            /* CONQUR_EXACT_F32 | CONQUR_TC_BF16 */
  int32_t  quant_bits;      /* 0: corner target on the rotated row (Eq. 2);
                               b in 2..8: per-token symmetric b-bit fake-quantisation of the
                               rotated row first (Appendix B, Q_sym), levels -(2^(b-1)-1)..(2^(b-1)-1),
                               round half to even */
  int32_t  ns_steps;        /* Newton-Schulz steps a problem's FIRST update plans for (a budget, not a cap: the
                               orthogonality check decides when the iteration ends, conqur_get_stats reports the steps
                               used; later updates start from the count learnt so far, see conqur_update);
                               0 = derive from ns_sigma_min_rel */
  int32_t  ns_max_steps;    /* hard cap on Newton-Schulz steps per update; 0 = max(planned schedule + 12, 40) */
  float    orth_tol;        /* accept R when max|R^T R - I| <= orth_tol; 0 = default 1e-4 */
  float    prior_rel;       /* lam_rel >= 0: update is polar(M + lam R_prev),
                               lam = lam_rel * ||M||_F / sqrt(d); 0 = the paper's update */
  float    ns_sigma_min_rel;/* assumed lower bound on sigma_min(M)/||M||_F from which the first update of a problem
                               plans its number of lifting steps; 0 = default 1e-9 */
  int64_t  n_max;           /* largest n of any step call (sizes the workspace) */
  int32_t  batch;           /* P >= 1 independent problems of size d */
  int32_t  quant_mode;      /* CONQUR_QUANT_SYMMETRIC: Q_sym of Appendix B (delta = max|y| / (2^(b-1)-1));
                               CONQUR_QUANT_ZEROPOINT: Q_zp of Appendix B (delta = c (max y - min y) / (2^b - 1), integer
                               zero-point, codes clamped to 0..2^b-1), the quantiser the paper's evaluation uses */
  float    clip_ratio;      /* c in (0, 1] for the zero-point quantiser (Appendix C uses 0.9 for activations); 0 = 1 */
  int32_t  diagnostics;     /* 1: every step also gathers the diagnostics of Section 4 (conqur_get_diagnostics); the step
                               then forms the rotated rows in memory first (two passes) */
  int32_t  defer_batches;   /* tensor-core contexts with batch == 1: conqur_step only normalises and keeps a bf16 copy of
                               its rows; the two products run once over all queued rows when this many batches are
                               queued, and at the next conqur_update / conqur_get_* / conqur_set_* call (Section 3.4:
                               the cross-covariance is accumulated with R fixed, so the grouping changes no result
                               beyond fp32 summation order).  Use the update cadence; the workspace grows by
                               4*d*n_max bytes per deferred batch.  0 or 1: every step runs its products at once */
  float    ns_gram_single_pass_tau;  /* tensor-core mode tuning: the Gram product of a Newton-Schulz step runs one bf16
                               pass instead of three while the iterate's mean squared singular value is below this;
                               0 = default */
  float    ns_lo_gap_budget;/* tensor-core mode tuning: bound on the Procrustes gap given up by dropping the low bf16
                               half of the iterate in the products of late steps (a worst-case bound: d directions at the
                               noise floor under one dominant one; measured gaps are 20-50x smaller); 0 = default 5e-4 */
  int32_t  debug_flags;     /* test hooks, 0 in production: CONQUR_DEBUG_CANARIES | CONQUR_DEBUG_SINGLE_CTA |
                               CONQUR_DEBUG_NO_GRAPH */
} conqur_config;

/* debug_flags bits.  CANARIES: every region of the workspace is followed by a 256-byte guard band with a fixed
 * pattern, checked by conqur_debug_check_canaries (a stand-in for a memory checker).  SINGLE_CTA: the tensor-core
 * products never use CTA pairs (exercises the single-CTA kernels on a device that would use pairs).  NO_GRAPH: the
 * update's launch sequence is enqueued directly every time instead of being replayed from a captured graph (so that a
 * profiler's launch list shows its kernels). */
enum { CONQUR_DEBUG_CANARIES = 1, CONQUR_DEBUG_SINGLE_CTA = 2, CONQUR_DEBUG_NO_GRAPH = 4 };

typedef struct {
  uint32_t struct_size;     /* = sizeof(conqur_stats) */
  int32_t  status;          /* latched device status (a conqur_status), cleared by the call */
  int32_t  ns_steps_used;   /* Newton-Schulz steps of the last update (max over problems) */
  int32_t  updates;         /* updates committed so far */
  float    orth_err;        /* max|X^T X - I| measured when the last update accepted R */
  float    orth_fro;        /* ||X^T X - I||_F at that point */
  float    scale;           /* ||M_eff||_F the last update divided by (M without the 1/sqrt(d)) */
  int64_t  n_skipped;       /* rows skipped (zero or non-finite norm) since init */
  double   last_J;          /* objective sum and token count consumed by the last update */
  int64_t  last_N;
  int32_t  ns_lift_plan;    /* lifting steps the next update will start with (learnt from the updates so far; max over problems) */
  int32_t  reserved;
} conqur_stats;

/* Bytes of device workspace conqur_init needs for (d, cfg).  Pure function; 0 on invalid arguments. */
size_t conqur_workspace_bytes(int32_t d, const conqur_config* cfg);

/*
 * Create a context: R <- I, M <- 0, J = N = 0 (Algorithm 1 takes the initial
 * rotations as inputs; use conqur_set_R to supply them).
 *   out            host: receives the context
 *   d              feature dimension, >= 2 (tensor-core mode: a multiple of 128)
 *   cfg            host
 *   workspace_dev  device, 256-byte aligned, >= conqur_workspace_bytes(d, cfg); owned by the
 *                  caller, must outlive the context, contents are the library's
 *   cuda_stream    a cudaStream_t (0 = default stream); all work of this context runs on it
 */
int conqur_init(conqur_ctx** out, int32_t d, const conqur_config* cfg,
                void* workspace_dev, size_t workspace_bytes, void* cuda_stream);

/* Release the host object (the workspace stays the caller's). */
int conqur_destroy(conqur_ctx* ctx);

/*
 * Replace the rotation(s).  R_dev: device fp32, batch x d x d, row-major, acting as
 * X_tilde @ R.  Must be orthogonal: max|R^T R - I| <= 1e-3 is checked (synchronises);
 * otherwise CONQUR_ERR_NOT_ORTHOGONAL_INPUT and the old R is kept.  Does not touch M, J, N.
 */
int conqur_set_R(conqur_ctx* ctx, const float* R_dev);

/*
 * One streamed batch with R fixed (Sections 3.3-3.4: normalise each row, rotate,
 * take the corner target of Eq. 2 -- after Q_sym when quant_bits > 0 -- and add
 * this batch's cross-covariance and objective to M, J, N):
 *   x_tilde_i = x_i / ||x_i||_2 ;  y_i = x_tilde_i R ;  c_i = sgn(y_i)/sqrt(d)
 *   M += X_tilde^T C ;  J += sum_i ||y_i||_1 / sqrt(d) ;  N += rows used
 * sgn(0) = 0.  Rows with zero or non-finite norm are skipped and counted.
 *   X_dev  device, n rows of d elements of cfg.in_dtype, row stride ld elements
 *          (tensor-core mode: X_dev 16-byte aligned and ld*sizeof(element) a multiple of 16)
 *   n      1..cfg.n_max (n = 0 is a no-op)
 * Single-problem contexts only (cfg.batch == 1).
 */
int conqur_step(conqur_ctx* ctx, const void* X_dev, int64_t n, int64_t ld);

/*
 * The per-head form (Section 3.4, "a Procrustes problem per head"): problem p of
 * cfg.batch reads its n rows at X_dev + p*problem_stride + i*ld (elements), each
 * row normalised by its own d-slice norm.  problem_stride = d, ld = P*d is the
 * head-interleaved layout; problem_stride = n*ld is stacked problems.
 * In tensor-core mode (d = 128) the fused kernel takes a row's norm from the rotated row, ||x R~|| with R~ the bf16
 * copy of R its product uses: equal to ||x|| for an orthogonal R, here within ||R~ R~^T - I||_2 / 2 of it (about
 * 1e-4 relative; the scale then enters the target tile rounded to bf16, 2^-9).  A uniform factor on the rows' scales
 * does not change the rotation an update returns.
 */
int conqur_step_batched(conqur_ctx* ctx, const void* X_dev, int64_t n, int64_t ld,
                        int64_t problem_stride);

/*
 * The same for a contiguous range of the context's problems: problems first_problem ..
 * first_problem + n_problems - 1 each take one batch (problem first_problem + q reads its rows at
 * X_dev + q*problem_stride + i*ld); the others are untouched.  This is how Algorithm 1's per-block
 * rotations R_{2,l} share one context of L*n_heads problems: block l feeds problems l*n_heads ..
 * (l+1)*n_heads - 1 when its o_proj input arrives, and one conqur_update at the end of the mini-batch
 * updates all of them (the problems are independent, so this equals updating each block inside the
 * loop).  conqur_update returns CONQUR_ERR_EMPTY_UPDATE while any problem of the context has
 * received no rows since the last update.
 */
int conqur_step_batched_range(conqur_ctx* ctx, const void* X_dev, int64_t n, int64_t ld, int64_t problem_stride,
                              int32_t first_problem, int32_t n_problems);

/*
 * R <- polar(M_eff) = U V^T of the SVD M_eff = U S V^T (Section 3.3), computed by
 * Newton-Schulz iterations and accepted only when max|R^T R - I| <= orth_tol;
 * then M, J, N <- 0 (Algorithm 1 starts every mini-batch with empty statistics).
 * The iteration first lifts the small singular values with a fixed quintic, then converges with a short
 * endgame.  How many lifting steps are needed depends on sigma_min(M), which nothing cheap bounds: each problem
 * starts from the planned count and then learns it from its own updates (a count that fell short costs a few
 * extra steps, never the result).  The rotation returned always passes the same orthogonality check; its last
 * bits depend on the number of steps taken, i.e. on the context's history.
 * Host errors: CONQUR_ERR_EMPTY_UPDATE (no step since the last update),
 * CONQUR_ERR_RANK_DEFICIENT (tokens enqueued < d and prior_rel == 0).
 * If the iteration does not converge within ns_max_steps the old R and M are kept
 * and CONQUR_ERR_NS_NOT_CONVERGED is latched; read it with conqur_get_stats (which also puts the
 * host-side row counts back, so that a later conqur_update sees the statistics that were kept)
 * before the next conqur_update.  The rank check counts rows enqueued, skipped rows included.
 */
int conqur_update(conqur_ctx* ctx);

/* Copy out the current rotation(s): device fp32 batch x d x d.  Synchronises. */
int conqur_get_R(conqur_ctx* ctx, float* R_out_dev);

/*
 * Objective accumulated since the last update, at the R those steps used:
 * J_sum[p] = sum_i ||y_i||_1/sqrt(d) (Section 3.2: the corner distance is 2N - 2J),
 * n_tokens[p] = rows used.  Host arrays of cfg.batch entries.  Synchronises.
 * Per-head contexts (batch > 1) in tensor-core mode without fake-quantisation do not accumulate the sum row by row:
 * with the rotation fixed between two updates, sum_i <x~_i R, s_i> = <R, sum_i x~_i^T s_i> = <R, M> (Eq. 4 with the
 * corner target), so the objective is formed from the accumulated cross-covariance, here and by conqur_update (the
 * value it consumes is reported as conqur_stats.last_J).  A rotation replaced by conqur_set_R between two updates is
 * then the one the whole sum is evaluated with.
 */
int conqur_get_objective(conqur_ctx* ctx, double* J_sum, int64_t* n_tokens);

/*
 * The same two arrays without stopping the stream: the values as of this point of the context's stream are copied to
 * J_sum_host / n_tokens_host (host arrays of cfg.batch entries; page-locked memory for the copy to overlap) by copies
 * enqueued on that stream, and the call returns at once.  The arrays hold the result, and must stay valid, once the
 * stream has passed this point (an event recorded on the stream after the call, or any synchronising call).  For a
 * training loop that logs the objective of every cycle without draining the queue: enqueue the read, then
 * conqur_update, and look at the numbers one cycle later.  Runs the products of queued batches first, like
 * conqur_get_objective.  Device-side conditions (CONQUR_ERR_NONFINITE ...) are reported by the next synchronising
 * call, not here.
 */
int conqur_get_objective_async(conqur_ctx* ctx, double* J_sum_host, int64_t* n_tokens_host);

/*
 * Diagnostics of Section 4 over the rows used since the last update, at the R those steps used (cfg.diagnostics = 1):
 *   sum_pr_over_d  sum_i PR(y_i)/d,  PR(y)/d = ||y||_2^4 / (d ||y||_4^4) in [1/d, 1]  (normalised participation ratio)
 *   sum_rho        sum_i rho(y_i),   rho(y) = ||y||_inf^2 / ||y||_2^2 in [1/d, 1]     (dynamic-range ratio, Appendix B)
 *   qerr_num/den   ||X R - Q(X R)||_F^2 and ||X||_F^2 on the un-normalised rows       (relative squared quantisation
 *                  error; num = 0 when quant_bits == 0), Q the configured per-token fake-quantiser
 * with y_i = x_i R.  out: host array of cfg.batch entries with struct_size set.  Synchronises.
 * Not gathered by tensor-core contexts with batch > 1 (conqur_init rejects that combination).
 */
typedef struct {
  uint32_t struct_size;     /* = sizeof(conqur_diagnostics) */
  int32_t  reserved;
  double   sum_pr_over_d, sum_rho, qerr_num, qerr_den;
  int64_t  n_tokens;
} conqur_diagnostics;
int conqur_get_diagnostics(conqur_ctx* ctx, conqur_diagnostics* out);

/* Cross-covariance accumulated since the last update, including the 1/sqrt(d):
 * device fp32 batch x d x d.  Synchronises. */
int conqur_get_M(conqur_ctx* ctx, float* M_out_dev);

/* Overwrite the accumulated cross-covariance (same scaling as conqur_get_M) and the sums:
 * resume / teacher forcing.  J_sum, n_tokens: host arrays of cfg.batch entries.  (Where the objective is formed from
 * M, see conqur_get_objective, J_sum is stored but superseded by <R, M> / sqrt(d) at the next read.) */
int conqur_set_M(conqur_ctx* ctx, const float* M_dev, const double* J_sum, const int64_t* n_tokens);

/* Sign decisions of the last step call (tie-aware parity, Eq. 2: which corner each row was sent to): device int8,
 * values -1/0/+1 (0 also for skipped rows), for every problem q the call covered its n x d matrix, row-major, problem
 * after problem ((q*n + i)*d + j).  A context with defer_batches > 1 reports the rows its products last ran over
 * instead: all batches queued since the run before, in order (n = their total).  capacity_rows: rows S_out_dev has
 * room for; fewer than problems * n returns CONQUR_ERR_INVALID_ARG and writes nothing.  Exact-mode contexts and single-problem tensor-core contexts (they keep
 * the targets of the last step in the workspace); CONQUR_ERR_UNSUPPORTED for tensor-core contexts with batch > 1,
 * see conqur_debug_capture_signs.  Synchronises. */
int conqur_debug_get_signs(conqur_ctx* ctx, int8_t* S_out_dev, int64_t capacity_rows);

/* The same read-out for tensor-core contexts with batch > 1, whose fused per-head kernel keeps the targets in shared
 * memory only (Section 3.4, a Procrustes problem per head): after this call every conqur_step_batched(_range) also
 * writes the decisions it takes to S_dev, laid out as above with q counted from the call's first problem; a call with
 * problems * n > capacity_rows then returns CONQUR_ERR_INVALID_ARG and enqueues nothing.  S_dev: device, 16-byte
 * aligned, owned by the caller, valid until replaced; NULL switches the capture off.  Synchronises. */
int conqur_debug_capture_signs(conqur_ctx* ctx, int8_t* S_dev, int64_t capacity_rows);

/* Measurement hook for the fused per-head step kernel (tensor-core contexts with batch > 1; no counterpart in the
 * paper): while a buffer is set, thread block 0 of every conqur_step_batched(_range) records SM-clock timestamps of
 * its first 96 token tiles, 16 int64 slots per tile: 0 copy of the tile issued, 1 / 2 first / second product issued,
 * 5 epilogue reaches the tile, 8 rotated tile available, 3 / 4 pass over it for the rows' scales begins / ends, 6 scales
 * available, 7 target buffer free, 13 / 14 / 15 first TMEM load back / first half written / second TMEM load back,
 * 9 epilogue done;
 * on a problem's last tile 10 / 11 / 12 accumulator awaited / being written out / written out.  trace_dev: device,
 * capacity >= 96 * 16 int64, owned by the caller; NULL stops the recording.  Synchronises. */
int conqur_debug_trace_heads(conqur_ctx* ctx, int64_t* trace_dev, int64_t capacity);

/* Test hook (no counterpart in the paper): with CONQUR_DEBUG_CANARIES set, counts the guard bands behind the
 * workspace regions whose pattern has been overwritten (0 = all intact; a kernel of this library wrote past a region
 * otherwise).  Returns that count, or a negative status (CONQUR_ERR_INVALID_ARG when the context was created without
 * the flag).  Synchronises. */
int conqur_debug_check_canaries(conqur_ctx* ctx);

/* Counters of the last update and the latched device status (cleared).  Synchronises. */
int conqur_get_stats(conqur_ctx* ctx, conqur_stats* out);

/*
 * Launch accounting (measurement support; no counterpart in the paper).  Kernel classes:
 * 0 row norms, 1 rotate+target, 2 accumulate, 3/4/5 the three Newton-Schulz products
 * (residual X^T X - I, polynomial, next iterate), 6 everything else (reductions, element-wise).
 * Launch counts are always kept.  With profiling enabled each contraction launch is bracketed by
 * CUDA events on the context's stream and conqur_update synchronises at its end (so enable it only
 * in a measurement pass); flops are those of the tiles a launch computes (2 * 128|256 * tile width * K per tile
 * and bf16 pass: a symmetric product counts its upper-triangle tiles only, a split product every pass it
 * takes), for launches that did not early-exit.
 */
#define CONQUR_KERNEL_CLASSES 8
typedef struct {
  uint32_t struct_size;                          /* = sizeof(conqur_profile) */
  int32_t  reserved;
  int64_t  launches[CONQUR_KERNEL_CLASSES];      /* kernels launched since conqur_set_profiling */
  int64_t  timed_launches[CONQUR_KERNEL_CLASSES];/* launches with event timing that ran to completion */
  double   flops[CONQUR_KERNEL_CLASSES];         /* algorithmic flops of the timed launches */
  double   ms[CONQUR_KERNEL_CLASSES];            /* summed event time of the timed launches */
  int64_t  total_launches;
} conqur_profile;

/* Reset the counters and switch per-launch event timing on or off.  Synchronises. */
int conqur_set_profiling(conqur_ctx* ctx, int32_t enabled);
/* Read the counters.  Synchronises. */
int conqur_get_profile(conqur_ctx* ctx, conqur_profile* out);

/*
 * Host-only introspection of the Newton-Schulz plan (no device needed): the odd quintics
 * p_k(x) = a x + b x^3 + c x^5 an update applies, in order, for a spectrum assumed to lie in
 * [sigma_min_rel, 1] after scaling (ns_steps > 0 instead plans for exactly that many steps).
 * abc_out: host, 3*max_steps doubles.  Returns the number of steps written, or a negative status.
 * No counterpart in the paper, which takes R <- U V^T from an SVD (Section 3.3); the polynomials
 * are this library's route to the same polar factor.
 */
int conqur_plan_schedule(double sigma_min_rel, int32_t ns_steps, double* abc_out, int32_t max_steps);

/*
 * Test hook for the tensor-core product every fused step is built on (no counterpart in the paper):
 *   D[m][n] = sum_k A(m,k) * B(n,k),  D_dev fp32 M x N row-major.
 * A_dev / B_dev: device bf16 row-major.  Orientation 0 (K-major): the matrix is [M|N rows][K cols];
 * orientation 1 (MN-major): it is [K rows][M|N cols].  split != 0: each operand is a stacked pair
 * [hi; lo] (twice the rows) and the product is hi*hi + hi*lo + lo*hi.  M, K multiples of 8, N of 32.
 * scratch_dev: >= 512 bytes of device memory.  Synchronises; returns CONQUR_ERR_TIMEOUT if a bounded
 * device-side wait expired.
 */
int conqur_debug_gemm(const void* A_dev, const void* B_dev, float* D_dev, int32_t M, int32_t N, int32_t K,
                      int32_t a_mn_major, int32_t b_mn_major, int32_t split, void* scratch_dev, void* cuda_stream);

/*
 * Test hook for the bounded device-side waits (no counterpart in the paper).  Every wait of the tensor-core kernels
 * (on a TMA completion, on the MMA pipeline, on a peer CTA) gives up after a cycle limit, latches
 * CONQUR_ERR_TIMEOUT and lets the kernel end normally, so that a protocol error can never hang the GPU.  This call
 * runs that mechanism on purpose: one thread waits, for at most limit_cycles SM clocks (1 .. 2e9), on a barrier
 * that nothing arrives at.  Returns CONQUR_ERR_TIMEOUT when the wait gave up as designed (the expected result),
 * CONQUR_OK if it did not.  scratch_dev: >= 512 bytes of device memory.  Synchronises the stream; the context
 * of the process stays usable.
 */
int conqur_debug_wait_timeout(void* scratch_dev, int64_t limit_cycles, void* cuda_stream);

/*
 * The corner objective of one batch without any device-memory allocation by anyone
 * (the paper has no counterpart; this serves callers that cannot call cudaMalloc -- e.g. code
 * running under a runtime that owns all device memory, or a plugin in a process whose device
 * memory is pre-assigned -- and therefore cannot provide the workspace conqur_init needs).
 *
 * Computes, in the exact fp32 arithmetic of conqur_step's exact mode and with R fixed,
 *   J = sum_i ||x_tilde_i R||_1 / sqrt(d)   and   N = rows with a finite, non-zero norm
 * (the quantities conqur_get_objective reports after one conqur_step on a fresh context).
 *   X_dev      device, n rows of d elements of in_dtype (CONQUR_F32 | CONQUR_BF16), row stride ld elements
 *   R_dev      device fp32 d x d row-major
 *   J_out_dev  device: one double;   N_out_dev: device: one int64.  Written on the stream; not synchronised.
 *   limits     n <= 32768 and d <= 8192: the scratch (row norms, per-CTA partial sums; about 260 KB) is a
 *              fixed array inside the library image, held by every GPU that loads the library until
 *              the process exits.  Larger sizes return CONQUR_ERR_UNSUPPORTED and do nothing.
 * The first call on each device looks up the array's device address (with that device current); make
 * that first call outside any stream capture.  The call uses no cudaMalloc/cudaFree and no allocating
 * library routine.  All calls on a device share the one array: it still holds the previous call's
 * contents (the counters are cleared at the start of each call), and two calls whose kernels overlap
 * on the GPU (different streams, different threads) race on it -- serialise them.
 */
int conqur_objective_noalloc(const void* X_dev, int32_t in_dtype, int64_t n, int32_t d, int64_t ld,
                             const float* R_dev, double* J_out_dev, int64_t* N_out_dev, void* cuda_stream);

/*
 * Appendix A, rotation invariance: with activations rotated as X_hat = X R, a linear layer y = x W^T
 * (W: rows = outputs, cols = inputs, row-major) keeps its function when the rotation is absorbed into W:
 *   CONQUR_FOLD_INPUT   the layer READS rotated activations (q/k/v/up/gate projections for R_1; o_proj for R_2):
 *                       W' = W R          since X W^T = (X R)(W R)^T
 *   CONQUR_FOLD_OUTPUT  the layer WRITES into the rotated space (o_proj and down projection for R_1, whose outputs
 *                       join the rotated residual stream; the value projection for R_2):
 *                       W' = R^T W        since (X W^T) R = X (R^T W)^T
 * R is block diagonal with square blocks of size `block` (one full rotation when block equals the folded
 * dimension; block = d_h for the per-head rotations R_2): R_dev holds the blocks one after another, each
 * block x block fp32 row-major.  The folded dimension (cols for INPUT, rows for OUTPUT) must be a multiple of
 * block.
 *   W_dev / out_dev   device fp32, rows x cols, row strides ldw / ldo elements (>= cols); out_dev must not
 *                     overlap W_dev
 *   mode              CONQUR_EXACT_F32: fp32 CUDA-core product.
 *                     CONQUR_TC_BF16: for one full rotation (block == folded dimension, a multiple of 128;
 *                     rows % 8 == 0 for INPUT, cols % 32 == 0 for OUTPUT; ldw, ldo multiples of 4; 16-byte
 *                     aligned pointers) both operands are split into bf16 hi + lo and the product is taken
 *                     in three tensor-core passes (hi hi, hi lo, lo hi) with fp32 accumulation, relative
 *                     error about 2^-16; shapes outside these limits return CONQUR_ERR_UNSUPPORTED.
 *                     Block-diagonal folds (block < folded dimension) use the fp32 product in either mode.
 *   scratch_dev       device memory, 256-byte aligned, >= conqur_fold_scratch_bytes(...) bytes (returns -1 for
 *                     invalid arguments); owned by the caller, free to reuse after the call returns
 * Synchronises the stream and returns the status (CONQUR_ERR_TIMEOUT if a bounded device wait expired).
 */
enum { CONQUR_FOLD_INPUT = 0, CONQUR_FOLD_OUTPUT = 1 };
int64_t conqur_fold_scratch_bytes(int32_t rows, int32_t cols, int32_t block, int32_t side, int32_t mode);
int conqur_fold_weight(const float* W_dev, int64_t ldw, int32_t rows, int32_t cols, const float* R_dev,
                       int32_t block, int32_t side, int32_t mode, float* out_dev, int64_t ldo, void* scratch_dev,
                       int64_t scratch_bytes, void* cuda_stream);

/*
 * The fixed online rotations R_3 / R_4 of Appendix A: every row times the orthonormal Walsh-Hadamard matrix,
 *   y = x H_d / sqrt(d),   H_d the Sylvester matrix, H[i][j] = (-1)^popcount(i & j).
 * d a power of two, 4 <= d <= 8192.
 *   X_dev   device, n rows of d elements of in_dtype (CONQUR_F32 | CONQUR_BF16), row stride ldx elements
 *   Y_dev   device, n rows of d elements of out_dtype, row stride ldy; may be X_dev itself (same type and
 *           stride): every row is read completely before it is written
 *   ldx, ldy multiples of 4; pointers aligned to 4 elements.
 * Enqueued on the stream; not synchronised.  Invalid arguments return CONQUR_ERR_INVALID_ARG and do nothing.
 * Arithmetic: fp32 throughout, error per element <= log2(d) 2^-24 ||x||_2 (plus the rounding of a bf16 output).
 *   - bf16 rows lying back to back (ldx == ldy == d, 16-byte aligned pointers, n*d a multiple of 128): H_d is
 *     taken as H_{d/128} (x) H_128; the 128-point transforms of all 128-element chunks run as one tensor-core
 *     product per tile with exact operands (the bf16 input and a +-1 matrix, fp32 accumulation), the remaining
 *     log2(d/128) butterfly levels in registers.  No d x d matrix is formed.
 *   - every other layout (fp32 input, strided or unaligned rows): log2(d) butterfly levels on the CUDA cores; rows
 *     that start on 16-byte boundaries are staged through shared memory by bulk asynchronous copies, others by
 *     plain loads.
 *
 * conqur_hadamard_status: synchronises the stream and returns CONQUR_ERR_TIMEOUT if, since the last call on
 * this device, a transform kernel abandoned a bounded wait for one of its copies or products (its output is then
 * incomplete), CONQUR_OK otherwise; clears the latch.
 */
enum { CONQUR_HADAMARD_CUDA_CORES_ONLY = 1 };   /* flags: never take the tensor-core kernel (tests compare the two) */
int conqur_hadamard_rows(const void* X_dev, int32_t in_dtype, int64_t n, int32_t d, int64_t ldx, void* Y_dev,
                         int32_t out_dtype, int64_t ldy, int32_t flags, void* cuda_stream);
int conqur_hadamard_status(void* cuda_stream);

const char* conqur_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* CONQUR_H_ */
