// Host side of the C ABI: argument checks, workspace carving, launch sequencing.
// Every step of the path runs in the kernels of conqur_simt.cuh / conqur_tc.cuh; this file only
// enqueues them.  There is no CPU fallback: without a CUDA device every entry point fails.
#include "../../include/conqur.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "conqur_internal.h"
#include "conqur_simt.cuh"
#include "conqur_tc.cuh"
#include "conqur_tc_batched.cuh"
#include "conqur_aux.cuh"
#include "conqur_hadamard_tc.cuh"
#include "ns_schedule.h"

using namespace conqur;

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }
inline int cdiv(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

struct Layout {
  size_t state, flags_agg, R, M, rnorm, rowmax, part_d, part_f, part_diag, sched, obj_out;
  size_t C;                 // exact: fp32 C' / Y (P x n_max x d); TC quant mode: fp32 Y
  size_t Xa, Xb, E, B;      // Newton-Schulz fp32 matrices (P x d x d each)
  size_t splitk;            // exact accumulate split-K partials
  TcLayout tc;              // tensor-core mode buffers
  size_t total;
  int64_t max_partials;
  int acc_splits;
  int64_t n_rows;           // rows the per-step buffers hold: n_max, times the deferred batches of a tensor-core context
  int n_guards;             // CONQUR_DEBUG_CANARIES: guard bands behind the regions, at guard[i]
  size_t guard[48];
};
constexpr size_t GUARD_BYTES = 256;
constexpr unsigned char GUARD_PATTERN = 0xC5;

struct Cfg {
  int d, P, in_dtype, mode, quant_bits, ns_max_steps, defer, debug_flags;
  QuantSpec qs;
  int diagnostics;
  int64_t n_max;
  float orth_tol, prior_rel, fro_tol, margin, lo_budget;
  bool simt_ns;             // the Newton-Schulz products run on the fp32 CUDA-core kernels (exact mode)
};

int pick_acc_splits(int d, int P, int64_t n_max) {
  const int tiles = cdiv(d, SG_BM) * cdiv(d, SG_BN) * P;
  if (tiles >= 148) return 1;
  int s = std::min<int64_t>(16, std::max<int64_t>(1, 148 / tiles));
  s = (int)std::min<int64_t>(s, std::max<int64_t>(1, n_max / 256));
  return std::max(1, s);
}

bool make_layout(int d, const conqur_config* c, Layout* L) {
  if (!c || c->struct_size != sizeof(conqur_config)) return false;
  if (d < 2 || d > 32768 || c->n_max < 1 || c->batch < 1 || c->batch > 65535) return false;
  if (c->in_dtype != CONQUR_F32 && c->in_dtype != CONQUR_BF16) return false;
  if (c->mode != CONQUR_EXACT_F32 && c->mode != CONQUR_TC_BF16) return false;
  if (c->quant_bits != 0 && (c->quant_bits < 2 || c->quant_bits > 8)) return false;
  if (c->quant_mode != CONQUR_QUANT_SYMMETRIC && c->quant_mode != CONQUR_QUANT_ZEROPOINT) return false;
  if (c->clip_ratio < 0.f || c->clip_ratio > 1.f) return false;
  if (c->diagnostics != 0 && c->diagnostics != 1) return false;
  if (c->diagnostics && c->mode == CONQUR_TC_BF16 && c->batch > 1) return false;   // the fused per-head kernel gathers none
  if (c->prior_rel < 0.f || c->orth_tol < 0.f || c->ns_sigma_min_rel < 0.f || c->ns_steps < 0 || c->ns_max_steps < 0)
    return false;
  if (c->mode == CONQUR_TC_BF16 && !tc_supported_shape(d, c->batch)) return false;
  if (c->defer_batches < 0 || c->defer_batches > 64) return false;
  if (c->defer_batches > 1 && (c->mode != CONQUR_TC_BF16 || c->batch != 1)) return false;
  if (c->ns_gram_single_pass_tau < 0.f || c->ns_lo_gap_budget < 0.f) return false;
  if (c->debug_flags & ~(CONQUR_DEBUG_CANARIES | CONQUR_DEBUG_SINGLE_CTA | CONQUR_DEBUG_NO_GRAPH)) return false;
  const int64_t P = c->batch;
  // a deferring context keeps the rows of up to defer_batches steps: every per-row buffer is that much longer
  const int64_t n = c->n_max * std::max(1, c->defer_batches);
  if (n > (int64_t)1 << 30) return false;
  L->n_rows = n;
  const size_t dd = (size_t)d * d;
  size_t off = 0;
  const bool guards = (c->debug_flags & CONQUR_DEBUG_CANARIES) != 0;
  L->n_guards = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes);
    if (guards && L->n_guards < 48) { L->guard[L->n_guards++] = off; off += GUARD_BYTES; }
    return o;
  };
  L->state = take(sizeof(DevState) * P);
  L->flags_agg = take(sizeof(int) * 4);
  L->R = take(sizeof(float) * dd * P);
  L->M = take(sizeof(float) * dd * P);
  L->rnorm = take(sizeof(float) * n * P);
  L->rowmax = take(sizeof(unsigned) * 2 * n * P);   // per row: ordered max, then ordered min (quant modes)
  int64_t mp = std::max<int64_t>((int64_t)cdiv(n, 128) * cdiv(d, 128), (int64_t)cdiv(d, 128) * cdiv(d, 128));
  mp = std::max<int64_t>(mp, cdiv(n, 8));
  mp = std::max<int64_t>(mp, 2 * (int64_t)cdiv(d, 128) * cdiv(d, 128) + 64);   // two partial arrays per Newton-Schulz product
  mp = std::max<int64_t>(mp, 1024);
  L->max_partials = mp;
  L->part_d = take(sizeof(double) * mp * P);
  L->part_f = take(sizeof(float) * mp * P);
  L->part_diag = c->diagnostics ? take(sizeof(double) * 4 * mp * P) : 0;
  L->sched = take(sizeof(SchedEntry) * NS_SCHED_MAX);
  L->obj_out = take(16 * P);                         // J (double) and N (int64) of every problem, for the asynchronous read
  L->acc_splits = 1;
  L->C = L->splitk = 0;
  // the four Newton-Schulz matrices form ONE region: a token-split per-head step borrows all of it as scratch
  const size_t ns_one = align_up(sizeof(float) * dd * P);
  L->Xa = take(4 * ns_one);
  L->Xb = L->Xa + ns_one;
  L->E = L->Xb + ns_one;
  L->B = L->E + ns_one;
  if (c->mode == CONQUR_EXACT_F32) {
    L->C = take(sizeof(float) * (size_t)n * d * P);
    L->acc_splits = pick_acc_splits(d, (int)P, n);
    if (L->acc_splits > 1) L->splitk = take(sizeof(float) * dd * P * L->acc_splits);
  } else {
    if ((c->quant_bits || c->diagnostics) && P == 1) L->C = take(sizeof(float) * (size_t)n * d);
    tc_make_layout(d, (int)P, n, c->quant_bits, c->in_dtype, &L->tc, take);
  }
  L->total = off;
  return true;
}

}  // namespace

struct conqur_ctx {
  Cfg cfg;
  Layout L;
  char* ws;
  cudaStream_t stream;
  std::vector<int64_t> tokens;   // per problem: rows enqueued since the last update
  std::vector<int64_t> tokens_at_update;   // ... as they stood when the last update was enqueued (restored if it is rejected)
  int64_t last_n;            // rows per problem of the last step (for debug_get_signs)
  int last_np;               // problems the last step call covered
  int64_t pending_rows = 0;  // deferring context: rows staged but not yet run through the two products
  int pending_batches = 0;
  int8_t* sign_capture = nullptr;   // conqur_debug_capture_signs: where the fused per-head kernel writes its decisions
  int64_t sign_capture_rows = 0;
  long long* heads_trace = nullptr;  // conqur_debug_trace_heads: timeline buffer of the fused per-head step kernel
  int n_sched, n_lift_init;   // device schedule: entry 0 = lifting quintic, 1 .. n_sched-1 = endgame; planned lifting steps
  std::vector<NsStep> sched;
  TcHost tc;                 // tensor maps etc. of the tensor-core mode
  Prof prof;
  // The update enqueues the same ~150 launches every time (same buffers, same order; which of them do work is
  // decided on the device), so after the first update it is captured once into a CUDA graph and replayed.
  cudaStream_t cap_stream = nullptr;       // side stream used only to capture
  cudaGraphExec_t upd_graph = nullptr;
  int updates_enqueued = 0;
  long long graph_launches[K_COUNT] = {0};     // launches of one graph replay (outside its loop, if it has one)
  long long loop_body_launches[K_COUNT] = {0}; // launches of one pass of the looped graph's body
  bool looped = false;                         // the graph holds a device-side loop
  long long loop_passes_seen = 0;              // passes already folded into the launch counts

  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
  DevState* state() const { return at<DevState>(L.state); }
};

namespace {

int cuda_fail(const char* what, cudaError_t e) {
  std::fprintf(stderr, "conqur: %s: %s\n", what, cudaGetErrorString(e));
  return CONQUR_ERR_CUDA;
}
#define CQ_CUDA(expr)                                        \
  do {                                                       \
    cudaError_t e__ = (expr);                                \
    if (e__ != cudaSuccess) return cuda_fail(#expr, e__);    \
  } while (0)
#define CQ_LAUNCH_CHECK() CQ_CUDA(cudaGetLastError())
// after a kernel launch of context c: check and count it
#define CQ_LAUNCHED(c, cls)          \
  do {                               \
    CQ_CUDA(cudaGetLastError());     \
    (c)->prof.count(cls);            \
  } while (0)

__global__ void or_flags_kernel(const DevState* st, int P, int* agg) {
  int f = 0;
  for (int i = threadIdx.x; i < P; i += blockDim.x) f |= st[i].status_flags;
  for (int o = 16; o > 0; o >>= 1) f |= __shfl_xor_sync(0xffffffffu, f, o);
  if ((threadIdx.x & 31) == 0 && f) atomicOr(agg, f);
}
__global__ void clear_flags_kernel(DevState* st, int P, int* agg) {
  for (int i = threadIdx.x; i < P; i += blockDim.x) st[i].status_flags = 0;
  if (threadIdx.x == 0) *agg = 0;
}
__global__ void arm_check_kernel(DevState* st, int P) {
  for (int i = threadIdx.x; i < P; i += blockDim.x) { st[i].ns_done = 0; st[i].ns_steps_used = 0; }
}
__global__ void export_sums_kernel(const DevState* st, double* J, long long* N, int P) {
  for (int i = threadIdx.x; i < P; i += blockDim.x) { J[i] = st[i].J; N[i] = st[i].N; }
}
__global__ void set_sums_kernel(DevState* st, const double* J, const long long* N, int P) {
  for (int i = threadIdx.x; i < P; i += blockDim.x) { st[i].J = J[i]; st[i].N = N[i]; }
}

int flags_to_status(int f) {
  if (f & STATUS_FLAG_TIMEOUT) return CONQUR_ERR_TIMEOUT;
  if (f & STATUS_FLAG_NS_FAILED) return CONQUR_ERR_NS_NOT_CONVERGED;
  if (f & STATUS_FLAG_NONFINITE) return CONQUR_ERR_NONFINITE_INPUT;
  return CONQUR_OK;
}

// Synchronise and return the latched device status (not cleared).
int sync_status(conqur_ctx* c) {
  int* agg = c->at<int>(c->L.flags_agg);
  CQ_CUDA(cudaMemsetAsync(agg, 0, sizeof(int), c->stream));
  or_flags_kernel<<<1, 256, 0, c->stream>>>(c->state(), c->cfg.P, agg);
  CQ_LAUNCHED(c, K_OTHER);
  int f = 0;
  CQ_CUDA(cudaMemcpyAsync(&f, agg, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  return flags_to_status(f);
}

int ew_blocks(int64_t count) { return (int)std::min<int64_t>(148 * 8, (count + 255) / 256); }

// ---------------------------------------------------------------- exact-mode step
template <typename TIn>
int step_exact(conqur_ctx* c, const TIn* X, int64_t n, int64_t ld, int64_t pstride, int p0, int np) {
  // problems [p0, p0 + np): state, R and M are theirs; the per-step scratch (row norms, targets, partials) is used
  // from its start
  const Cfg& g = c->cfg;
  const int d = g.d, P = np;
  const int64_t pdd = (int64_t)p0 * d * d;
  DevState* st = c->state() + p0;
  float* rnorm = c->at<float>(c->L.rnorm);
  float* C = c->at<float>(c->L.C);
  double* part = c->at<double>(c->L.part_d);
  const int64_t c_ps = (int64_t)g.n_max * d;
  rownorm_kernel<TIn><<<dim3(cdiv(n, 8), P), 256, 0, c->stream>>>(X, n, d, ld, pstride, rnorm, g.n_max, st, 1);
  CQ_LAUNCHED(c, K_ROWNORM);
  const dim3 grid1(cdiv(d, SG_BN), cdiv(n, SG_BM), P);
  int per_problem;
  double* pdiag = g.diagnostics ? c->at<double>(c->L.part_diag) : nullptr;
  if (g.quant_bits == 0 && !g.diagnostics) {
    rotate_target_exact_kernel<TIn, false><<<grid1, SG_THREADS, 0, c->stream>>>(
        X, ld, pstride, c->at<float>(c->L.R) + pdd, (int)n, d, rnorm, g.n_max, C, c_ps, nullptr, nullptr, part);
    CQ_LAUNCHED(c, K_ROTATE);
    per_problem = grid1.x * grid1.y;
  } else {
    unsigned* rowmax = c->at<unsigned>(c->L.rowmax);
    unsigned* rowmin = rowmax + g.n_max * g.P;
    CQ_CUDA(cudaMemsetAsync(rowmax, 0, sizeof(unsigned) * g.n_max * P, c->stream));
    CQ_CUDA(cudaMemsetAsync(rowmin, 0xff, sizeof(unsigned) * g.n_max * P, c->stream));
    rotate_target_exact_kernel<TIn, true><<<grid1, SG_THREADS, 0, c->stream>>>(
        X, ld, pstride, c->at<float>(c->L.R) + pdd, (int)n, d, rnorm, g.n_max, C, c_ps, rowmax, rowmin, part);
    CQ_LAUNCHED(c, K_ROTATE);
    quant_target_kernel<<<dim3(cdiv(n, 8), P), 256, 0, c->stream>>>(C, n, d, c_ps, rnorm, g.n_max, rowmax, rowmin, g.qs,
                                                                    part, pdiag);
    CQ_LAUNCHED(c, K_OTHER);
    per_problem = cdiv(n, 8);
  }
  finalize_step_kernel<<<P, 256, 0, c->stream>>>(st, part, per_problem, n, 1.0 / std::sqrt((double)d), pdiag,
                                                 pdiag ? cdiv(n, 8) : 0);
  CQ_LAUNCHED(c, K_OTHER);
  const int S = c->L.acc_splits;
  accumulate_exact_kernel<TIn><<<dim3(cdiv(d, SG_BN), cdiv(d, SG_BM), P * S), SG_THREADS, 0, c->stream>>>(
      X, ld, pstride, C, c_ps, rnorm, g.n_max, (int)n, d, S, c->at<float>(c->L.M) + pdd,
      S > 1 ? c->at<float>(c->L.splitk) : nullptr);
  CQ_LAUNCHED(c, K_ACCUM);
  if (S > 1) {
    splitk_reduce_add_kernel<<<dim3(ew_blocks((int64_t)d * d), P), 256, 0, c->stream>>>(
        c->at<float>(c->L.M) + pdd, c->at<float>(c->L.splitk), (int64_t)d * d, S);
    CQ_LAUNCHED(c, K_OTHER);
  }
  return CONQUR_OK;
}

// A deferring context (cfg.defer_batches > 1) queues the staged rows of its steps; this runs the two products over
// everything queued.  Called when the queue is full and before anything reads or replaces the statistics or R.
int flush_pending(conqur_ctx* c) {
  if (c->pending_rows == 0) return CONQUR_OK;
  const int rc = tc_process(c->tc, c->stream, c->pending_rows);
  c->last_n = c->pending_rows;                 // what debug_get_signs reports: the rows this run covered
  c->pending_rows = 0;
  c->pending_batches = 0;
  return rc;
}

// CONQUR_DEBUG_CANARIES: one block per guard band; counts the bands that no longer hold the pattern.
struct GuardList { int n; unsigned long long off[48]; };
__global__ void check_guards_kernel(const unsigned char* ws, const GuardList gl, int* bad) {
  __shared__ int hit;
  if (threadIdx.x == 0) hit = 0;
  __syncthreads();
  if (ws[gl.off[blockIdx.x] + threadIdx.x] != GUARD_PATTERN) hit = 1;
  __syncthreads();
  if (threadIdx.x == 0 && hit) atomicAdd(bad, 1);
}

// ---------------------------------------------------------------- update (both modes share the control flow)
// residual check of the fp32 matrix X (P x d x d) into E; fills the partials.
int launch_residual(conqur_ctx* c, const float* X, int buf) {
  const Cfg& g = c->cfg;
  const int T = cdiv(g.d, SG_BM);
  if (g.simt_ns) {
    ns_gemm_exact_kernel<EPI_RESIDUAL><<<dim3(T, T, g.P), SG_THREADS, 0, c->stream>>>(
        X, X, nullptr, c->at<float>(c->L.E), g.d, c->state(), c->at<float>(c->L.part_f), c->at<double>(c->L.part_d));
    CQ_LAUNCHED(c, K_NS_RESID);
    return CONQUR_OK;
  }
  return tc_ns_residual(c->tc, c->stream, buf);
}
int ns_parts(const conqur_ctx* c) {
  if (c->cfg.simt_ns) { const int T = cdiv(c->cfg.d, SG_BM); return T * T; }
  return tc_ns_parts(c->tc);
}

// The update in three parts, so that it can be enqueued unrolled (every step a fixed set of launches that early-exit once
// the iteration has finished) or as a captured graph whose middle part is a device-side loop.
int update_prologue(conqur_ctx* c) {
  const Cfg& g = c->cfg;
  const int d = g.d, P = g.P;
  const int64_t dd = (int64_t)d * d;
  DevState* st = c->state();
  float* M = c->at<float>(c->L.M);
  float* R = c->at<float>(c->L.R);
  double* pd = c->at<double>(c->L.part_d);
  const int use_shift = g.simt_ns ? 0 : 1;
  const int nb = (int)std::min<int64_t>(1024, (dd + 1023) / 1024);
  const float isd = (float)(1.0 / std::sqrt((double)d));
  sumsq_kernel<<<dim3(nb, P), 256, 0, c->stream>>>(M, R, dd, st, 0, pd);
  CQ_LAUNCHED(c, K_OTHER);
  ns_setup_kernel<<<P, 256, 0, c->stream>>>(st, pd, nb, 0, g.prior_rel, isd, g.margin, d, use_shift, c->tc.e1_tau, c->n_lift_init);
  CQ_LAUNCHED(c, K_OTHER);
  if (g.prior_rel > 0.f) {
    sumsq_kernel<<<dim3(nb, P), 256, 0, c->stream>>>(M, R, dd, st, 1, pd);
    CQ_LAUNCHED(c, K_OTHER);
  }
  ns_setup_kernel<<<P, 256, 0, c->stream>>>(st, pd, nb, 1, g.prior_rel, isd, g.margin, d, use_shift, c->tc.e1_tau, c->n_lift_init);
  CQ_LAUNCHED(c, K_OTHER);
  if (g.simt_ns) {
    ns_x0_kernel<<<dim3(ew_blocks(dd), P), 256, 0, c->stream>>>(M, R, c->at<float>(c->L.Xa), dd, st);
    CQ_LAUNCHED(c, K_OTHER);
    return CONQUR_OK;
  }
  return tc_ns_begin(c->tc, c->stream);          // the same X0, written as the bf16 pair the products read
}

// One Newton-Schulz step on the iterate in buffer `cur`: residual product, control decision, and (unless `last`)
// the polynomial and next-iterate products.  k: the step's index, or -1 to take it from the device state.
int update_step(conqur_ctx* c, int k, int cur, bool last) {
  const Cfg& g = c->cfg;
  const int d = g.d, P = g.P;
  DevState* st = c->state();
  float* Xa = c->at<float>(c->L.Xa);
  float* Xb = c->at<float>(c->L.Xb);
  float* E = c->at<float>(c->L.E);
  float* B = c->at<float>(c->L.B);
  double* pd = c->at<double>(c->L.part_d);
  float* pf = c->at<float>(c->L.part_f);
  const int use_shift = g.simt_ns ? 0 : 1;
  const int T = cdiv(d, SG_BM);
  const int parts = ns_parts(c);
  const NsControlParams ncp{c->at<SchedEntry>(c->L.sched), c->n_sched, c->n_lift_init, g.ns_max_steps, d, use_shift, g.orth_tol,
                            g.fro_tol, g.margin, g.lo_budget, 1.0 / (double)d};
  float* X = cur ? Xb : Xa;
  float* Xn = cur ? Xa : Xb;
  c->tc.ns_k = k;
  int rc = launch_residual(c, X, cur);
  if (rc) return rc;
  ns_control_kernel<<<P, 256, 0, c->stream>>>(st, pf, pd, use_shift ? pd + parts : nullptr, parts, k, cur, ncp);
  CQ_LAUNCHED(c, K_OTHER);
  if (last) return CONQUR_OK;
  if (g.simt_ns) {
    ns_gemm_exact_kernel<EPI_POLY><<<dim3(T, T, P), SG_THREADS, 0, c->stream>>>(E, E, E, B, d, st, nullptr, nullptr);
    CQ_LAUNCHED(c, K_NS_POLY);
    ns_gemm_exact_kernel<EPI_NEXT><<<dim3(T, T, P), SG_THREADS, 0, c->stream>>>(X, B, X, Xn, d, st, nullptr, nullptr);
    CQ_LAUNCHED(c, K_NS_NEXT);
    return CONQUR_OK;
  }
  return tc_ns_poly_next(c->tc, c->stream, cur);
}

int update_epilogue(conqur_ctx* c) {
  const Cfg& g = c->cfg;
  const int64_t dd = (int64_t)g.d * g.d;
  DevState* st = c->state();
  if (g.simt_ns) {
    ns_commit_kernel<<<dim3(ew_blocks(dd), g.P), 256, 0, c->stream>>>(st, c->at<float>(c->L.Xa), c->at<float>(c->L.Xb),
                                                                     c->at<float>(c->L.R), c->at<float>(c->L.M), dd);
    CQ_LAUNCHED(c, K_OTHER);
  } else {
    int rc = tc_ns_commit(c->tc, c->stream);
    if (rc) return rc;
  }
  if (g.mode == CONQUR_TC_BF16) { int rc = tc_refresh_R(c->tc, c->stream, /*only_if_converged=*/1); if (rc) return rc; }
  ns_commit_state_kernel<<<g.P, 32, 0, c->stream>>>(st, c->n_sched - 1);
  CQ_LAUNCHED(c, K_OTHER);
  c->tc.ns_k = -1;
  return CONQUR_OK;
}

int update_impl(conqur_ctx* c) {
  const Cfg& g = c->cfg;
  if (g.mode == CONQUR_TC_BF16 && g.P > 1) {
    // many small problems: the whole iteration of a problem runs inside one CTA
    const NsControlParams ncp{c->at<SchedEntry>(c->L.sched), c->n_sched, c->n_lift_init, g.ns_max_steps, g.d, 1,
                              g.orth_tol, g.fro_tol, g.margin, g.lo_budget, 1.0 / (double)g.d};
    return tcb_update(c->tc, c->stream, ncp, g.prior_rel, g.margin);
  }
  int rc = update_prologue(c);
  if (rc) return rc;
  for (int k = 0; k <= g.ns_max_steps; ++k) {
    rc = update_step(c, k, k & 1, k == g.ns_max_steps);
    if (rc) return rc;
  }
  rc = update_epilogue(c);
  if (rc) return rc;
  if (c->prof.enabled) {
    // profiling pass only: find out how many of the enqueued steps actually ran
    DevState h0;
    CQ_CUDA(cudaMemcpyAsync(&h0, c->state(), sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
    CQ_CUDA(cudaStreamSynchronize(c->stream));
    c->prof.fold(h0.ns_steps_used, h0.seg_log);
  }
  return CONQUR_OK;
}

// Ends one pass of the graph's loop body (two Newton-Schulz steps): go round again while the iteration is running.
// The pass counter bounds the loop whatever the data (the control kernel ends the iteration at ns_max_steps anyway).
__global__ void ns_loop_condition_kernel(DevState* st, cudaGraphConditionalHandle handle, int max_passes) {
  const int passes = ++st->loop_passes;
  st->loop_passes_total += 1;
  cudaGraphSetConditional(handle, (st->ns_done == 0 && passes < max_passes) ? 1u : 0u);
}

// The update as a graph: prologue, a WHILE node whose body is two steps (the iterate ping-pongs between two buffers,
// and the tensor maps of a launch are fixed) and the loop condition, epilogue.  Steps that the iteration does not
// need are then never launched.  Returns false if the driver cannot build it (the caller falls back to an unrolled capture).
bool build_looped_update_graph(conqur_ctx* c) {
  cudaGraph_t graph = nullptr;
  if (cudaGraphCreate(&graph, 0) != cudaSuccess) { cudaGetLastError(); return false; }
  cudaStream_t body_stream = nullptr;
  bool ok = false, capturing = false, capturing_body = false;
  cudaStream_t user = c->stream;
  long long before[K_COUNT], total_before = c->prof.total;
  for (int i = 0; i < K_COUNT; ++i) before[i] = c->prof.launches[i];
  do {
    cudaGraphConditionalHandle handle;
    if (cudaGraphConditionalHandleCreate(&handle, graph, 1, cudaGraphCondAssignDefault) != cudaSuccess) break;
    if (cudaStreamCreateWithFlags(&body_stream, cudaStreamNonBlocking) != cudaSuccess) break;
    if (cudaStreamBeginCaptureToGraph(c->cap_stream, graph, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal) != cudaSuccess) break;
    capturing = true;
    c->stream = c->cap_stream;
    if (update_prologue(c) != CONQUR_OK) break;
    cudaStreamCaptureStatus status;
    const cudaGraphNode_t* deps = nullptr;
    size_t n_deps = 0;
    if (cudaStreamGetCaptureInfo_v2(c->cap_stream, &status, nullptr, nullptr, &deps, &n_deps) != cudaSuccess) break;
    cudaGraphNodeParams np = {};
    np.type = cudaGraphNodeTypeConditional;
    np.conditional.handle = handle;
    np.conditional.type = cudaGraphCondTypeWhile;
    np.conditional.size = 1;
    cudaGraphNode_t loop_node;
    if (cudaGraphAddNode(&loop_node, graph, deps, n_deps, &np) != cudaSuccess) break;
    cudaGraph_t body = np.conditional.phGraph_out[0];
    // ---- the loop body, captured on a stream of its own into the node's graph
    for (int i = 0; i < K_COUNT; ++i) c->loop_body_launches[i] = -c->prof.launches[i];
    if (cudaStreamBeginCaptureToGraph(body_stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal) != cudaSuccess) break;
    capturing_body = true;
    c->stream = body_stream;
    if (update_step(c, -1, 0, false) != CONQUR_OK || update_step(c, -1, 1, false) != CONQUR_OK) break;
    ns_loop_condition_kernel<<<1, 1, 0, body_stream>>>(c->state(), handle, c->cfg.ns_max_steps / 2 + 2);
    if (cudaGetLastError() != cudaSuccess) break;
    c->prof.count(K_OTHER);
    cudaGraph_t body_out = nullptr;
    capturing_body = false;
    if (cudaStreamEndCapture(body_stream, &body_out) != cudaSuccess) break;
    for (int i = 0; i < K_COUNT; ++i) c->loop_body_launches[i] += c->prof.launches[i];
    // ---- what follows the loop
    c->stream = c->cap_stream;
    if (cudaStreamUpdateCaptureDependencies(c->cap_stream, &loop_node, 1, cudaStreamSetCaptureDependencies) != cudaSuccess) break;
    if (update_epilogue(c) != CONQUR_OK) break;
    cudaGraph_t out = nullptr;
    capturing = false;
    if (cudaStreamEndCapture(c->cap_stream, &out) != cudaSuccess) break;
    if (cudaGraphInstantiate(&c->upd_graph, graph, 0) != cudaSuccess) { c->upd_graph = nullptr; break; }
    ok = true;
  } while (false);
  c->stream = user;
  c->tc.ns_k = -1;
  cudaGraph_t junk = nullptr;
  if (capturing_body) cudaStreamEndCapture(body_stream, &junk);
  if (capturing) cudaStreamEndCapture(c->cap_stream, &junk);
  if (body_stream) cudaStreamDestroy(body_stream);
  cudaGraphDestroy(graph);
  cudaGetLastError();
  // launches of one replay outside the loop (the loop body's are added from the device's pass counter)
  for (int i = 0; i < K_COUNT; ++i) {
    c->graph_launches[i] = ok ? c->prof.launches[i] - before[i] - c->loop_body_launches[i] : 0;
    c->prof.launches[i] = before[i];
  }
  c->prof.total = total_before;
  c->looped = ok;
  return ok;
}

// Enqueue one update: directly the first time (kernel attributes get set), then through a captured graph.
int update_enqueue(conqur_ctx* c) {
  const bool no_graph = (c->cfg.debug_flags & CONQUR_DEBUG_NO_GRAPH) != 0;
  const bool eligible = !no_graph && c->cfg.mode == CONQUR_TC_BF16 && c->cfg.P == 1 && !c->prof.enabled;
  if (!eligible || c->updates_enqueued++ == 0) return update_impl(c);
  if (!c->upd_graph) {
    if (!c->cap_stream && cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) != cudaSuccess) {
      cudaGetLastError();
      return update_impl(c);
    }
    if (!build_looped_update_graph(c)) {
      // no conditional nodes: capture the unrolled sequence instead
      long long before[K_COUNT];
      for (int i = 0; i < K_COUNT; ++i) before[i] = c->prof.launches[i];
      const long long total_before = c->prof.total;
      if (cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        cudaGetLastError();
        return update_impl(c);
      }
      cudaStream_t user = c->stream;
      c->stream = c->cap_stream;
      const int rc = update_impl(c);
      c->stream = user;
      cudaGraph_t graph = nullptr;
      const cudaError_t e = cudaStreamEndCapture(c->cap_stream, &graph);
      for (int i = 0; i < K_COUNT; ++i) { c->graph_launches[i] = c->prof.launches[i] - before[i]; c->prof.launches[i] = before[i]; }
      c->prof.total = total_before;
      if (rc != CONQUR_OK || e != cudaSuccess || !graph ||
          cudaGraphInstantiate(&c->upd_graph, graph, 0) != cudaSuccess) {
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
        c->upd_graph = nullptr;
        c->updates_enqueued = -(1 << 30);          // stay on direct launches
        return update_impl(c);
      }
      cudaGraphDestroy(graph);
    }
  }
  CQ_CUDA(cudaGraphLaunch(c->upd_graph, c->stream));
  for (int i = 0; i < K_COUNT; ++i) { c->prof.launches[i] += c->graph_launches[i]; c->prof.total += c->graph_launches[i]; }
  return CONQUR_OK;
}

}  // namespace

// ================================================================== C ABI

extern "C" size_t conqur_workspace_bytes(int32_t d, const conqur_config* cfg) {
  Layout L;
  if (!make_layout(d, cfg, &L)) return 0;
  return L.total;
}

extern "C" int conqur_init(conqur_ctx** out, int32_t d, const conqur_config* cfg, void* workspace_dev,
                           size_t workspace_bytes, void* cuda_stream) {
  if (!out) return CONQUR_ERR_INVALID_ARG;
  *out = nullptr;
  Layout L;
  if (!make_layout(d, cfg, &L)) return CONQUR_ERR_INVALID_ARG;
  if (!workspace_dev || (reinterpret_cast<uintptr_t>(workspace_dev) % ALIGN) != 0) return CONQUR_ERR_INVALID_ARG;
  if (workspace_bytes < L.total) return CONQUR_ERR_WORKSPACE_TOO_SMALL;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    std::fprintf(stderr, "conqur: no CUDA device; there is no CPU fallback\n");
    return CONQUR_ERR_CUDA;
  }
  conqur_ctx* c = new (std::nothrow) conqur_ctx();
  if (!c) return CONQUR_ERR_INVALID_ARG;
  c->L = L;
  c->ws = static_cast<char*>(workspace_dev);
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->tokens.assign(cfg->batch, 0);
  c->last_n = 0;
  c->last_np = 0;
  Cfg& g = c->cfg;
  g.d = d; g.P = cfg->batch; g.in_dtype = cfg->in_dtype; g.mode = cfg->mode; g.quant_bits = cfg->quant_bits;
  g.n_max = cfg->n_max;
  g.defer = (g.mode == CONQUR_TC_BF16 && g.P == 1) ? std::max(1, cfg->defer_batches) : 1;
  g.debug_flags = cfg->debug_flags;
  g.qs = QuantSpec{cfg->quant_bits, cfg->quant_mode, cfg->clip_ratio > 0.f ? cfg->clip_ratio : 1.0f};
  g.diagnostics = cfg->diagnostics;
  g.simt_ns = (g.mode == CONQUR_EXACT_F32);
  g.ns_max_steps = cfg->ns_max_steps > 0 ? std::min(cfg->ns_max_steps, 120) : 0;   // 0: set from the schedule below
  g.orth_tol = cfg->orth_tol > 0.f ? cfg->orth_tol : 1e-4f;
  g.prior_rel = cfg->prior_rel;
  g.fro_tol = 0.1f;
  // bf16 products perturb the singular values by up to ~1e-3 per step, fp32 products by ~1e-6
  g.margin = g.simt_ns ? 1e-3f : 2e-2f;
  NsPlanParams pp;
  pp.l0 = cfg->ns_sigma_min_rel > 0.f ? cfg->ns_sigma_min_rel : 1e-9;
  pp.margin = g.margin;
  pp.d = g.simt_ns ? 0 : d;
  pp.max_len = NS_SCHED_MAX;
  if (cfg->ns_lo_gap_budget > 0.f) pp.gap_budget = cfg->ns_lo_gap_budget;
  g.lo_budget = (float)pp.gap_budget;
  c->sched = plan_device_schedule(pp, &c->n_lift_init);
  c->n_sched = (int)c->sched.size();
  // ns_steps > 0: the caller's budget of steps; the lifting count starts from what the budget leaves after the endgame
  if (cfg->ns_steps > 0) c->n_lift_init = std::max(0, std::min(cfg->ns_steps, NS_SCHED_MAX) - (c->n_sched - 1));
  // generous: with the looped update graph steps that are not needed are never launched, and a lifting count learnt on
  // easy updates must leave room for a hard one
  if (g.ns_max_steps == 0) g.ns_max_steps = std::min(120, std::max(c->n_lift_init + c->n_sched - 1 + 12, 40));
  std::vector<SchedEntry> coef(NS_SCHED_MAX);
  for (int i = 0; i < NS_SCHED_MAX; ++i) {
    const NsStep& s = c->sched[std::min(i, c->n_sched - 1)];
    coef[i] = SchedEntry{(float)s.a, (float)s.b, (float)s.c, (float)s.l, s.lift, s.seg_x};
  }
  auto fail = [&](int rc) { delete c; return rc; };
  for (int i = 0; i < L.n_guards; ++i)
    if (cudaMemsetAsync(c->ws + L.guard[i], GUARD_PATTERN, GUARD_BYTES, c->stream) != cudaSuccess) return fail(CONQUR_ERR_CUDA);
  if (cudaMemsetAsync(c->ws, 0, sizeof(DevState) * g.P, c->stream) != cudaSuccess) return fail(CONQUR_ERR_CUDA);
  if (cudaMemsetAsync(c->ws + L.flags_agg, 0, sizeof(int) * 4, c->stream) != cudaSuccess) return fail(CONQUR_ERR_CUDA);
  if (cudaMemsetAsync(c->ws + L.M, 0, sizeof(float) * (size_t)d * d * g.P, c->stream) != cudaSuccess)
    return fail(CONQUR_ERR_CUDA);
  if (cudaMemcpyAsync(c->ws + L.sched, coef.data(), sizeof(SchedEntry) * NS_SCHED_MAX, cudaMemcpyHostToDevice,
                      c->stream) != cudaSuccess)
    return fail(CONQUR_ERR_CUDA);
  set_identity_kernel<<<ew_blocks((int64_t)d * d * g.P), 256, 0, c->stream>>>(c->at<float>(L.R), d, g.P);
  if (cudaGetLastError() != cudaSuccess) return fail(CONQUR_ERR_CUDA);
  if (g.mode == CONQUR_TC_BF16) {
    int rc = tc_init(&c->tc, c->ws, L.tc, d, g.P, L.n_rows, g.quant_bits, c->at<float>(L.R), c->at<float>(L.M),
                     c->at<float>(L.Xa), c->at<float>(L.Xb), c->at<float>(L.E), c->at<float>(L.B),
                     c->at<float>(L.rnorm), c->state(), c->at<double>(L.part_d), c->at<float>(L.part_f),
                     (cfg->quant_bits || cfg->diagnostics) ? c->at<float>(L.C) : nullptr, c->at<unsigned>(L.rowmax), g.qs,
                     g.diagnostics, g.diagnostics ? c->at<double>(L.part_diag) : nullptr, &c->prof,
                     (g.debug_flags & CONQUR_DEBUG_SINGLE_CTA) != 0, cfg->ns_gram_single_pass_tau, g.lo_budget);
    if (rc) return fail(rc);
    rc = tc_refresh_R(c->tc, c->stream, 0);
    if (rc) return fail(rc);
  }
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(CONQUR_ERR_CUDA);   // coef is a local
  *out = c;
  return CONQUR_OK;
}

extern "C" int conqur_destroy(conqur_ctx* ctx) {
  if (!ctx) return CONQUR_ERR_INVALID_ARG;
  cudaStreamSynchronize(ctx->stream);
  if (ctx->upd_graph) cudaGraphExecDestroy(ctx->upd_graph);
  if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
  delete ctx;
  return CONQUR_OK;
}

extern "C" int conqur_set_R(conqur_ctx* c, const float* R_dev) {
  if (!c || !R_dev) return CONQUR_ERR_INVALID_ARG;
  const Cfg& g = c->cfg;
  const int64_t dd = (int64_t)g.d * g.d;
  { const int frc = flush_pending(c); if (frc) return frc; }      // queued rows belong to the rotation being replaced
  // check orthogonality with the exact fp32 residual product, whatever the mode
  float* Xa = c->at<float>(c->L.Xa);
  CQ_CUDA(cudaMemcpyAsync(Xa, R_dev, sizeof(float) * dd * g.P, cudaMemcpyDeviceToDevice, c->stream));
  arm_check_kernel<<<1, 256, 0, c->stream>>>(c->state(), g.P);
  CQ_LAUNCHED(c, K_OTHER);
  const int T = cdiv(g.d, SG_BM);
  ns_gemm_exact_kernel<EPI_RESIDUAL><<<dim3(T, T, g.P), SG_THREADS, 0, c->stream>>>(
      Xa, Xa, nullptr, c->at<float>(c->L.E), g.d, c->state(), c->at<float>(c->L.part_f), c->at<double>(c->L.part_d));
  CQ_LAUNCHED(c, K_OTHER);
  std::vector<float> pm((size_t)T * T * g.P);
  CQ_CUDA(cudaMemcpyAsync(pm.data(), c->at<float>(c->L.part_f), sizeof(float) * pm.size(), cudaMemcpyDeviceToHost,
                          c->stream));
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  float mx = 0.f;
  for (float v : pm) mx = (v == v) ? std::max(mx, v) : INFINITY;
  if (!(mx <= 1e-3f)) return CONQUR_ERR_NOT_ORTHOGONAL_INPUT;
  CQ_CUDA(cudaMemcpyAsync(c->at<float>(c->L.R), R_dev, sizeof(float) * dd * g.P, cudaMemcpyDeviceToDevice, c->stream));
  if (g.mode == CONQUR_TC_BF16) return tc_refresh_R(c->tc, c->stream, 0);
  return CONQUR_OK;
}

static int step_common(conqur_ctx* c, const void* X, int64_t n, int64_t ld, int64_t pstride, int p0, int np) {
  if (!c || !X) return CONQUR_ERR_INVALID_ARG;
  const Cfg& g = c->cfg;
  if (n < 0 || n > g.n_max || ld < g.d || pstride < 0 || (np > 1 && pstride == 0)) return CONQUR_ERR_INVALID_ARG;
  if (p0 < 0 || np < 1 || p0 + np > g.P) return CONQUR_ERR_INVALID_ARG;
  if (n == 0) return CONQUR_OK;
  int rc;
  if (g.mode == CONQUR_EXACT_F32) {
    rc = (g.in_dtype == CONQUR_F32)
             ? step_exact<float>(c, static_cast<const float*>(X), n, ld, pstride, p0, np)
             : step_exact<__nv_bfloat16>(c, static_cast<const __nv_bfloat16*>(X), n, ld, pstride, p0, np);
  } else {
    if (g.P > 1 && c->sign_capture && (int64_t)np * n > c->sign_capture_rows) return CONQUR_ERR_INVALID_ARG;
    if (g.P > 1) {
      rc = tcb_step(c->tc, c->stream, X, g.in_dtype, n, ld, pstride, p0, np, c->sign_capture, c->heads_trace);
    } else {
      // stage the rows behind those already queued; run the products when the queue is full (at once if not deferring)
      if (c->pending_rows + n > c->L.n_rows) { rc = flush_pending(c); if (rc) return rc; }
      rc = tc_stage(c->tc, c->stream, X, g.in_dtype, n, ld, c->pending_rows);
      if (rc == CONQUR_OK) {
        c->pending_rows += n;
        if (++c->pending_batches >= g.defer) rc = flush_pending(c);
      }
    }
  }
  if (rc == CONQUR_OK) {
    for (int p = p0; p < p0 + np; ++p) c->tokens[p] += n;
    if (!(g.mode == CONQUR_TC_BF16 && g.P == 1)) c->last_n = n;      // (set by flush_pending for queueing contexts)
    c->last_np = np;
  }
  return rc;
}

extern "C" int conqur_step(conqur_ctx* c, const void* X_dev, int64_t n, int64_t ld) {
  if (!c || c->cfg.P != 1) return CONQUR_ERR_INVALID_ARG;
  return step_common(c, X_dev, n, ld, 0, 0, 1);
}

extern "C" int conqur_step_batched(conqur_ctx* c, const void* X_dev, int64_t n, int64_t ld, int64_t problem_stride) {
  if (!c) return CONQUR_ERR_INVALID_ARG;
  return step_common(c, X_dev, n, ld, problem_stride, 0, c->cfg.P);
}

extern "C" int conqur_step_batched_range(conqur_ctx* c, const void* X_dev, int64_t n, int64_t ld, int64_t problem_stride,
                                         int32_t first_problem, int32_t n_problems) {
  if (!c) return CONQUR_ERR_INVALID_ARG;
  return step_common(c, X_dev, n, ld, problem_stride, first_problem, n_problems);
}

extern "C" int conqur_update(conqur_ctx* c) {
  if (!c) return CONQUR_ERR_INVALID_ARG;
  const int64_t fewest = *std::min_element(c->tokens.begin(), c->tokens.end());     // every problem is updated
  if (fewest == 0) return CONQUR_ERR_EMPTY_UPDATE;
  if (fewest < c->cfg.d && c->cfg.prior_rel == 0.f) return CONQUR_ERR_RANK_DEFICIENT;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const int rc = update_enqueue(c);
  if (rc == CONQUR_OK) {
    c->tokens_at_update = c->tokens;
    std::fill(c->tokens.begin(), c->tokens.end(), 0);
  }
  return rc;
}

extern "C" int conqur_get_R(conqur_ctx* c, float* R_out_dev) {
  if (!c || !R_out_dev) return CONQUR_ERR_INVALID_ARG;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const size_t bytes = sizeof(float) * (size_t)c->cfg.d * c->cfg.d * c->cfg.P;
  CQ_CUDA(cudaMemcpyAsync(R_out_dev, c->at<float>(c->L.R), bytes, cudaMemcpyDeviceToDevice, c->stream));
  return sync_status(c);
}

extern "C" int conqur_get_objective(conqur_ctx* c, double* J_sum, int64_t* n_tokens) {
  if (!c || !J_sum || !n_tokens) return CONQUR_ERR_INVALID_ARG;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const int P = c->cfg.P;
  if (c->cfg.mode == CONQUR_TC_BF16) { const int orc = tcb_refresh_objective(c->tc, c->stream); if (orc) return orc; }
  std::vector<DevState> h(P);
  CQ_CUDA(cudaMemcpyAsync(h.data(), c->state(), sizeof(DevState) * P, cudaMemcpyDeviceToHost, c->stream));
  const int rc = sync_status(c);
  for (int p = 0; p < P; ++p) { J_sum[p] = h[p].J; n_tokens[p] = h[p].N; }
  return rc;
}

extern "C" int conqur_get_objective_async(conqur_ctx* c, double* J_sum_host, int64_t* n_tokens_host) {
  if (!c || !J_sum_host || !n_tokens_host) return CONQUR_ERR_INVALID_ARG;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const int P = c->cfg.P;
  if (c->cfg.mode == CONQUR_TC_BF16) { const int orc = tcb_refresh_objective(c->tc, c->stream); if (orc) return orc; }
  double* dJ = c->at<double>(c->L.obj_out);
  long long* dN = reinterpret_cast<long long*>(dJ + P);
  export_sums_kernel<<<1, 256, 0, c->stream>>>(c->state(), dJ, dN, P);
  CQ_LAUNCHED(c, K_OTHER);
  CQ_CUDA(cudaMemcpyAsync(J_sum_host, dJ, sizeof(double) * P, cudaMemcpyDeviceToHost, c->stream));
  CQ_CUDA(cudaMemcpyAsync(n_tokens_host, dN, sizeof(long long) * P, cudaMemcpyDeviceToHost, c->stream));
  return CONQUR_OK;
}

extern "C" int conqur_get_diagnostics(conqur_ctx* c, conqur_diagnostics* out) {
  if (!c || !out || !c->cfg.diagnostics) return CONQUR_ERR_INVALID_ARG;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const int P = c->cfg.P;
  for (int p = 0; p < P; ++p)
    if (out[p].struct_size != sizeof(conqur_diagnostics)) return CONQUR_ERR_INVALID_ARG;
  std::vector<DevState> h(P);
  CQ_CUDA(cudaMemcpyAsync(h.data(), c->state(), sizeof(DevState) * P, cudaMemcpyDeviceToHost, c->stream));
  const int rc = sync_status(c);
  for (int p = 0; p < P; ++p) {
    out[p].sum_pr_over_d = h[p].diag_pr; out[p].sum_rho = h[p].diag_rho;
    out[p].qerr_num = h[p].diag_qnum; out[p].qerr_den = h[p].diag_qden; out[p].n_tokens = h[p].N;
  }
  return rc;
}

extern "C" int conqur_get_M(conqur_ctx* c, float* M_out_dev) {
  if (!c || !M_out_dev) return CONQUR_ERR_INVALID_ARG;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const int64_t count = (int64_t)c->cfg.d * c->cfg.d * c->cfg.P;
  scale_copy_kernel<<<ew_blocks(count), 256, 0, c->stream>>>(c->at<float>(c->L.M), M_out_dev, count,
                                                             (float)(1.0 / std::sqrt((double)c->cfg.d)));
  CQ_LAUNCHED(c, K_OTHER);
  return sync_status(c);
}

extern "C" int conqur_set_M(conqur_ctx* c, const float* M_dev, const double* J_sum, const int64_t* n_tokens) {
  if (!c || !M_dev || !J_sum || !n_tokens) return CONQUR_ERR_INVALID_ARG;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const int P = c->cfg.P;
  const int64_t count = (int64_t)c->cfg.d * c->cfg.d * P;
  scale_copy_kernel<<<ew_blocks(count), 256, 0, c->stream>>>(M_dev, c->at<float>(c->L.M), count,
                                                             (float)std::sqrt((double)c->cfg.d));
  CQ_LAUNCHED(c, K_OTHER);
  // stage the sums through the partials buffer
  double* dJ = c->at<double>(c->L.part_d);
  long long* dN = reinterpret_cast<long long*>(dJ + P);
  std::vector<long long> n64(n_tokens, n_tokens + P);
  CQ_CUDA(cudaMemcpyAsync(dJ, J_sum, sizeof(double) * P, cudaMemcpyHostToDevice, c->stream));
  CQ_CUDA(cudaMemcpyAsync(dN, n64.data(), sizeof(long long) * P, cudaMemcpyHostToDevice, c->stream));
  set_sums_kernel<<<1, 256, 0, c->stream>>>(c->state(), dJ, dN, P);
  CQ_LAUNCHED(c, K_OTHER);
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  for (int p = 0; p < P; ++p) c->tokens[p] = n_tokens[p];
  return CONQUR_OK;
}

extern "C" int conqur_debug_get_signs(conqur_ctx* c, int8_t* S_out_dev, int64_t capacity_rows) {
  if (!c || !S_out_dev) return CONQUR_ERR_INVALID_ARG;
  const Cfg& g = c->cfg;
  if (g.mode == CONQUR_TC_BF16 && g.P > 1) return CONQUR_ERR_UNSUPPORTED;     // nothing of a fused step stays in memory
  { const int frc = flush_pending(c); if (frc) return frc; }
  if (c->last_n == 0 || c->last_np == 0) return CONQUR_ERR_INVALID_ARG;
  if (capacity_rows < c->last_n * c->last_np) return CONQUR_ERR_INVALID_ARG;
  const int64_t total = c->last_n * g.d;
  const dim3 grid(ew_blocks(total), c->last_np);
  if (g.mode == CONQUR_EXACT_F32) {
    signs_from_c_kernel<<<grid, 256, 0, c->stream>>>(c->at<float>(c->L.C), nullptr, c->last_n, g.d, (int64_t)g.n_max * g.d,
                                                     S_out_dev);
  } else {
    signs_from_c_kernel<<<grid, 256, 0, c->stream>>>(nullptr, tc_cp_ptr(c->tc), c->last_n, g.d, 0, S_out_dev);
  }
  CQ_LAUNCHED(c, K_OTHER);
  return sync_status(c);
}

extern "C" int conqur_debug_capture_signs(conqur_ctx* c, int8_t* S_dev, int64_t capacity_rows) {
  if (!c || capacity_rows < 0 || (S_dev && capacity_rows == 0)) return CONQUR_ERR_INVALID_ARG;
  if (c->cfg.mode != CONQUR_TC_BF16 || c->cfg.P == 1) return CONQUR_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(S_dev) & 15) return CONQUR_ERR_INVALID_ARG;
  CQ_CUDA(cudaStreamSynchronize(c->stream));           // no step in flight still writes to the previous buffer
  c->sign_capture = S_dev;
  c->sign_capture_rows = S_dev ? capacity_rows : 0;
  return CONQUR_OK;
}

extern "C" int conqur_debug_trace_heads(conqur_ctx* c, int64_t* trace_dev, int64_t capacity) {
  if (!c || capacity < 0) return CONQUR_ERR_INVALID_ARG;
  if (c->cfg.mode != CONQUR_TC_BF16 || c->cfg.P == 1) return CONQUR_ERR_UNSUPPORTED;
  if (trace_dev && capacity < (int64_t)TCB_TRACE_TILES * 16) return CONQUR_ERR_INVALID_ARG;
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  c->heads_trace = reinterpret_cast<long long*>(trace_dev);
  return CONQUR_OK;
}

extern "C" int conqur_debug_check_canaries(conqur_ctx* c) {
  if (!c || !(c->cfg.debug_flags & CONQUR_DEBUG_CANARIES) || c->L.n_guards == 0) return CONQUR_ERR_INVALID_ARG;
  GuardList gl;
  gl.n = c->L.n_guards;
  for (int i = 0; i < gl.n; ++i) gl.off[i] = c->L.guard[i];
  int* bad = c->at<int>(c->L.flags_agg) + 1;
  CQ_CUDA(cudaMemsetAsync(bad, 0, sizeof(int), c->stream));
  check_guards_kernel<<<gl.n, (int)GUARD_BYTES, 0, c->stream>>>(reinterpret_cast<const unsigned char*>(c->ws), gl, bad);
  CQ_LAUNCHED(c, K_OTHER);
  int h = 0;
  CQ_CUDA(cudaMemcpyAsync(&h, bad, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  return h;
}

extern "C" int conqur_get_stats(conqur_ctx* c, conqur_stats* out) {
  if (!c || !out || out->struct_size != sizeof(conqur_stats)) return CONQUR_ERR_INVALID_ARG;
  { const int frc = flush_pending(c); if (frc) return frc; }
  const int P = c->cfg.P;
  std::vector<DevState> h(P);
  CQ_CUDA(cudaMemcpyAsync(h.data(), c->state(), sizeof(DevState) * P, cudaMemcpyDeviceToHost, c->stream));
  const int rc = sync_status(c);
  if (rc == CONQUR_ERR_CUDA) return rc;
  if (rc == CONQUR_ERR_NS_NOT_CONVERGED && !c->tokens_at_update.empty()) {
    // the device kept M, J and N of the rejected update: the host's row counts go back to match
    for (size_t p = 0; p < c->tokens.size(); ++p) c->tokens[p] += c->tokens_at_update[p];
    c->tokens_at_update.clear();
  }
  clear_flags_kernel<<<1, 256, 0, c->stream>>>(c->state(), P, c->at<int>(c->L.flags_agg));
  CQ_LAUNCHED(c, K_OTHER);
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  out->status = rc;
  out->ns_steps_used = 0; out->orth_err = 0.f; out->orth_fro = 0.f; out->n_skipped = 0;
  out->last_J = 0.0; out->last_N = 0; out->ns_lift_plan = 0; out->reserved = 0;
  out->updates = h[0].updates; out->scale = h[0].scale;
  for (int p = 0; p < P; ++p) {
    out->ns_steps_used = std::max(out->ns_steps_used, h[p].ns_steps_used);
    out->orth_err = std::max(out->orth_err, h[p].last_orth);
    out->orth_fro = std::max(out->orth_fro, h[p].last_fro);
    out->n_skipped += h[p].n_skipped;
    out->last_J += h[p].last_J;
    out->last_N += h[p].last_N;
    out->updates = std::min(out->updates, h[p].updates);
    out->ns_lift_plan = std::max(out->ns_lift_plan, h[p].lift_init ? h[p].lift_plan : c->n_lift_init);
  }
  return CONQUR_OK;
}

// The launches inside the update graph's loop: passes counted on the device x launches per pass (after a synchronise).
static int fold_loop_launches(conqur_ctx* c) {
  if (!c->looped) return CONQUR_OK;
  DevState h0;
  CQ_CUDA(cudaMemcpy(&h0, c->state(), sizeof(DevState), cudaMemcpyDeviceToHost));
  const long long fresh = h0.loop_passes_total - c->loop_passes_seen;
  c->loop_passes_seen = h0.loop_passes_total;
  for (int i = 0; i < K_COUNT; ++i) { c->prof.launches[i] += fresh * c->loop_body_launches[i]; c->prof.total += fresh * c->loop_body_launches[i]; }
  return CONQUR_OK;
}

extern "C" int conqur_set_profiling(conqur_ctx* c, int32_t enabled) {
  if (!c) return CONQUR_ERR_INVALID_ARG;
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  { const int lrc = fold_loop_launches(c); if (lrc) return lrc; }
  c->prof.fold(1 << 30);
  c->prof.reset();
  c->prof.enabled = enabled != 0;
  return CONQUR_OK;
}

extern "C" int conqur_get_profile(conqur_ctx* c, conqur_profile* out) {
  if (!c || !out || out->struct_size != sizeof(conqur_profile)) return CONQUR_ERR_INVALID_ARG;
  CQ_CUDA(cudaStreamSynchronize(c->stream));
  c->prof.fold(1 << 30);
  { const int lrc = fold_loop_launches(c); if (lrc) return lrc; }
  for (int i = 0; i < CONQUR_KERNEL_CLASSES; ++i) {
    out->launches[i] = c->prof.launches[i];
    out->timed_launches[i] = c->prof.timed[i];
    out->flops[i] = c->prof.flops[i];
    out->ms[i] = c->prof.ms[i];
  }
  out->total_launches = c->prof.total;
  return CONQUR_OK;
}

extern "C" int conqur_plan_schedule(double sigma_min_rel, int32_t ns_steps, double* abc_out, int32_t max_steps) {
  if (!abc_out || max_steps < 1 || sigma_min_rel < 0.0 || sigma_min_rel >= 1.0 || ns_steps < 0)
    return CONQUR_ERR_INVALID_ARG;
  NsPlanParams pp;
  pp.l0 = sigma_min_rel > 0.0 ? sigma_min_rel : 1e-9;
  const std::vector<NsStep> s = ns_steps > 0 ? plan_schedule_for_steps(ns_steps, pp) : plan_schedule(pp);
  const int n = std::min<int>((int)s.size(), max_steps);
  for (int i = 0; i < n; ++i) { abc_out[3 * i] = s[i].a; abc_out[3 * i + 1] = s[i].b; abc_out[3 * i + 2] = s[i].c; }
  return n;
}

extern "C" int conqur_debug_gemm(const void* A_dev, const void* B_dev, float* D_dev, int32_t M, int32_t N, int32_t K,
                                 int32_t a_mn_major, int32_t b_mn_major, int32_t split, void* scratch_dev,
                                 void* cuda_stream) {
  if (!A_dev || !B_dev || !D_dev || !scratch_dev) return CONQUR_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  CQ_CUDA(cudaMemsetAsync(scratch_dev, 0, sizeof(DevState), s));
  int rc = tc_plain_gemm(static_cast<const __nv_bfloat16*>(A_dev), static_cast<const __nv_bfloat16*>(B_dev), D_dev, M,
                         N, K, a_mn_major, b_mn_major, split, static_cast<DevState*>(scratch_dev), s);
  if (rc) return rc;
  DevState h;
  CQ_CUDA(cudaMemcpyAsync(&h, scratch_dev, sizeof(DevState), cudaMemcpyDeviceToHost, s));
  CQ_CUDA(cudaStreamSynchronize(s));
  return flags_to_status(h.status_flags);
}

extern "C" int conqur_debug_wait_timeout(void* scratch_dev, int64_t limit_cycles, void* cuda_stream) {
  if (!scratch_dev || limit_cycles < 1 || limit_cycles > 2000000000ll) return CONQUR_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  CQ_CUDA(cudaMemsetAsync(scratch_dev, 0, sizeof(DevState), s));
  tc_wait_probe_kernel<<<1, 32, 0, s>>>(static_cast<DevState*>(scratch_dev), (long long)limit_cycles);
  CQ_CUDA(cudaGetLastError());
  DevState h;
  CQ_CUDA(cudaMemcpyAsync(&h, scratch_dev, sizeof(DevState), cudaMemcpyDeviceToHost, s));
  CQ_CUDA(cudaStreamSynchronize(s));
  return flags_to_status(h.status_flags);
}

// ---------------------------------------------------------------- Appendix A: weight folding, online Hadamard
namespace {
bool fold_args_ok(int64_t ldw, int32_t rows, int32_t cols, int32_t block, int32_t side, int64_t ldo) {
  if (rows < 1 || cols < 1 || block < 1 || ldw < cols || ldo < cols) return false;
  if (side == CONQUR_FOLD_INPUT) return cols % block == 0;
  if (side == CONQUR_FOLD_OUTPUT) return rows % block == 0;
  return false;
}
// the tensor-core route: one full rotation, sizes the stand-alone product accepts
bool fold_tc_shape(int32_t rows, int32_t cols, int32_t block, int32_t side) {
  const int d = block;
  if (d % 128) return false;
  return side == CONQUR_FOLD_INPUT ? (cols == d && rows % 8 == 0) : (rows == d && cols % 32 == 0);
}
}  // namespace

extern "C" int64_t conqur_fold_scratch_bytes(int32_t rows, int32_t cols, int32_t block, int32_t side, int32_t mode) {
  if (!fold_args_ok(cols, rows, cols, block, side, cols)) return -1;
  if (mode == CONQUR_EXACT_F32) return 512;
  if (mode != CONQUR_TC_BF16) return -1;
  if (!fold_tc_shape(rows, cols, block, side)) return 512;          // block-diagonal folds run on the fp32 kernel
  return (int64_t)(512 + align_up((size_t)rows * cols * 4) + align_up((size_t)block * block * 4));
}

extern "C" int conqur_fold_weight(const float* W_dev, int64_t ldw, int32_t rows, int32_t cols, const float* R_dev,
                                  int32_t block, int32_t side, int32_t mode, float* out_dev, int64_t ldo,
                                  void* scratch_dev, int64_t scratch_bytes, void* cuda_stream) {
  if (!W_dev || !R_dev || !out_dev || !scratch_dev || W_dev == out_dev) return CONQUR_ERR_INVALID_ARG;
  if (!fold_args_ok(ldw, rows, cols, block, side, ldo)) return CONQUR_ERR_INVALID_ARG;
  if (mode != CONQUR_EXACT_F32 && mode != CONQUR_TC_BF16) return CONQUR_ERR_INVALID_ARG;
  const int64_t need = conqur_fold_scratch_bytes(rows, cols, block, side, mode);
  if (need < 0) return CONQUR_ERR_INVALID_ARG;
  if (scratch_bytes < need) return CONQUR_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const int nblk = (side == CONQUR_FOLD_INPUT ? cols : rows) / block;
  if (mode == CONQUR_TC_BF16 && nblk == 1) {
    if (!fold_tc_shape(rows, cols, block, side)) return CONQUR_ERR_UNSUPPORTED;
    if ((ldw % 4) || (ldo % 4) || (reinterpret_cast<uintptr_t>(W_dev) & 15) || (reinterpret_cast<uintptr_t>(out_dev) & 15) ||
        (reinterpret_cast<uintptr_t>(R_dev) & 15) || (reinterpret_cast<uintptr_t>(scratch_dev) & 255))
      return CONQUR_ERR_INVALID_ARG;
    const int d = block;
    uint8_t* base = static_cast<uint8_t*>(scratch_dev);
    DevState* st = reinterpret_cast<DevState*>(base);
    __nv_bfloat16* Ws = reinterpret_cast<__nv_bfloat16*>(base + 512);
    __nv_bfloat16* Rs = reinterpret_cast<__nv_bfloat16*>(base + 512 + align_up((size_t)rows * cols * 4));
    CQ_CUDA(cudaMemsetAsync(st, 0, sizeof(DevState), s));
    split_bf16_2d_kernel<<<ew_blocks((int64_t)rows * cols / 4), 256, 0, s>>>(W_dev, ldw, rows, cols, Ws);
    CQ_LAUNCH_CHECK();
    split_bf16_2d_kernel<<<ew_blocks((int64_t)d * d / 4), 256, 0, s>>>(R_dev, d, d, d, Rs);
    CQ_LAUNCH_CHECK();
    int rc;
    if (side == CONQUR_FOLD_INPUT)     // out (rows x d) = W R: A = W, K-major; B(n, k) = R[k][n], MN-major
      rc = tc_plain_gemm(Ws, Rs, out_dev, rows, d, d, 0, 1, 1, st, s, ldo);
    else                               // out (d x cols) = R^T W: A(m, k) = R[k][m] and B(n, k) = W[k][n], both MN-major
      rc = tc_plain_gemm(Rs, Ws, out_dev, d, cols, d, 1, 1, 1, st, s, ldo);
    if (rc) return rc;
    DevState h;
    CQ_CUDA(cudaMemcpyAsync(&h, st, sizeof(DevState), cudaMemcpyDeviceToHost, s));
    CQ_CUDA(cudaStreamSynchronize(s));
    return flags_to_status(h.status_flags);
  }
  if (side == CONQUR_FOLD_INPUT) {
    const dim3 grid(cdiv(block, SG_BN), cdiv(rows, SG_BM), nblk);
    fold_exact_kernel<0><<<grid, SG_THREADS, 0, s>>>(W_dev, ldw, R_dev, block, rows, cols, out_dev, ldo);
  } else {
    const dim3 grid(cdiv(cols, SG_BN), cdiv(block, SG_BM), nblk);
    fold_exact_kernel<1><<<grid, SG_THREADS, 0, s>>>(W_dev, ldw, R_dev, block, rows, cols, out_dev, ldo);
  }
  CQ_LAUNCH_CHECK();
  CQ_CUDA(cudaStreamSynchronize(s));
  return CONQUR_OK;
}

extern "C" int conqur_hadamard_rows(const void* X_dev, int32_t in_dtype, int64_t n, int32_t d, int64_t ldx, void* Y_dev,
                                    int32_t out_dtype, int64_t ldy, int32_t flags, void* cuda_stream) {
  if (flags & ~CONQUR_HADAMARD_CUDA_CORES_ONLY) return CONQUR_ERR_INVALID_ARG;
  if (n < 0 || d < 4 || d > 8192 || (d & (d - 1)) || ldx < d || ldy < d) return CONQUR_ERR_INVALID_ARG;
  if (n > 0 && (!X_dev || !Y_dev)) return CONQUR_ERR_INVALID_ARG;
  if ((in_dtype != CONQUR_F32 && in_dtype != CONQUR_BF16) || (out_dtype != CONQUR_F32 && out_dtype != CONQUR_BF16))
    return CONQUR_ERR_INVALID_ARG;
  // 4-element vector accesses
  const uintptr_t am = (in_dtype == CONQUR_F32) ? 15 : 7, bm = (out_dtype == CONQUR_F32) ? 15 : 7;
  if ((ldx % 4) || (ldy % 4) || (reinterpret_cast<uintptr_t>(X_dev) & am) || (reinterpret_cast<uintptr_t>(Y_dev) & bm))
    return CONQUR_ERR_INVALID_ARG;
  if (n == 0) return CONQUR_OK;
  int logd = 0;
  while ((1 << logd) < d) ++logd;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  using bf = __nv_bfloat16;
  // bf16 rows that lie back to back: the 128-point sub-transforms run on the tensor cores
  const bool simt_only = (flags & CONQUR_HADAMARD_CUDA_CORES_ONLY) != 0;
  if (!simt_only && in_dtype == CONQUR_BF16 && ldx == d && ldy == d && (reinterpret_cast<uintptr_t>(X_dev) & 15) == 0 &&
      (reinterpret_cast<uintptr_t>(Y_dev) & 15) == 0 && (n * d) % 128 == 0) {
    const int rc = (out_dtype == CONQUR_F32) ? hadamard_tc_launch(static_cast<const bf*>(X_dev), static_cast<float*>(Y_dev), n, logd, s)
                                             : hadamard_tc_launch(static_cast<const bf*>(X_dev), static_cast<bf*>(Y_dev), n, logd, s);
    if (rc != CONQUR_ERR_UNSUPPORTED) return rc;
  }
  if (in_dtype == CONQUR_F32 && out_dtype == CONQUR_F32)
    return hadamard_launch(static_cast<const float*>(X_dev), ldx, static_cast<float*>(Y_dev), ldy, n, logd, s);
  if (in_dtype == CONQUR_F32)
    return hadamard_launch(static_cast<const float*>(X_dev), ldx, static_cast<bf*>(Y_dev), ldy, n, logd, s);
  if (out_dtype == CONQUR_F32)
    return hadamard_launch(static_cast<const bf*>(X_dev), ldx, static_cast<float*>(Y_dev), ldy, n, logd, s);
  return hadamard_launch(static_cast<const bf*>(X_dev), ldx, static_cast<bf*>(Y_dev), ldy, n, logd, s);
}

extern "C" int conqur_hadamard_status(void* cuda_stream) {
  CQ_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
  int f = 0;
  CQ_CUDA(cudaMemcpyFromSymbol(&f, g_aux_status_flags, sizeof(int)));
  if (f) {
    const int zero = 0;
    CQ_CUDA(cudaMemcpyToSymbol(g_aux_status_flags, &zero, sizeof(int)));
  }
  return flags_to_status(f);
}

extern "C" const char* conqur_strerror(int s) {
  switch (s) {
    case CONQUR_OK: return "ok";
    case CONQUR_ERR_INVALID_ARG: return "invalid argument";
    case CONQUR_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CONQUR_ERR_NOT_ORTHOGONAL_INPUT: return "rotation passed to set_R is not orthogonal";
    case CONQUR_ERR_EMPTY_UPDATE: return "update with no accumulated tokens";
    case CONQUR_ERR_RANK_DEFICIENT: return "fewer tokens than dimensions and prior_rel == 0";
    case CONQUR_ERR_NS_NOT_CONVERGED: return "Newton-Schulz did not converge; previous rotation kept";
    case CONQUR_ERR_NONFINITE_INPUT: return "non-finite input row (skipped)";
    case CONQUR_ERR_TIMEOUT: return "bounded device-side wait expired";
    case CONQUR_ERR_CUDA: return "CUDA error";
    case CONQUR_ERR_UNSUPPORTED: return "unsupported configuration";
    default: return "unknown status";
  }
}
