// conqur_objective_noalloc: the corner objective of one batch with every byte of scratch taken from a
// fixed array inside the library image, for callers that are not allowed to allocate device memory.
//
// The regular path (conqur_step + conqur_get_objective) keeps its per-row norms and per-CTA partial sums
// in a caller-allocated workspace.  Some callers have no allocator to ask: code running inside a
// memory-pool-managed runtime that forbids raw cudaMalloc, or a plugin loaded into a process whose device
// memory is entirely pre-assigned.  This entry point serves them: same arithmetic as the exact (fp32)
// rotate/objective kernels, scratch from `g_scratch` below.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <mutex>

#include "../../include/conqur.h"
#include "conqur_internal.h"
#include "conqur_simt.cuh"

using namespace conqur;

namespace {

// Limits of the fixed scratch: rows per call, feature dimension, and the CTA grid they imply.
constexpr int NA_MAX_ROWS = 32768;
constexpr int NA_MAX_D = 8192;
constexpr int NA_MAX_PARTIALS = (NA_MAX_ROWS / SG_BM) * (NA_MAX_D / SG_BN);   // 16384

struct NaScratch {
  DevState state;                      // skip counters / status of the call in flight
  double partials[NA_MAX_PARTIALS];    // one objective partial per CTA
  float rnorm[NA_MAX_ROWS];            // 1 / ||x_i||
};

// Every GPU that loads the library holds this array (about 260 KB) until the process exits.
static __device__ __align__(256) unsigned char g_scratch[sizeof(NaScratch)];

// Host code must not pass `g_scratch` itself to a kernel: in host code that name is only a handle for
// the runtime.  The device address is looked up once per device and cached here.
constexpr int NA_MAX_DEVICES = 64;
NaScratch* g_dev_ptr[NA_MAX_DEVICES] = {nullptr};
std::mutex g_mu;

int scratch_for_current_device(NaScratch** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return CONQUR_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_dev_ptr[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_scratch);     // address on the CURRENT device
    if (e != cudaSuccess || !p) {
      std::fprintf(stderr, "conqur: cudaGetSymbolAddress(g_scratch): %s\n", cudaGetErrorString(e));
      return CONQUR_ERR_CUDA;
    }
    g_dev_ptr[dev] = static_cast<NaScratch*>(p);
  }
  *out = g_dev_ptr[dev];
  return CONQUR_OK;
}

// Y = X R on the CUDA cores (same main loop as the exact rotate kernel); nothing but the objective partial
// leaves the CTA: sum_ij |y_ij| * rnorm_i.
template <typename TIn>
__global__ void __launch_bounds__(SG_THREADS) na_objective_kernel(const TIn* __restrict__ X, int64_t ld,
                                                                  const float* __restrict__ R, int n, int d,
                                                                  const float* __restrict__ rnorm,
                                                                  double* __restrict__ partials) {
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  float acc[8][8];
  sg_mainloop<TIn, false, float, true>(X, ld, R, d, n, d, 0, d, m0, n0, acc);
  double asum = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + sg_row(i);
    if (row >= n) continue;
    const float r = rnorm[row];
    float rs = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (n0 + sg_col(j) < d) rs += fabsf(acc[i][j]);
    if (r > 0.f) asum += (double)(rs * r);
  }
  __shared__ double red[SG_THREADS / 32];
  const double tot = block_sum_d<SG_THREADS>(asum, red);
  if (threadIdx.x == 0) partials[(int64_t)blockIdx.y * gridDim.x + blockIdx.x] = tot;
}

__global__ void na_finalize_kernel(NaScratch* s, int nparts, int64_t n, double inv_sqrt_d, double* J_out,
                                   long long* N_out) {
  __shared__ double red[8];
  double v = 0.0;
  for (int i = threadIdx.x; i < nparts; i += 256) v += s->partials[i];
  const double tot = block_sum_d<256>(v, red);
  if (threadIdx.x == 0) {
    *J_out = tot * inv_sqrt_d;
    *N_out = n - s->state.step_skipped;
  }
}

}  // namespace

extern "C" int conqur_objective_noalloc(const void* X_dev, int32_t in_dtype, int64_t n, int32_t d, int64_t ld,
                                        const float* R_dev, double* J_out_dev, int64_t* N_out_dev,
                                        void* cuda_stream) {
  if (!X_dev || !R_dev || !J_out_dev || !N_out_dev) return CONQUR_ERR_INVALID_ARG;
  if (in_dtype != CONQUR_F32 && in_dtype != CONQUR_BF16) return CONQUR_ERR_INVALID_ARG;
  if (n < 1 || d < 2 || ld < d) return CONQUR_ERR_INVALID_ARG;
  if (n > NA_MAX_ROWS || d > NA_MAX_D) {
    std::fprintf(stderr, "conqur_objective_noalloc: n=%lld, d=%d exceed the fixed scratch (n <= %d, d <= %d)\n",
                 (long long)n, d, NA_MAX_ROWS, NA_MAX_D);
    return CONQUR_ERR_UNSUPPORTED;
  }
  NaScratch* s = nullptr;
  int rc = scratch_for_current_device(&s);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps the previous call's contents: the counters must start at zero
  if (cudaMemsetAsync(&s->state, 0, sizeof(DevState), st) != cudaSuccess) return CONQUR_ERR_CUDA;
  const dim3 rgrid((unsigned)((n + 7) / 8), 1);
  const dim3 grid((unsigned)((d + SG_BN - 1) / SG_BN), (unsigned)((n + SG_BM - 1) / SG_BM));
  if (in_dtype == CONQUR_F32) {
    rownorm_kernel<float><<<rgrid, 256, 0, st>>>(static_cast<const float*>(X_dev), n, d, ld, 0, s->rnorm, 0,
                                                 &s->state, 0);
    na_objective_kernel<float><<<grid, SG_THREADS, 0, st>>>(static_cast<const float*>(X_dev), ld, R_dev, (int)n, d,
                                                            s->rnorm, s->partials);
  } else {
    rownorm_kernel<__nv_bfloat16><<<rgrid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(X_dev), n, d, ld, 0,
                                                         s->rnorm, 0, &s->state, 0);
    na_objective_kernel<__nv_bfloat16><<<grid, SG_THREADS, 0, st>>>(static_cast<const __nv_bfloat16*>(X_dev), ld,
                                                                    R_dev, (int)n, d, s->rnorm, s->partials);
  }
  na_finalize_kernel<<<1, 256, 0, st>>>(s, (int)(grid.x * grid.y), n, 1.0 / std::sqrt((double)d), J_out_dev,
                                        reinterpret_cast<long long*>(N_out_dev));
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}
