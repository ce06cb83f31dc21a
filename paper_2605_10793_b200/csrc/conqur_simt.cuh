// fp32 CUDA-core kernels: the exact mode of every step of the path, and the
// reductions / element-wise passes both modes share.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "conqur_internal.h"

namespace conqur {

// ------------------------------------------------------------------ small helpers

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum in double, fixed order (lane tree, then warp 0 over the warp results).
template <int THREADS>
__device__ __forceinline__ double block_sum_d(double v, double* smem /* THREADS/32 */) {
  v = warp_sum_d(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) smem[w] = v;
  __syncthreads();
  double r = 0.0;
  if (w == 0) {
    r = (l < THREADS / 32) ? smem[l] : 0.0;
    r = warp_sum_d(r);
  }
  __syncthreads();
  return r;  // valid in warp 0
}
template <int THREADS>
__device__ __forceinline__ float block_max_f(float v, float* smem) {
  v = warp_max(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) smem[w] = v;
  __syncthreads();
  float r = 0.f;
  if (w == 0) {
    r = (l < THREADS / 32) ? smem[l] : 0.f;
    r = warp_max(r);
  }
  __syncthreads();
  return r;
}

__device__ __forceinline__ float ld_as_float(const float* p) { return *p; }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }

__device__ __forceinline__ void ld4_as_float(const float* p, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void ld4_as_float(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 t = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}

__device__ __forceinline__ float sgnf(float v) { return (v > 0.f) ? 1.f : ((v < 0.f) ? -1.f : 0.f); }

// Order-preserving map float -> unsigned, so that integer atomicMax / atomicMin give an exact, order-independent
// row maximum / minimum of signed values.
__device__ __forceinline__ unsigned f2ord(float f) {
  const unsigned b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord2f(unsigned u) { return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u); }

// Per-token fake-quantiser (Appendix B), as a rule "k = clamp(rint(y * inv), klo, khi); Q(y) = delta * k":
//   symmetric : delta = max|y| / (2^(b-1) - 1), k in [-(2^(b-1)-1), 2^(b-1)-1]
//   zero-point: delta = c (max y - min y) / (2^b - 1), zeta = -rint(c min y / delta), k = q - zeta in [-zeta, 2^b - 1 - zeta]
// (c = clipping ratio of Appendix C).  The same rule works on the un-normalised products (a positive row scale
// changes neither k nor zeta); the caller multiplies delta by the row's 1/norm.
struct QuantSpec { int bits, mode; float clip; };          // bits == 0: no fake-quantisation
struct RowQuant { float inv, delta, klo, khi; };
__device__ __forceinline__ RowQuant row_quant(const QuantSpec q, float vmax, float vmin, bool good) {
  RowQuant r{0.f, 0.f, 0.f, 0.f};
  if (q.mode == 0) {
    const float L = (float)((1 << (q.bits - 1)) - 1);
    const float mx = fmaxf(fabsf(vmax), fabsf(vmin));
    if (good && mx > 0.f) { r.inv = L / mx; r.delta = mx / L; r.klo = -L; r.khi = L; }
  } else {
    const float L = (float)((1 << q.bits) - 1);
    const float lo = q.clip * vmin, hi = q.clip * vmax;
    const float range = hi - lo;
    if (good && range > 0.f) {
      r.inv = L / range; r.delta = range / L;
      const float zeta = -rintf(lo * r.inv);
      r.klo = -zeta; r.khi = L - zeta;
    }
  }
  return r;
}

// ------------------------------------------------------------------ a1: row norms
// One warp per row: rnorm_i = 1/||x_i||_2 in fp32.  Rows whose sum of squares is zero
// or not finite get rnorm = 0 (they then contribute nothing anywhere) and are counted.
template <typename TIn>
__global__ void __launch_bounds__(256) rownorm_kernel(const TIn* __restrict__ X, int64_t n, int d, int64_t ld,
                                                      int64_t problem_stride, float* __restrict__ rnorm,
                                                      int64_t rnorm_stride, DevState* st, int state_stride_problems) {
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int p = blockIdx.y;
  if (row >= n) return;
  const TIn* x = X + (int64_t)p * problem_stride + row * ld;
  float ss = 0.f;
  const bool vec = ((d & 3) == 0) && ((reinterpret_cast<uintptr_t>(x) & (sizeof(TIn) * 4 - 1)) == 0);
  if (vec) {
    for (int k = lane * 4; k < d; k += 128) {
      float v[4];
      ld4_as_float(x + k, v);
      ss = fmaf(v[0], v[0], ss); ss = fmaf(v[1], v[1], ss); ss = fmaf(v[2], v[2], ss); ss = fmaf(v[3], v[3], ss);
    }
  } else {
    for (int k = lane; k < d; k += 32) {
      const float v = ld_as_float(x + k);
      ss = fmaf(v, v, ss);
    }
  }
  ss = warp_sum(ss);
  if (lane == 0) {
    float r = 0.f;
    DevState* s = st + (state_stride_problems ? p : 0);
    if (ss > 0.f && ss <= 3.0e38f) {
      r = 1.0f / sqrtf(ss);
    } else {
      atomicAdd(reinterpret_cast<unsigned long long*>(&s->step_skipped), 1ull);
      if (!(ss == 0.f)) atomicOr(&s->status_flags, STATUS_FLAG_NONFINITE);
    }
    rnorm[(int64_t)p * rnorm_stride + row] = r;
  }
}

// ------------------------------------------------------------------ generic SIMT GEMM main loop
// acc[i][j] = sum_k A(m_i, k) * B(k, n_j) over a 128 x 128 tile, BK = 16, 256 threads.
// A(m,k) lives at A[m*lda + k] (A_M_CONTIG = false) or A[k*lda + m] (true);
// B(k,n) lives at B[k*ldb + n] (B_N_CONTIG = true) or B[n*ldb + k] (false).
// Thread (tx, ty) owns rows {ty*4+i, 64+ty*4+i}, cols {tx*4+j, 64+tx*4+j}, i,j in 0..3.
constexpr int SG_BM = 128, SG_BN = 128, SG_BK = 16, SG_THREADS = 256, SG_PAD = 4;

// kmask (optional, MN_CONTIG only): rows k with kmask[k] == 0 are read as zeros (skipped tokens).
template <typename T, bool MN_CONTIG>
__device__ __forceinline__ void sg_load_tile(const T* __restrict__ P, int64_t ld, int mn0, int k0, int MN, int K,
                                             float (*S)[SG_BM + SG_PAD], const float* __restrict__ kmask = nullptr) {
  const int t = threadIdx.x;
  const bool aligned = ((ld & 3) == 0) && ((reinterpret_cast<uintptr_t>(P) & (sizeof(T) * 4 - 1)) == 0);
  if (MN_CONTIG) {
    // element (mn, k) at P[k*ld + mn]; 4 consecutive mn per thread
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int k = (t >> 5) + 8 * r;
      const int mn = (t & 31) * 4;
      float v[4] = {0.f, 0.f, 0.f, 0.f};
      const int gk = k0 + k, gmn = mn0 + mn;
      if (gk < K && (kmask == nullptr || kmask[gk] > 0.f)) {
        const T* src = P + (int64_t)gk * ld + gmn;
        if (aligned && gmn + 3 < MN && ((gmn & 3) == 0)) {
          ld4_as_float(src, v);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (gmn + j < MN) v[j] = ld_as_float(src + j);
        }
      }
      *reinterpret_cast<float4*>(&S[k][mn]) = make_float4(v[0], v[1], v[2], v[3]);
    }
  } else {
    // element (mn, k) at P[mn*ld + k]; 4 consecutive k per thread, stored transposed
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int mn = (t >> 2) + 64 * r;
      const int k = (t & 3) * 4;
      float v[4] = {0.f, 0.f, 0.f, 0.f};
      const int gk = k0 + k, gmn = mn0 + mn;
      if (gmn < MN) {
        const T* src = P + (int64_t)gmn * ld + gk;
        if (aligned && gk + 3 < K && ((gk & 3) == 0)) {
          ld4_as_float(src, v);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (gk + j < K) v[j] = ld_as_float(src + j);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) S[k + j][mn] = v[j];
    }
  }
}

template <typename TA, bool A_M_CONTIG, typename TB, bool B_N_CONTIG>
__device__ __forceinline__ void sg_mainloop(const TA* __restrict__ A, int64_t lda, const TB* __restrict__ B,
                                            int64_t ldb, int M, int N, int k_begin, int k_end, int m0, int n0,
                                            float (&acc)[8][8], const float* __restrict__ kmask = nullptr) {
  __shared__ __align__(16) float As[SG_BK][SG_BM + SG_PAD];
  __shared__ __align__(16) float Bs[SG_BK][SG_BN + SG_PAD];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  for (int k0 = k_begin; k0 < k_end; k0 += SG_BK) {
    sg_load_tile<TA, A_M_CONTIG>(A, lda, m0, k0, M, k_end, As, kmask);
    sg_load_tile<TB, B_N_CONTIG>(B, ldb, n0, k0, N, k_end, Bs);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SG_BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

__device__ __forceinline__ int sg_row(int i) { return ((threadIdx.x >> 4) * 4) + (i & 3) + ((i >> 2) * 64); }
__device__ __forceinline__ int sg_col(int j) { return ((threadIdx.x & 15) * 4) + (j & 3) + ((j >> 2) * 64); }

// ------------------------------------------------------------------ a2-a4 exact: Y = X R, target, objective
// grid (ceil(d/128), ceil(n/128), P).  Plain mode: writes C'[i][j] = sgn(y_ij) * rnorm_i (fp32) and one
// objective partial per CTA (sum |acc_ij| * rnorm_i).  Quant mode: writes the raw products Y and the
// per-row max |acc| (integer atomicMax on the bit pattern: exact and order independent).
template <typename TIn, bool QUANT>
__global__ void __launch_bounds__(SG_THREADS) rotate_target_exact_kernel(
    const TIn* __restrict__ X, int64_t ld, int64_t x_pstride, const float* __restrict__ R, int n, int d,
    const float* __restrict__ rnorm, int64_t rnorm_pstride, float* __restrict__ Cp /* n x d */,
    int64_t c_pstride, unsigned int* __restrict__ rowmax_ord, unsigned int* __restrict__ rowmin_ord,
    double* __restrict__ partials) {
  const int p = blockIdx.z;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  float acc[8][8];
  sg_mainloop<TIn, false, float, true>(X + (int64_t)p * x_pstride, ld, R + (int64_t)p * d * d, d, n, d, 0, d, m0,
                                        n0, acc);
  const float* rn = rnorm + (int64_t)p * rnorm_pstride;
  float* C = Cp + (int64_t)p * c_pstride;
  double asum = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + sg_row(i);
    if (row >= n) continue;
    const float r = rn[row];
    float rs = 0.f, rmax = -3.0e38f, rmin = 3.0e38f;
#pragma unroll
    for (int jh = 0; jh < 2; ++jh) {
      const int col = n0 + sg_col(jh * 4);
      float o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float v = acc[i][jh * 4 + j];
        if (QUANT) {
          o[j] = v;
          if (col + j < d) { rmax = fmaxf(rmax, v); rmin = fminf(rmin, v); }
        } else {
          o[j] = sgnf(v) * r;
          rs += fabsf(v);
        }
      }
      float* dst = C + (int64_t)row * d + col;
      if (col + 3 < d && ((d & 3) == 0)) {
        *reinterpret_cast<float4*>(dst) = make_float4(o[0], o[1], o[2], o[3]);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (col + j < d) dst[j] = o[j];
      }
    }
    if (QUANT) {
      if (r > 0.f) {
        atomicMax(rowmax_ord + (int64_t)p * rnorm_pstride + row, f2ord(rmax));
        atomicMin(rowmin_ord + (int64_t)p * rnorm_pstride + row, f2ord(rmin));
      }
    } else {
      if (r > 0.f) asum += (double)(rs * r);
    }
  }
  if (!QUANT) {
    __shared__ double red[SG_THREADS / 32];
    const double tot = block_sum_d<SG_THREADS>(asum, red);
    if (threadIdx.x == 0)
      partials[((int64_t)p * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = tot;
  }
}

// Quant mode, second pass (Appendix B, per token).  One warp per row: k = clamp(rint(acc * inv), klo, khi),
// C' = sgn(k) * rnorm, objective partial = rnorm * delta * sum_j |k_j|.  Works in place: Y and C' share the buffer.
// Per-row quantities of the second pass, shared by both modes.  `y` is the row's un-normalised product, r = 1/||x||.
//   k       code of the fake-quantiser (or y itself when bits == 0)
//   returns the target sign; accumulates the objective term and, if asked, the Section-4 diagnostics
struct RowDiag { float s2, s4, mx, qe; };       // sums over the row of yh^2, yh^4, max |yh|, (yh - Q(yh))^2 with yh = y r
__device__ __forceinline__ float second_pass_elem(float y, float r, const QuantSpec qs, const RowQuant rq, float& qsum,
                                                  bool diag, RowDiag& dg) {
  float k, qv;
  if (qs.bits == 0) { k = y; qv = y; }
  else { k = fminf(fmaxf(rintf(y * rq.inv), rq.klo), rq.khi); qv = k * rq.delta; }
  qsum += fabsf(k);
  if (diag) {
    const float yh = y * r, t2 = yh * yh, e = (y - qv) * r;
    dg.s2 += t2; dg.s4 = fmaf(t2, t2, dg.s4); dg.mx = fmaxf(dg.mx, fabsf(yh)); dg.qe = fmaf(e, e, dg.qe);
  }
  return sgnf(k);
}
// warp-reduce a row's diagnostics and turn them into the four per-row terms (valid in lane 0)
__device__ __forceinline__ void row_diag_terms(RowDiag dg, float r, int d, bool live, double (&out)[4]) {
  dg.s2 = warp_sum(dg.s2); dg.s4 = warp_sum(dg.s4); dg.qe = warp_sum(dg.qe); dg.mx = warp_max(dg.mx);
  out[0] = out[1] = out[2] = out[3] = 0.0;
  if (live && dg.s4 > 0.f) {
    out[0] = (double)dg.s2 * (double)dg.s2 / ((double)d * (double)dg.s4);     // PR / d
    out[1] = (double)dg.mx * (double)dg.mx / (double)dg.s2;                    // rho
    const double x2 = 1.0 / ((double)r * (double)r);                           // ||x||^2
    out[2] = (double)dg.qe * x2;                                               // ||y - Q(y)||^2, un-normalised
    out[3] = x2;
  }
}

// Second pass of the two-pass step (exact mode; Appendix B per token).  One warp per row; works in place: Y and C'
// share the buffer.  part_diag (optional): 4 arrays of per-block partial sums of the diagnostics.
static __global__ void __launch_bounds__(256) quant_target_kernel(float* __restrict__ YC, int64_t n, int d,
                                                           int64_t c_pstride, const float* __restrict__ rnorm,
                                                           int64_t rnorm_pstride,
                                                           const unsigned int* __restrict__ rowmax_ord,
                                                           const unsigned int* __restrict__ rowmin_ord, QuantSpec qs,
                                                           double* __restrict__ partials /* per block */,
                                                           double* __restrict__ part_diag) {
  const int p = blockIdx.y;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const bool diag = part_diag != nullptr;
  double contrib = 0.0, dterm[4] = {0.0, 0.0, 0.0, 0.0};
  if (row < n) {
    const float r = rnorm[(int64_t)p * rnorm_pstride + row];
    RowQuant rq{0.f, 1.f, 0.f, 0.f};
    if (qs.bits) rq = row_quant(qs, ord2f(rowmax_ord[(int64_t)p * rnorm_pstride + row]),
                                ord2f(rowmin_ord[(int64_t)p * rnorm_pstride + row]), r > 0.f);
    const bool live = qs.bits ? (rq.inv > 0.f) : (r > 0.f);
    float* y = YC + (int64_t)p * c_pstride + row * d;
    float qsum = 0.f;
    RowDiag dg{0.f, 0.f, 0.f, 0.f};
    for (int j = lane; j < d; j += 32) {
      const float sg = second_pass_elem(y[j], r, qs, rq, qsum, diag && live, dg);
      y[j] = live ? sg * r : 0.f;
    }
    qsum = warp_sum(qsum);
    if (live) contrib = (double)(r * rq.delta) * (double)qsum;
    if (diag) row_diag_terms(dg, r, d, live, dterm);
  }
  __shared__ double red[8][5];
  if (lane == 0) {
    red[threadIdx.x >> 5][0] = contrib;
    for (int k = 0; k < 4; ++k) red[threadIdx.x >> 5][1 + k] = dterm[k];
  }
  __syncthreads();
  if (threadIdx.x < 5) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += red[w][threadIdx.x];
    const int64_t nb = gridDim.x;
    if (threadIdx.x == 0) partials[(int64_t)p * nb + blockIdx.x] = t;
    else if (diag) part_diag[((int64_t)p * 4 + (threadIdx.x - 1)) * nb + blockIdx.x] = t;
  }
}

// ------------------------------------------------------------------ a5 exact: M_raw (+)= X^T C'
// grid (ceil(d/128), ceil(d/128), splits*P).  splits == 1: read-modify-write of M.  splits > 1: each
// split writes its own partial; splitk_reduce_add_kernel adds them to M in a fixed order.
template <typename TIn>
__global__ void __launch_bounds__(SG_THREADS) accumulate_exact_kernel(const TIn* __restrict__ X, int64_t ld,
                                                                      int64_t x_pstride,
                                                                      const float* __restrict__ Cp,
                                                                      int64_t c_pstride,
                                                                      const float* __restrict__ rnorm,
                                                                      int64_t rnorm_pstride, int n, int d,
                                                                      int splits,
                                                                      float* __restrict__ M,
                                                                      float* __restrict__ partial) {
  const int p = blockIdx.z / splits, s = blockIdx.z % splits;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  int chunk = (n + splits - 1) / splits;
  chunk = (chunk + SG_BK - 1) / SG_BK * SG_BK;
  const int kb = min(n, s * chunk), ke = min(n, kb + chunk);
  float acc[8][8];
  sg_mainloop<TIn, true, float, true>(X + (int64_t)p * x_pstride, ld, Cp + (int64_t)p * c_pstride, d, d, d, kb, ke,
                                       m0, n0, acc, rnorm + (int64_t)p * rnorm_pstride);
  float* dst = (splits == 1) ? (M + (int64_t)p * d * d) : (partial + ((int64_t)p * splits + s) * d * d);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + sg_row(i);
    if (row >= d) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int col = n0 + sg_col(j);
      if (col >= d) continue;
      float* q = dst + (int64_t)row * d + col;
      if (splits == 1) *q += acc[i][j]; else *q = acc[i][j];
    }
  }
}

static __global__ void splitk_reduce_add_kernel(float* __restrict__ M, const float* __restrict__ partial, int64_t dd,
                                         int splits) {
  const int p = blockIdx.y;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < dd; i += (int64_t)gridDim.x * blockDim.x) {
    float v = M[p * dd + i];
    for (int s = 0; s < splits; ++s) v += partial[((int64_t)p * splits + s) * dd + i];
    M[p * dd + i] = v;
  }
}

// Adds the step's objective partials (fixed order; none when `partials` is null) and token counts to the running sums.
static __global__ void finalize_step_kernel(DevState* st, const double* __restrict__ partials, int per_problem, int64_t n,
                                     double inv_sqrt_d, const double* __restrict__ part_diag = nullptr, int diag_blocks = 0) {
  const int p = blockIdx.x;
  __shared__ double red[8];
  double v = 0.0;
  if (partials)
    for (int i = threadIdx.x; i < per_problem; i += 256) v += partials[(int64_t)p * per_problem + i];
  const double tot = block_sum_d<256>(v, red);
  double dsum[4] = {0.0, 0.0, 0.0, 0.0};
  if (part_diag) {
    for (int k = 0; k < 4; ++k) {
      double w = 0.0;
      for (int i = threadIdx.x; i < diag_blocks; i += 256) w += part_diag[((int64_t)p * 4 + k) * diag_blocks + i];
      dsum[k] = block_sum_d<256>(w, red);
    }
  }
  if (threadIdx.x == 0) {
    DevState* s = st + p;
    s->J += tot * inv_sqrt_d;
    s->N += n - s->step_skipped;
    s->n_skipped += s->step_skipped;
    s->step_skipped = 0;
    if (part_diag) { s->diag_pr += dsum[0]; s->diag_rho += dsum[1]; s->diag_qnum += dsum[2]; s->diag_qden += dsum[3]; }
  }
}

// ------------------------------------------------------------------ a6/a7 exact: Newton-Schulz products
enum { EPI_RESIDUAL = 0, EPI_POLY = 1, EPI_NEXT = 2 };

// EPI_RESIDUAL: D = X^T X - I, plus per-CTA max|D| and sum D^2            (A = B = X, contraction over rows)
// EPI_POLY:     D = beta2 * (E E) + beta1 * E                             (A = B = Cin = E)
// EPI_NEXT:     D = X B + gamma * X                                       (A = Cin = X)
// All early-exit when the problem's iteration has finished.
template <int EPI>
__global__ void __launch_bounds__(SG_THREADS) ns_gemm_exact_kernel(const float* __restrict__ A,
                                                                   const float* __restrict__ B,
                                                                   const float* __restrict__ Cin,
                                                                   float* __restrict__ D, int d, DevState* st,
                                                                   float* __restrict__ part_max,
                                                                   double* __restrict__ part_sq) {
  const int p = blockIdx.z;
  const DevState* s = st + p;
  if (s->ns_done) return;
  const int64_t off = (int64_t)p * d * d;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  float acc[8][8];
  if constexpr (EPI == EPI_RESIDUAL)
    sg_mainloop<float, true, float, true>(A + off, d, B + off, d, d, d, 0, d, m0, n0, acc);
  else
    sg_mainloop<float, false, float, true>(A + off, d, B + off, d, d, d, 0, d, m0, n0, acc);
  const float c0 = s->coef[0], c1 = s->coef[1], c2 = s->coef[2];  // gamma, beta1, beta2
  float mx = 0.f;
  double sq = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + sg_row(i);
    if (row >= d) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int col = n0 + sg_col(j);
      if (col >= d) continue;
      const int64_t idx = off + (int64_t)row * d + col;
      float v = acc[i][j];
      if (EPI == EPI_RESIDUAL) {
        v -= (row == col) ? 1.f : 0.f;
        mx = fmaxf(mx, fabsf(v));
        sq += (double)v * (double)v;
      } else if (EPI == EPI_POLY) {
        v = fmaf(c2, v, c1 * Cin[idx]);
      } else {
        v = fmaf(c0, Cin[idx], v);
      }
      D[idx] = v;
    }
  }
  if (EPI == EPI_RESIDUAL) {
    __shared__ double redd[SG_THREADS / 32];
    __shared__ float redf[SG_THREADS / 32];
    const double tsq = block_sum_d<SG_THREADS>(sq, redd);
    const float tmx = block_max_f<SG_THREADS>(mx, redf);
    if (threadIdx.x == 0) {
      const int64_t slot = ((int64_t)p * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
      part_max[slot] = tmx;
      part_sq[slot] = tsq;
    }
  }
}

// ------------------------------------------------------------------ update: scalar control + element-wise
// sum of squares of M (optionally of M + lam*R) -> per-block double partials
static __global__ void __launch_bounds__(256) sumsq_kernel(const float* __restrict__ M, const float* __restrict__ R,
                                                    int64_t dd, const DevState* st, int use_lam,
                                                    double* __restrict__ partials) {
  const int p = blockIdx.y;
  const float lam = use_lam ? st[p].lam : 0.f;
  double v = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < dd; i += (int64_t)gridDim.x * 256) {
    float t = M[p * dd + i];
    if (use_lam) t = fmaf(lam, R[p * dd + i], t);
    v += (double)t * (double)t;
  }
  __shared__ double red[8];
  const double tot = block_sum_d<256>(v, red);
  if (threadIdx.x == 0) partials[(int64_t)p * gridDim.x + blockIdx.x] = tot;
}

// Arm the lifting phase of an update: the count learnt so far, or the planned one on a problem's first update.
__device__ __forceinline__ void ns_arm_lifting(DevState* s, int n_lift_init) {
  if (!s->lift_init) {
    s->lift_plan = n_lift_init; s->lift_succ = 0; s->lift_patience = 3; s->lift_trial = 0; s->lift_ema = 0.f;
    s->lift_init = 1;
  }
  s->lift_left = s->lift_plan;
  s->reentries = 0;
  s->loop_passes = 0;
  s->ns_idx = 1;                       // first endgame entry of the device schedule (entry 0 is the lifting quintic)
  s->growth = 1.0f;
}

// After an update: learn how many lifting steps the next one should start with.  The plan was lift_plan lifting +
// n_endgame endgame steps; an update that needed `extra` more ran them as the slower continuation of the endgame
// (nothing is lost but time).  Measured on streams of the workloads, steps(count) is count + n_endgame once the count
// suffices and erratic below (one lifting step short costs between nothing and five extra steps, depending on the
// matrix), and which count suffices wanders by one or two from update to update.  One lifting step more costs exactly
// one step per update, so the count that minimises the mean is the smallest whose mean shortfall stays below one:
//   * the running mean of `extra` at the current count (weight 1/4 on the newest) above 1: one step more (at once by
//     (extra + 1) / 2 when the count is far too short, extra >= 6);
//   * lift_patience updates in a row without an extra step and a mean below 1/4: try one step fewer.  If the mean
//     then exceeds 1 within the next 8 updates the descent did not pay: back up, and wait max(2, extra) times as
//     long before the next try.
// Before the first shortfall of a problem the count comes down by thirds per update (the planned count assumes a bound
// on the smallest singular value that is usually far too pessimistic); the first shortfall ends that phase.
__device__ __forceinline__ void ns_adapt_lift_plan(DevState* s, int n_endgame, int converged) {
  const int plan = s->lift_plan;
  if (!converged) {
    s->lift_plan = min(plan + 2, 60); s->lift_ema = 0.f; s->lift_succ = 0; s->lift_trial = 0;
    return;
  }
  const int extra = max(s->ns_steps_used - (plan + n_endgame), 0);
  s->lift_ema = 0.75f * s->lift_ema + 0.25f * (float)extra;
  s->lift_succ = extra == 0 ? s->lift_succ + 1 : 0;
  if (s->lift_init == 1) {
    // no update of this problem has fallen short yet: the planned count came from an assumed bound on the smallest
    // singular value, usually far too pessimistic; come down by thirds until one does
    // (lift_succ holds the last count that sufficed while this phase lasts)
    if (extra == 0) {
      s->lift_succ = plan;
      s->lift_plan = plan > 0 ? plan - max(1, (plan + 1) / 3) : 0;
      s->lift_ema = 0.f;
      return;
    }
    s->lift_init = 2;
    s->lift_plan = min(min(plan + max(1, (extra + 1) / 2), s->lift_succ > plan ? s->lift_succ : 60), 60);
    s->lift_ema = 0.f; s->lift_succ = 0;
    return;
  }
  const bool trial = s->lift_trial > 0;
  if (trial) s->lift_trial -= 1;
  if (s->lift_ema > 1.0f) {
    const int up = (trial || extra < 6) ? 1 : (extra + 1) / 2;
    s->lift_plan = min(plan + up, 60);
    s->lift_ema = 0.f; s->lift_succ = 0; s->lift_trial = 0;
    if (trial) s->lift_patience = min(128, s->lift_patience * max(2, extra));
  } else if (s->lift_succ >= s->lift_patience && s->lift_ema < 0.25f && plan > 0) {
    s->lift_plan = plan - 1;
    s->lift_ema = 0.f; s->lift_succ = 0; s->lift_trial = 8;
  }
}

// phase 0: lam = prior_rel * ||M_raw||_F / sqrt(d)      (reads partials of sumsq over M)
// phase 1: scale = ||M_raw + lam R||_F ; arms the iteration
static __global__ void ns_setup_kernel(DevState* st, const double* __restrict__ partials, int nblocks, int phase,
                                float prior_rel, float inv_sqrt_d, float margin, int d, int use_shift, float e1_tau,
                                int n_lift_init) {
  const int p = blockIdx.x;
  __shared__ double red[8];
  double v = 0.0;
  for (int i = threadIdx.x; i < nblocks; i += 256) v += partials[(int64_t)p * nblocks + i];
  const double tot = block_sum_d<256>(v, red);
  if (threadIdx.x == 0) {
    DevState* s = st + p;
    const float fro = (float)sqrt(tot);
    if (phase == 0) {
      s->lam = prior_rel * fro * inv_sqrt_d;
    } else {
      s->scale = fro;
      const bool ok = (fro > 0.f) && (fro <= 3.0e38f) && (s->N > 0);
      s->x0_scale = ok ? 1.0f / (fro * (1.0f + margin)) : 0.f;
      s->ns_done = ok ? 0 : NS_DONE_FAILED;
      s->ns_steps_used = 0;
      s->ns_final_buf = 0;
      ns_arm_lifting(s, n_lift_init);
      s->seg_x = 2;
      // ||X_0||_F = 1/(1+margin): mean sigma^2 of the first iterate (the tensor-core mode shifts by it)
      s->tau = use_shift ? 1.0f / ((1.0f + margin) * (1.0f + margin) * (float)d) : 1.0f;
      s->seg_e = (use_shift && s->tau < e1_tau) ? 1 : 3;
    }
  }
}

// X0 = (M_raw + lam R) * x0_scale
static __global__ void ns_x0_kernel(const float* __restrict__ M, const float* __restrict__ R, float* __restrict__ X0,
                             int64_t dd, const DevState* st) {
  const int p = blockIdx.y;
  const float lam = st[p].lam, sc = st[p].x0_scale;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < dd; i += (int64_t)gridDim.x * blockDim.x)
    X0[p * dd + i] = fmaf(lam, R[p * dd + i], M[p * dd + i]) * sc;
}

// After the residual product of step k: reduce the per-tile partials (max|G - I|, sum (G - I)^2, trace G with
// G = X^T X), decide convergence, and pick the quintic of this step from the device schedule (entry 0 = the lifting
// quintic p_f, entries 1 .. n_sched-1 = the endgame for a spectrum in [floor of p_f, 1]):
//   * while lifting steps are left (the count is learnt per problem, see ns_adapt_lift_plan): p_f;
//   * then the endgame entries in order;
//   * once ||G - I||_F < 0.7 every singular value is known to lie above sqrt(1 - ||G - I||_F), so the schedule
//     jumps to the last endgame entry fitted for an interval that still contains the spectrum;
//   * if the endgame ran out without convergence (the lifting phase was too short for the smallest singular value):
//     the last, order-3 convergent entry again while only a little is missing (||G - I||_F < 0.97: whatever lags has
//     sigma^2 > 0.03 and doubles per step), otherwise 2, then 4, 8, 16 more lifting steps (safe to repeat: they never
//     push a singular value below their floor) and the endgame again.
// The very first step also rescales: ||G_0||_F^(1/2) = (sum sigma^4)^(1/4) bounds the largest singular value of X_0
// from above, far more tightly than the Frobenius norm X_0 was scaled by, and dividing X_0 by it is the same as
// applying p(x / s): a / s, b / s^3, c / s^5.
// The step is handed to the product kernels in shifted residual form (see ns_schedule.h): coef = (gamma + kappa,
// beta1, beta2, kappa) where kappa = mean diagonal of beta1 E + beta2 E^2 is moved from the matrix that gets
// rounded to bf16 into the scalar multiple of X.  use_shift == 0 (exact mode): tau = 1, kappa = 0.
struct NsControlParams {
  const SchedEntry* sched;
  int n_sched, n_lift_init, max_steps, d, use_shift;
  float tol, fro_tol, margin;
  float lo_budget;          // tensor-core mode: the iterate enters the last product as hi + lo while d 2^-8 / growth exceeds this
  double inv_d;             // 1 / d (the decision runs on one thread between two products: no divisions there)
};

// The decision itself (one thread): tmx = max|G - I|, tsq = ||G - I||_F^2, ttr = tr G of step k.
// The part of a problem's state the per-step decision reads and writes.  A kernel that iterates a problem in place keeps
// it in registers between the steps (ns_ctl_load once, ns_ctl_store at the end).
struct NsCtl {
  float e_max, e_fro, tau, growth;
  float coef[4];
  int ns_done, ns_final_buf, ns_idx, lift_left, reentries, seg_x, seg_e, ns_steps_used;
};
__device__ __forceinline__ void ns_ctl_load(NsCtl& t, const DevState* s) {
  t.e_max = s->e_max; t.e_fro = s->e_fro; t.tau = s->tau; t.growth = s->growth;
  t.coef[0] = s->coef[0]; t.coef[1] = s->coef[1]; t.coef[2] = s->coef[2]; t.coef[3] = s->coef[3];
  t.ns_done = s->ns_done; t.ns_final_buf = s->ns_final_buf; t.ns_idx = s->ns_idx; t.lift_left = s->lift_left;
  t.reentries = s->reentries; t.seg_x = s->seg_x; t.seg_e = s->seg_e; t.ns_steps_used = s->ns_steps_used;
}
__device__ __forceinline__ void ns_ctl_store(const NsCtl& t, DevState* s) {
  s->e_max = t.e_max; s->e_fro = t.e_fro; s->tau = t.tau; s->growth = t.growth;
  s->coef[0] = t.coef[0]; s->coef[1] = t.coef[1]; s->coef[2] = t.coef[2]; s->coef[3] = t.coef[3];
  s->ns_done = t.ns_done; s->ns_final_buf = t.ns_final_buf; s->ns_idx = t.ns_idx; s->lift_left = t.lift_left;
  s->reentries = t.reentries; s->seg_x = t.seg_x; s->seg_e = t.seg_e; s->ns_steps_used = t.ns_steps_used;
}

// Returns the step's entry of the pass log (seg_x | seg_e << 4), or 0 when no step follows.
__device__ __forceinline__ unsigned char ns_control_decide(NsCtl* s, float tmx, double tsq, double ttr, int k, int cur_buf,
                                                           const NsControlParams& c) {
  unsigned char log_entry = 0;
  const float fro = sqrtf((float)tsq);
  s->e_max = tmx;
  s->e_fro = fro;
  if (!(tmx == tmx) || !(fro == fro)) {
    s->ns_done = NS_DONE_FAILED;
  } else if (tmx <= c.tol && fro <= c.fro_tol) {
    s->ns_done = NS_DONE_CONVERGED;
    s->ns_final_buf = cur_buf;
  } else if (k >= c.max_steps) {
    s->ns_done = NS_DONE_FAILED;
  } else {
    int idx = s->ns_idx;
    bool lifting = false;
    if (fro < 0.7f) {
      s->lift_left = 0;                                            // nothing is small any more
      const float lb = sqrtf(1.0f - fro);
      for (int j = c.n_sched - 1; j >= 1; --j)
        if (c.sched[j].l <= lb) { if (j > idx || idx >= c.n_sched) idx = j; break; }
    }
    if (s->lift_left > 0) {
      lifting = true;
      s->lift_left -= 1;
    } else if (idx >= c.n_sched) {
      if (fro < 0.97f) { idx = c.n_sched - 1; }
      else {
        // 2, 4, 8, 16 more lifting steps, then the endgame again: a plan that was far too short (a much worse
        // conditioned matrix than the ones the count was learnt on) still gets there within ns_max_steps
        lifting = true;
        s->lift_left = (2 << min(s->reentries, 3)) - 1;
        s->reentries += 1;
        idx = 1;
      }
    }
    const SchedEntry e = c.sched[lifting ? 0 : idx];
    if (!lifting) idx += 1;
    double a = e.a, b = e.b, cc = e.c;
    if (k == 0 && c.use_shift) {
      const double g2 = tsq + 2.0 * ttr - (double)c.d;            // ||G||_F^2 = ||G - I||_F^2 + 2 tr G - d
      if (g2 > 0.0) {
        const double sm = sqrt(sqrt(g2)) * (1.0 + (double)c.margin);
        if (sm < 1.0) { const double s2 = sm * sm; a /= sm; b /= sm * s2; cc /= sm * s2 * s2; }
      }
    }
    const double tau = c.use_shift ? (double)s->tau : 1.0;
    const double b1 = b + 2.0 * cc * tau;
    double kappa = 0.0;
    if (c.use_shift) {
      // ||E_tau||_F^2 and tr E_tau from the statistics of G - I and tr G
      const double dd = (double)c.d;
      const double e2 = fmax(0.0, tsq + 2.0 * (1.0 - tau) * ttr + dd * (tau * tau - 1.0));
      kappa = (cc * e2 + b1 * (ttr - dd * tau)) * c.inv_d;
    }
    s->coef[0] = (float)(a + b * tau + cc * tau * tau + kappa);
    s->coef[1] = (float)b1;
    s->coef[2] = (float)cc;
    s->coef[3] = (float)kappa;
    // bf16 rounding of X adds noise of spectral size about 2^-8; after a cumulative growth G of the small singular
    // values the directions it can scramble had sigma_0 <= 2^-8 / G, at most d of them: Procrustes gap <= d 2^-8 / G
    const int seg_x = (!c.use_shift || (float)c.d * (1.0f / 256.0f) / s->growth > c.lo_budget) ? 2 : 1;
    s->growth *= (float)a;
    s->seg_x = seg_x;
    log_entry = (unsigned char)(seg_x | (s->seg_e << 4));           // seg_e: what this step's residual product used
    s->ns_idx = idx;
    s->ns_steps_used = k + 1;
  }
  return log_entry;
}

static __global__ void ns_control_kernel(DevState* st, const float* __restrict__ part_max,
                                  const double* __restrict__ part_sq, const double* __restrict__ part_tr,
                                  int nparts, int k, int cur_buf, const NsControlParams c) {
  const int p = blockIdx.x;
  DevState* s = st + p;
  if (s->ns_done) return;
  if (k < 0) k = s->ns_steps_used;           // inside the update graph's loop: the step's index lives on the device
  __shared__ double redd[8];
  __shared__ float redf[8];
  double sq = 0.0, tr = 0.0;
  float mx = 0.f;
  for (int i = threadIdx.x; i < nparts; i += 256) {
    sq += part_sq[(int64_t)p * nparts + i];
    mx = fmaxf(mx, part_max[(int64_t)p * nparts + i]);
    if (part_tr) tr += part_tr[(int64_t)p * nparts + i];
  }
  const double tsq = block_sum_d<256>(sq, redd);
  const double ttr = block_sum_d<256>(tr, redd);
  const float tmx = block_max_f<256>(mx, redf);
  if (threadIdx.x == 0) {
    NsCtl t;
    ns_ctl_load(t, s);
    const unsigned char log_entry = ns_control_decide(&t, tmx, tsq, ttr, k, cur_buf, c);
    ns_ctl_store(t, s);
    if (log_entry && k < 128) s->seg_log[k] = log_entry;
  }
}

// tau of the next residual product = mean sigma^2 of the new iterate = ||X||_F^2 / d (tensor-core mode), and how
// many bf16 passes that product takes.  Dropping the iterate's lo part changes G = X^T X by about
// 4.4e-3 sqrt(tau) sigma_max (a symmetric perturbation).  One pass is enough
//   * while the iterate is tiny (tau below e1_tau): the perturbation is small in absolute terms;
//   * for a late lifting step, once the small singular values have grown so far (same bound as for the iterate's
//     lo part in the last product: d 2^-8 / growth <= lo_budget) that the directions such noise can still scramble
//     carry no weight.  Endgame steps and the acceptance check always take three passes: there a perturbation of
//     G by a few 1e-3 costs a whole extra step.
static __global__ void ns_tau_kernel(DevState* st, const double* __restrict__ part_x2, int nparts, int d, float e1_tau,
                                     float lo_budget) {
  DevState* s = st + blockIdx.x;
  if (s->ns_done) return;
  __shared__ double redd[8];
  double v = 0.0;
  for (int i = threadIdx.x; i < nparts; i += 256) v += part_x2[(int64_t)blockIdx.x * nparts + i];
  const double tot = block_sum_d<256>(v, redd);
  if (threadIdx.x == 0) {
    s->tau = (float)(tot / (double)d);
    const bool grown = (float)d * (1.0f / 256.0f) / s->growth <= lo_budget;
    const bool next_is_lifting = s->lift_left > 0 && s->e_fro >= 0.7f;     // (control drops the rest of the lifting below 0.7)
    s->seg_e = (s->tau < e1_tau || (grown && next_is_lifting)) ? 1 : 3;
  }
}

// Accept or reject the update.  On success: R <- X_final, M <- 0, sums <- 0.
static __global__ void ns_commit_kernel(DevState* st, const float* __restrict__ Xa, const float* __restrict__ Xb,
                                 float* __restrict__ R, float* __restrict__ M, int64_t dd) {
  const int p = blockIdx.y;
  DevState* s = st + p;
  if (s->ns_done != NS_DONE_CONVERGED) return;
  const float* X = (s->ns_final_buf ? Xb : Xa) + p * dd;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < dd; i += (int64_t)gridDim.x * blockDim.x) {
    R[p * dd + i] = X[i];
    M[p * dd + i] = 0.f;
  }
}
static __global__ void ns_commit_state_kernel(DevState* st, int n_endgame) {
  DevState* s = st + blockIdx.x;
  if (threadIdx.x != 0) return;
  ns_adapt_lift_plan(s, n_endgame, s->ns_done == NS_DONE_CONVERGED);
  if (s->ns_done == NS_DONE_CONVERGED) {
    s->last_J = s->J;
    s->last_N = s->N;
    s->J = 0.0;
    s->N = 0;
    s->diag_pr = s->diag_rho = s->diag_qnum = s->diag_qden = 0.0;
    s->updates += 1;
    s->last_orth = s->e_max;
    s->last_fro = s->e_fro;
  } else {
    atomicOr(&s->status_flags, STATUS_FLAG_NS_FAILED);
  }
}

// ------------------------------------------------------------------ misc element-wise
static __global__ void scale_copy_kernel(const float* __restrict__ src, float* __restrict__ dst, int64_t count, float f) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    dst[i] = src[i] * f;
}
static __global__ void set_identity_kernel(float* __restrict__ R, int d, int P) {
  const int64_t dd = (int64_t)d * d;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < dd * P; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t e = i % dd;
    R[i] = ((e / d) == (e % d)) ? 1.f : 0.f;
  }
}
// sign matrices of the last step from C' (per problem n x d, row-major, problems src_ps elements apart) held as fp32
// (exact mode) or bf16 (tensor-core mode); written densely, problem after problem.  grid.y = problems.
static __global__ void signs_from_c_kernel(const float* __restrict__ C, const __nv_bfloat16* __restrict__ Cb, int64_t n,
                                    int d, int64_t src_ps, int8_t* __restrict__ S) {
  const int64_t total = n * d;
  const int64_t src0 = (int64_t)blockIdx.y * src_ps;
  int8_t* out = S + (int64_t)blockIdx.y * total;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const float v = C ? C[src0 + i] : __bfloat162float(Cb[src0 + i]);
    out[i] = (v > 0.f) ? 1 : ((v < 0.f) ? -1 : 0);
  }
}

}  // namespace conqur
