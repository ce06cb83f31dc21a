// Around the calibration path (Appendix A): folding a learned rotation into a linear layer's weight, and the
// fixed online Walsh-Hadamard transform (the R_3 / R_4 rotations).
#pragma once
#include "conqur_simt.cuh"

namespace conqur {

// ------------------------------------------------------------------ weight folding, fp32 CUDA cores
// R = blockdiag(R_0 .. R_{nblk-1}), blocks db x db, row-major, one after another.
//   SIDE 0 (the layer reads rotated activations):        out[:, b] = W[:, b] R_b      (column block b of W)
//   SIDE 1 (the layer writes into the rotated space):    out[b, :] = R_b^T W[b, :]    (row block b of W)
// grid (ceil(N/128), ceil(M/128), nblk) with (M, N) = (rows, db) for SIDE 0 and (db, cols) for SIDE 1.
template <int SIDE>
__global__ void __launch_bounds__(SG_THREADS) fold_exact_kernel(const float* __restrict__ W, int64_t ldw,
                                                                const float* __restrict__ R, int db, int rows, int cols,
                                                                float* __restrict__ out, int64_t ldo) {
  const int b = blockIdx.z;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  const float* Rb = R + (int64_t)b * db * db;
  float acc[8][8];
  int M, N;
  float* o;
  if (SIDE == 0) {
    M = rows; N = db;
    sg_mainloop<float, false, float, true>(W + (int64_t)b * db, ldw, Rb, db, M, N, 0, db, m0, n0, acc);
    o = out + (int64_t)b * db;
  } else {
    M = db; N = cols;
    sg_mainloop<float, true, float, true>(Rb, db, W + (int64_t)b * db * ldw, ldw, M, N, 0, db, m0, n0, acc);
    o = out + (int64_t)b * db * ldo;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int m = m0 + sg_row(i);
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int n = n0 + sg_col(j);
      if (n < N) o[(int64_t)m * ldo + n] = acc[i][j];
    }
  }
}

// fp32 (row stride ld) -> dense bf16 [hi; lo] stack, each part rows x cols
static __global__ void split_bf16_2d_kernel(const float* __restrict__ src, int64_t ld, int rows, int cols,
                                            __nv_bfloat16* __restrict__ dst) {
  const int c4 = cols >> 2;
  const int64_t total = (int64_t)rows * c4, lo = (int64_t)rows * cols;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / c4;
    const int c = (int)(i - r * c4) * 4;
    const float4 t = *reinterpret_cast<const float4*>(src + r * ld + c);
    const __nv_bfloat16 h0 = __float2bfloat16_rn(t.x), h1 = __float2bfloat16_rn(t.y), h2 = __float2bfloat16_rn(t.z),
                        h3 = __float2bfloat16_rn(t.w);
    __nv_bfloat16* ph = dst + r * cols + c;
    __nv_bfloat16* pl = ph + lo;
    *reinterpret_cast<__nv_bfloat162*>(ph) = __nv_bfloat162(h0, h1);
    *reinterpret_cast<__nv_bfloat162*>(ph + 2) = __nv_bfloat162(h2, h3);
    *reinterpret_cast<__nv_bfloat162*>(pl) =
        __nv_bfloat162(__float2bfloat16_rn(t.x - __bfloat162float(h0)), __float2bfloat16_rn(t.y - __bfloat162float(h1)));
    *reinterpret_cast<__nv_bfloat162*>(pl + 2) =
        __nv_bfloat162(__float2bfloat16_rn(t.z - __bfloat162float(h2)), __float2bfloat16_rn(t.w - __bfloat162float(h3)));
  }
}

// ------------------------------------------------------------------ Walsh-Hadamard transform of rows
// y = x H_d / sqrt(d), H_d the Sylvester matrix (H[i][j] = (-1)^popcount(i & j)), d = 2^logd, 4 <= d <= 256 E.
//
// A CTA of 256 threads transforms a block of 256 E consecutive elements (one row, or several whole rows when d is
// smaller).  The transform is a butterfly over each of the logd index bits, in any order:
//   load     thread t reads the 16-byte pieces t, t+256, ... (coalesced); element index = 4 (t + 256 j) + e, so
//            bits 0-1 (e) and bits 10.. (j) of the index are in the thread's own registers: those butterflies run
//            right away, and the values go to shared memory;
//   passes   bits 2..9 in one or two passes through shared memory: a thread gathers the 2^B elements that differ
//            only in the pass's B bits, transforms them in registers and puts them back (in place, disjoint groups);
//   store    pieces are read back in the load order, scaled by 1/sqrt(d) and written out (coalesced).
// Shared-memory index swizzle: bits 2-4 ^= bits 6-8, which keeps 16-byte pieces whole and spreads both the
// stride-4 groups of the first pass and the stride-64 groups of the second over the banks.
constexpr int HAD_THREADS = 256;

__device__ __forceinline__ int had_swz(int i) { return i ^ (((i >> 6) & 7) << 2); }

template <int B>
__device__ __forceinline__ void had_pass(float* sm, int s, int groups) {
  for (int q = 0; q < groups; ++q) {
    const int u = threadIdx.x + HAD_THREADS * q;
    const int base = ((u >> s) << (s + B)) | (u & ((1 << s) - 1));
    float w[1 << B];
#pragma unroll
    for (int k = 0; k < (1 << B); ++k) w[k] = sm[had_swz(base | (k << s))];
#pragma unroll
    for (int m = 0; m < B; ++m)
#pragma unroll
      for (int k = 0; k < (1 << B); ++k)
        if (!(k & (1 << m))) {
          const float a = w[k], c = w[k | (1 << m)];
          w[k] = a + c; w[k | (1 << m)] = a - c;
        }
#pragma unroll
    for (int k = 0; k < (1 << B); ++k) sm[had_swz(base | (k << s))] = w[k];
  }
}

__device__ __forceinline__ void had_pass_n(float* sm, int s, int b, int E) {
  switch (b) {
    case 1: had_pass<1>(sm, s, E >> 1); break;
    case 2: had_pass<2>(sm, s, E >> 2); break;
    case 3: had_pass<3>(sm, s, E >> 3); break;
    case 4: had_pass<4>(sm, s, E >> 4); break;
    default: break;
  }
}

__device__ __forceinline__ void st4_from_float(float* p, const float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4_from_float(__nv_bfloat16* p, const float4 v) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 o;
  o.x = *reinterpret_cast<const uint32_t*>(&a);
  o.y = *reinterpret_cast<const uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = o;
}

template <typename TIn, typename TOut, int E>
__global__ void __launch_bounds__(HAD_THREADS) hadamard_rows_kernel(const TIn* X, int64_t ldx,
                                                                     TOut* Y, int64_t ldy, int64_t n, int logd,
                                                                     float scale) {
  __shared__ __align__(16) float sm[HAD_THREADS * E];
  const int d = 1 << logd;
  const int t = threadIdx.x;
  const int64_t row0 = (int64_t)blockIdx.x * ((HAD_THREADS * E) >> logd);
  float v[E];
#pragma unroll
  for (int j = 0; j < E / 4; ++j) {
    const int i = 4 * (t + HAD_THREADS * j);
    const int64_t row = row0 + (i >> logd);
    float x[4] = {0.f, 0.f, 0.f, 0.f};
    if (row < n) ld4_as_float(X + row * ldx + (i & (d - 1)), x);
    // bits 0 and 1
    const float s0 = x[0] + x[1], d0 = x[0] - x[1], s1 = x[2] + x[3], d1 = x[2] - x[3];
    v[4 * j + 0] = s0 + s1; v[4 * j + 1] = d0 + d1; v[4 * j + 2] = s0 - s1; v[4 * j + 3] = d0 - d1;
  }
  // index bits 10.. are the bits 2.. of the register index
#pragma unroll
  for (int m = 2; (1 << m) < E; ++m)
    if (logd > 8 + m) {
#pragma unroll
      for (int k = 0; k < E; ++k)
        if (!(k & (1 << m))) {
          const float a = v[k], c = v[k | (1 << m)];
          v[k] = a + c; v[k | (1 << m)] = a - c;
        }
    }
#pragma unroll
  for (int j = 0; j < E / 4; ++j)
    *reinterpret_cast<float4*>(&sm[had_swz(4 * (t + HAD_THREADS * j))]) =
        make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
  const int r = (logd < 10 ? logd : 10) - 2;          // index bits 2 .. 2+r-1 go through shared memory
  if (r > 0) {
    __syncthreads();
    had_pass_n(sm, 2, r < 4 ? r : 4, E);
    if (r > 4) {
      __syncthreads();
      had_pass_n(sm, 6, r - 4, E);
    }
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < E / 4; ++j) {
    const int i = 4 * (t + HAD_THREADS * j);
    const int64_t row = row0 + (i >> logd);
    if (row >= n) continue;
    float4 o = *reinterpret_cast<const float4*>(&sm[had_swz(i)]);
    o.x *= scale; o.y *= scale; o.z *= scale; o.w *= scale;
    st4_from_float(Y + row * ldy + (i & (d - 1)), o);
  }
}

template <typename TIn, typename TOut>
inline int hadamard_launch(const TIn* X, int64_t ldx, TOut* Y, int64_t ldy, int64_t n, int logd, cudaStream_t s) {
  const float scale = (float)(1.0 / sqrt((double)(1 << logd)));
  if (logd <= 12) {
    const int64_t rows_per_block = (HAD_THREADS * 16) >> logd;
    const int64_t blocks = (n + rows_per_block - 1) / rows_per_block;
    if (blocks > 0x7fffffffll) return CONQUR_ERR_INVALID_ARG;
    hadamard_rows_kernel<TIn, TOut, 16><<<(unsigned)blocks, HAD_THREADS, 0, s>>>(X, ldx, Y, ldy, n, logd, scale);
  } else {
    if (n > 0x7fffffffll) return CONQUR_ERR_INVALID_ARG;
    hadamard_rows_kernel<TIn, TOut, 32><<<(unsigned)n, HAD_THREADS, 0, s>>>(X, ldx, Y, ldy, n, logd, scale);
  }
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}

}  // namespace conqur
