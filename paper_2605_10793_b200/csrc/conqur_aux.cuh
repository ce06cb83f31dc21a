// Around the calibration path (Appendix A): folding a learned rotation into a linear layer's weight, and the
// fixed online Walsh-Hadamard transform (the R_3 / R_4 rotations).
#pragma once
#include "conqur_simt.cuh"
#include "conqur_tc.cuh"

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
// A CTA of 256 threads transforms blocks of 256 E consecutive elements (one row, or several whole rows when d is
// smaller).  The transform is a butterfly over each of the logd index bits, in any order; the bits are handled in
// up to three groups, each while the thread that owns an element also owns its partners:
//   first    thread t takes the 16-byte pieces t, t+256, ... of the block (coalesced; element index =
//            4 (t + 256 j) + e): index bits 0-1 (e) and 10.. (j) are inside the thread, their butterflies run in
//            registers, and the values go to a work buffer in shared memory;
//   middle   bits 2-5: a thread gathers the 16 elements that differ only in these bits (stride 4), transforms them
//            in registers and puts them back in place;
//   last     bits 6-9: the same with stride 64;
//   store    pieces are read back in the first group's layout, scaled by 1/sqrt(d), converted and written out
//            (coalesced 16- or 8-byte pieces; storing straight from the last group's registers, 2 or 4 bytes per
//            lane, measured 1.5x slower).
// Work-buffer layout: 4 floats of padding after every 64, i.e. position i lives at i + 4 (i >> 6): every
// access pattern above is free of bank conflicts and every offset inside a group is a compile-time constant.
//
// The input is staged by bulk asynchronous copies (the TMA engine's 1-D form): a persistent CTA walks its blocks
// with a ring of S raw-input stages in shared memory, each filled by `cp.async.bulk` (one copy per block when the
// rows are contiguous, else one per row) that signals an mbarrier; the copy of block i+S is issued as soon as every
// thread has taken block i out of its stage.  The data in flight lives in shared memory rather than in registers:
// S stages x the resident CTAs hold > 100 KB in flight per SM.  Needs 16-byte aligned rows (base and row stride);
// other layouts take the plain-load kernel below (one block per CTA).  Every wait is bounded; a wait that gives up
// latches the TIMEOUT flag in g_aux_status_flags, lets the copies in flight land, and the CTA ends.
constexpr int HAD_THREADS = 256;
static __device__ int g_aux_status_flags;

namespace ptx {
__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
}  // namespace ptx

__device__ __forceinline__ int had_pad(int i) { return i + ((i >> 6) << 2); }
template <int E> struct HadWork { static constexpr int FLOATS = HAD_THREADS * E + HAD_THREADS * E / 16; };

template <int N>
__device__ __forceinline__ void had_butterflies(float (&w)[N], int nbits) {
#pragma unroll
  for (int m = 0; (1 << m) < N; ++m)
    if (m < nbits) {
#pragma unroll
      for (int k = 0; k < N; ++k)
        if (!(k & (1 << m))) {
          const float a = w[k], c = w[k | (1 << m)];
          w[k] = a + c; w[k | (1 << m)] = a - c;
        }
    }
}

__device__ __forceinline__ void st4_from_float(float* p, const float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4_from_float(__nv_bfloat16* p, const float4 v) {
  uint2 o;
  o.x = bf16x2_pack(v.x, v.y);
  o.y = bf16x2_pack(v.z, v.w);
  *reinterpret_cast<uint2*>(p) = o;
}
__device__ __forceinline__ void st1_from_float(float* p, float v) { *p = v; }
__device__ __forceinline__ void st1_from_float(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// First group for one block: `src` is the block's raw input (global memory, or a stage in shared memory) addressed
// through row(i) -> pointer; the values land in the work buffer.
template <typename TIn, int E, typename RowPtr>
__device__ __forceinline__ void had_first(float* sm, int logd, int64_t rows_left, RowPtr&& elem_ptr) {
  const int t = threadIdx.x;
  float v[E];
#pragma unroll
  for (int j = 0; j < E / 4; ++j) {
    const int i = 4 * (t + HAD_THREADS * j);
    float x[4] = {0.f, 0.f, 0.f, 0.f};
    if ((i >> logd) < rows_left) ld4_as_float(elem_ptr(i), x);
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
    *reinterpret_cast<float4*>(&sm[had_pad(4 * (t + HAD_THREADS * j))]) =
        make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
}

// Middle group (bits 2-5, `nbits` of them), in place.
template <int E>
__device__ __forceinline__ void had_middle(float* sm, int nbits) {
#pragma unroll
  for (int q = 0; q < E / 16; ++q) {
    const int u = threadIdx.x + HAD_THREADS * q;
    float* p = sm + had_pad(((u >> 2) << 6) | (u & 3));
    float w[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) w[k] = p[4 * k];
    had_butterflies(w, nbits);
#pragma unroll
    for (int k = 0; k < 16; ++k) p[4 * k] = w[k];
  }
}

// Last group (bits 6-9, `nbits` of them), in place.
template <int E>
__device__ __forceinline__ void had_last(float* sm, int nbits) {
#pragma unroll
  for (int q = 0; q < E / 16; ++q) {
    const int u = threadIdx.x + HAD_THREADS * q;
    float* p = sm + had_pad(((u >> 6) << 10) | (u & 63));
    float w[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) w[k] = p[68 * k];
    had_butterflies(w, nbits);
#pragma unroll
    for (int k = 0; k < 16; ++k) p[68 * k] = w[k];
  }
}

// Out of the work buffer in the first group's layout: scaled, converted, 16-byte (fp32) / 8-byte (bf16) pieces.
template <typename TOut, int E>
__device__ __forceinline__ void had_plain_store(const float* sm, int logd, int64_t rows_left, float scale, TOut* Yblk, int64_t ldy) {
  const int d = 1 << logd;
#pragma unroll
  for (int j = 0; j < E / 4; ++j) {
    const int i = 4 * (threadIdx.x + HAD_THREADS * j);
    if ((i >> logd) >= rows_left) continue;
    float4 o = *reinterpret_cast<const float4*>(&sm[had_pad(i)]);
    o.x *= scale; o.y *= scale; o.z *= scale; o.w *= scale;
    st4_from_float(Yblk + (int64_t)(i >> logd) * ldy + (i & (d - 1)), o);
  }
}

// Everything after the first group for one block (the work buffer is filled; ends with the block stored).
template <typename TOut, int E>
__device__ __forceinline__ void had_finish(float* sm, int logd, int64_t rows_left, float scale, TOut* Yblk, int64_t ldy) {
  const int r = (logd < 10 ? logd : 10) - 2;                // index bits 2 .. 2+r-1 go through the work buffer
  if (r > 0) had_middle<E>(sm, r < 4 ? r : 4);
  if (r > 4) {
    __syncthreads();
    had_last<E>(sm, r - 4);
  }
  __syncthreads();
  had_plain_store<TOut, E>(sm, logd, rows_left, scale, Yblk, ldy);
}

template <typename TIn, typename TOut, int E>
__global__ void __launch_bounds__(HAD_THREADS) hadamard_rows_kernel(const TIn* X, int64_t ldx, TOut* Y, int64_t ldy, int64_t n,
                                                                     int logd, float scale) {
  __shared__ __align__(16) float sm[HadWork<E>::FLOATS];
  const int d = 1 << logd;
  const int64_t row0 = (int64_t)blockIdx.x * ((HAD_THREADS * E) >> logd);
  const TIn* Xblk = X + row0 * ldx;
  had_first<TIn, E>(sm, logd, n - row0, [&](int i) { return Xblk + (int64_t)(i >> logd) * ldx + (i & (d - 1)); });
  __syncthreads();
  had_finish<TOut, E>(sm, logd, n - row0, scale, Y + row0 * ldy, ldy);
}

template <typename TIn, int E, int S>
constexpr int had_bulk_smem_bytes() { return HadWork<E>::FLOATS * 4 + S * HAD_THREADS * E * (int)sizeof(TIn) + 128; }

template <typename TIn, typename TOut, int E, int S>
__global__ void __launch_bounds__(HAD_THREADS, E == 16 ? 4 : 2) hadamard_rows_bulk_kernel(const TIn* X, int64_t ldx, TOut* Y,
                                                                                           int64_t ldy, int64_t n, int logd,
                                                                                           float scale, int64_t nblocks) {
  extern __shared__ __align__(128) uint8_t had_smem[];
  constexpr int NB = HAD_THREADS * E;                       // elements per block
  constexpr int WORK_BYTES = HadWork<E>::FLOATS * 4;
  float* sm = reinterpret_cast<float*>(had_smem);
  TIn* stage = reinterpret_cast<TIn*>(had_smem + WORK_BYTES);
  uint64_t* full = reinterpret_cast<uint64_t*>(had_smem + WORK_BYTES + S * NB * sizeof(TIn));
  __shared__ int abort_flag;
  const int d = 1 << logd;
  const int rows_per_block = NB >> logd;
  const int t = threadIdx.x;

  auto issue = [&](int64_t blk, int s) {                    // one thread
    const int64_t row0 = blk * rows_per_block;
    const int rows = (int)((n - row0 < rows_per_block) ? (n - row0) : rows_per_block);
    const uint32_t row_bytes = (uint32_t)d * sizeof(TIn);
    ptx::mbar_expect_tx(&full[s], (uint32_t)rows * row_bytes);
    TIn* dst = stage + (size_t)s * NB;
    if (ldx == d) {
      ptx::bulk_load_1d(dst, X + row0 * ldx, (uint32_t)rows * row_bytes, &full[s]);
    } else {
      for (int r = 0; r < rows; ++r) ptx::bulk_load_1d(dst + (size_t)r * d, X + (row0 + r) * ldx, row_bytes, &full[s]);
    }
  };

  if (t == 0) {
    for (int s = 0; s < S; ++s) ptx::mbar_init(&full[s], 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  __syncthreads();
  int issued = 0;
  if (t == 0)
    for (int s = 0; s < S; ++s) {
      const int64_t blk = (int64_t)blockIdx.x + (int64_t)s * gridDim.x;
      if (blk < nblocks) { issue(blk, s); ++issued; }
    }
  int s = 0;
  uint32_t parity = 0;
  bool bad = false;
  for (int64_t blk = blockIdx.x; blk < nblocks; blk += gridDim.x) {
    const bool ok = tc_wait(&full[s], parity, &abort_flag);
    const int64_t row0 = blk * rows_per_block;
    const TIn* src = stage + (size_t)s * NB;
    // (the work buffer is free: the previous block's last group ended with a barrier)
    had_first<TIn, E>(sm, logd, ok ? n - row0 : 0, [&](int i) { return src + i; });
    // everyone has taken this block out of its stage (and knows whether a wait gave up)
    if (__syncthreads_or(!ok)) { bad = true; break; }
    if (t == 0) {
      const int64_t nxt = blk + (int64_t)S * gridDim.x;
      if (nxt < nblocks) { issue(nxt, s); ++issued; }
    }
    had_finish<TOut, E>(sm, logd, n - row0, scale, Y + row0 * ldy, ldy);
    __syncthreads();
    if (++s == S) { s = 0; parity ^= 1u; }
  }
  if (bad && t == 0) {
    atomicOr(&g_aux_status_flags, STATUS_FLAG_TIMEOUT);
    if (issued > 0) {                                       // let the copies in flight land before the CTA's shared memory goes
      const long long t0 = clock64();
      while (clock64() - t0 < 4000000ll) {}
    }
  }
}

template <typename TIn, typename TOut, int E, int S>
inline int hadamard_launch_bulk(const TIn* X, int64_t ldx, TOut* Y, int64_t ldy, int64_t n, int logd, float scale,
                                cudaStream_t s) {
  constexpr int smem = had_bulk_smem_bytes<TIn, E, S>();
  auto kern = hadamard_rows_bulk_kernel<TIn, TOut, E, S>;
  // per device: the shared-memory attribute, and how many CTAs fit (looked up once, under a lock)
  struct Facts { int known, ctas_per_sm, sms; };
  static std::mutex mu;
  static Facts facts[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return CONQUR_ERR_CUDA;
  int ctas_per_sm = 0, sms = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    Facts& f = facts[dev];
    if (!f.known) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return CONQUR_ERR_CUDA;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&f.ctas_per_sm, kern, HAD_THREADS, smem) != cudaSuccess) return CONQUR_ERR_CUDA;
      if (cudaDeviceGetAttribute(&f.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return CONQUR_ERR_CUDA;
      if (f.ctas_per_sm < 1) return CONQUR_ERR_UNSUPPORTED;
      f.known = 1;
    }
    ctas_per_sm = f.ctas_per_sm; sms = f.sms;
  }
  const int64_t rows_per_block = (HAD_THREADS * E) >> logd;
  const int64_t nblocks = (n + rows_per_block - 1) / rows_per_block;
  const int64_t grid = nblocks < (int64_t)sms * ctas_per_sm ? nblocks : (int64_t)sms * ctas_per_sm;
  kern<<<(unsigned)grid, HAD_THREADS, smem, s>>>(X, ldx, Y, ldy, n, logd, scale, nblocks);
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}

template <typename TIn, typename TOut>
inline int hadamard_launch(const TIn* X, int64_t ldx, TOut* Y, int64_t ldy, int64_t n, int logd, cudaStream_t s) {
  const float scale = (float)(1.0 / sqrt((double)(1 << logd)));
  const int d = 1 << logd;
  // bulk copies need 16-byte aligned rows of a multiple of 16 bytes
  const bool bulk = ((reinterpret_cast<uintptr_t>(X) & 15) == 0) && ((ldx * sizeof(TIn)) % 16 == 0) && ((d * sizeof(TIn)) % 16 == 0);
  if (bulk) {
    if (logd <= 12) return hadamard_launch_bulk<TIn, TOut, 16, sizeof(TIn) == 2 ? 4 : 3>(X, ldx, Y, ldy, n, logd, scale, s);
    return hadamard_launch_bulk<TIn, TOut, 32, 2>(X, ldx, Y, ldy, n, logd, scale, s);
  }
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
