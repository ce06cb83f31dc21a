// Walsh-Hadamard rows on the tensor cores (bf16 input, contiguous rows).
//
// H_d = H_c (x) H_128 for d = 128 c (index = chunk * 128 + e), so y = x H_d / sqrt(d) splits into
//   level 1   every 128-element chunk times H_128: one tcgen05 product with EXACT operands (the bf16 input and a
//             +-1 matrix), fp32 accumulation in TMEM;
//   level 2   a c-point transform across the chunks of a row: log2(c) butterfly levels in fp32 registers.
// (d <= 128: the 128-element chunk holds 128/d rows and level 1 uses the block-diagonal I (x) H_d; no level 2.)
//
// The input is read as a flat matrix of chunks [NC][128].  Per tile of 256 chunks:
//   TMA            chunk tile (256 x 128 bf16, K-major, 64 KB)                      -> shared memory (ring of 2)
//   tcgen05.mma    D[e'][chunk] = sum_e A[e'][e] X[chunk][e]   (A = +-1 matrix, resident in shared memory)  -> TMEM
//                  M = 128 (e'), N = 256 (chunks), K = 128; the accumulator is double-buffered (2 x 256 columns)
//   epilogue       thread = TMEM lane e': a 32-column load gives it 32 consecutive chunks of the same e', i.e. whole
//                  rows' worth of level-2 inputs (c <= 32; two loads for c = 64) -> butterflies in registers ->
//                  scale -> transposed through a per-warp staging block in shared memory -> 8/16-byte stores to
//                  y[chunk][e'].
// Algorithmic traffic = the input once + the output once; the CUDA cores do log2(c) instead of log2(d) additions
// per element.  Warp roles: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..17 = epilogue (four warps per TMEM
// lane quarter, 64 columns each).  Every wait is bounded; a wait that gives up latches TIMEOUT in
// g_aux_status_flags and the CTA drains and ends.
#pragma once
#include "conqur_aux.cuh"

namespace conqur {

constexpr int HTC_N = 256;                          // chunks per tile
constexpr int HTC_STAGES = 2;
constexpr int HTC_EPI_WARPS = 16;
constexpr int HTC_THREADS = 64 + 32 * HTC_EPI_WARPS;
constexpr int HTC_A_BYTES = 128 * 128 * 2;          // two 64-column swizzled chunks of 16 KB
constexpr int HTC_X_BYTES = HTC_N * 128 * 2;        // two 64-column swizzled chunks of 32 KB
constexpr int HTC_STG_BYTES = 32 * 32 * 4;          // per epilogue warp
constexpr int HTC_AUX_BYTES = 256;
constexpr int HTC_SMEM_BYTES = HTC_A_BYTES + HTC_STAGES * HTC_X_BYTES + HTC_EPI_WARPS * HTC_STG_BYTES + HTC_AUX_BYTES + 1024;

struct HtcAux {
  uint64_t xfull[HTC_STAGES], xempty[HTC_STAGES];
  uint64_t dfull[2], dempty[2];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(HtcAux) <= HTC_AUX_BYTES, "the barrier block must fit its reserved shared memory");

template <typename TOut>
__global__ void __launch_bounds__(HTC_THREADS, 1)
hadamard_tc_kernel(const __grid_constant__ CUtensorMap tmX, TOut* Y, long long NC, int logd, float scale) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sX = smem + HTC_A_BYTES;
  uint8_t* sStg = sX + HTC_STAGES * HTC_X_BYTES;
  HtcAux* aux = reinterpret_cast<HtcAux*>(sStg + HTC_EPI_WARPS * HTC_STG_BYTES);
  volatile int* abort_flag = &aux->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long tiles = (NC + HTC_N - 1) / HTC_N;

  if (threadIdx.x == 0) {
    for (int s = 0; s < HTC_STAGES; ++s) { ptx::mbar_init(&aux->xfull[s], 1); ptx::mbar_init(&aux->xempty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&aux->dfull[b], 1); ptx::mbar_init(&aux->dempty[b], HTC_EPI_WARPS); }
    aux->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmX);
  }
  // A[e'][e] = +-1 inside diagonal blocks of size min(d, 128), 0 outside: (-1)^popcount(e' & e & (block - 1)).
  // Layout: what TMA would write for a K-major 128 x 128 bf16 tile (two 64-column chunks, 128-byte swizzle).
  {
    const int blk = (logd < 7) ? (1 << logd) : 128;
    for (int i = threadIdx.x; i < 128 * 16; i += HTC_THREADS) {        // 16-byte pieces: row m, columns 8 c16 .. 8 c16 + 7
      const int m = i >> 4, c16 = i & 15;
      uint32_t w[4];
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        uint32_t pair = 0;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int k = c16 * 8 + h * 2 + e;
          uint32_t v = 0;
          if ((m & ~(blk - 1)) == (k & ~(blk - 1))) v = (__popc(m & k & (blk - 1)) & 1) ? 0xBF80u : 0x3F80u;
          pair |= v << (16 * e);
        }
        w[h] = pair;
      }
      *reinterpret_cast<uint4*>(sA + (c16 >> 3) * 16384 + m * 128 + (((c16 & 7) ^ (m & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    ptx::fence_proxy_async();                      // the matrix is read by the tensor-core proxy
  }
  if (warp == 1) { ptx::tmem_alloc(&aux->tmem_base, 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = aux->tmem_base;
  int timeout_site = 0;

  if (warp == 0) {
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      int issued = 0;
      bool ok = true;
      for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        if (!tc_wait(&aux->xempty[s], ph ^ 1u, abort_flag)) { ok = false; timeout_site = 1; break; }
        uint8_t* dst = sX + s * HTC_X_BYTES;
        ptx::mbar_expect_tx(&aux->xfull[s], HTC_X_BYTES);
        ptx::tma_load_2d(dst, &tmX, &aux->xfull[s], 0, (int)(t * HTC_N));
        ptx::tma_load_2d(dst + HTC_X_BYTES / 2, &tmX, &aux->xfull[s], 64, (int)(t * HTC_N));
        ++issued;
        if (++s == HTC_STAGES) { s = 0; ph ^= 1u; }
      }
      if (!ok && issued > 0) {                     // let the copies in flight land before the CTA exits
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) {}
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 256
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HTC_N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t sA_a = ptx::smem_u32(sA), sX_a = ptx::smem_u32(sX);
      int s = 0; uint32_t ph = 0;
      int it = 0;
      for (long long t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
        const int buf = it & 1;
        if (!tc_wait(&aux->xfull[s], ph, abort_flag)) { timeout_site = 2; break; }
        if (!tc_wait(&aux->dempty[buf], (((uint32_t)it >> 1) & 1u) ^ 1u, abort_flag)) { timeout_site = 3; break; }
        ptx::tc_fence_after();
        const uint32_t xb = sX_a + s * HTC_X_BYTES;
#pragma unroll
        for (int j = 0; j < 8; ++j)                // 16 e per instruction: chunk j / 4, 32 bytes per step inside the swizzled row
          ptx::umma_bf16(tmem_base + (uint32_t)(buf * HTC_N), tc_smem_desc(sA_a + (j >> 2) * 16384 + (j & 3) * 32, 16, 1024),
                         tc_smem_desc(xb + (j >> 2) * (HTC_X_BYTES / 2) + (j & 3) * 32, 16, 1024), idesc, j > 0 ? 1u : 0u);
        ptx::umma_commit(&aux->xempty[s]);
        ptx::umma_commit(&aux->dfull[buf]);
        if (++s == HTC_STAGES) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    const int ew = warp - 2;                       // 0..15
    const int q = warp & 3;                        // TMEM lane quarter this warp may read
    const int cq = ew >> 2;                        // which 64 of the 256 columns
    const int e_out = q * 32 + lane;               // e' of this thread
    float* stg = reinterpret_cast<float*>(sStg + ew * HTC_STG_BYTES);
    const int lc = (logd > 7) ? (logd - 7) : 0;    // level-2 butterfly levels (c = 2^lc chunks per row)
    int it = 0;
    // one 32-column group: level-2 levels < 5, scale, transpose, store
    auto finish32 = [&](float (&v)[32], long long chunk0) {
      had_butterflies(v, lc < 5 ? lc : 5);
#pragma unroll
      for (int k = 0; k < 32; ++k) stg[k * 32 + lane] = v[k] * scale;
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int r = i * 4 + (lane >> 3), p4 = (lane & 7) * 4;
        const float4 o = *reinterpret_cast<const float4*>(&stg[r * 32 + p4]);
        if (chunk0 + r < NC) st4_from_float(Y + (chunk0 + r) * 128 + q * 32 + p4, o);
      }
      __syncwarp();
    };
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
      const int buf = it & 1;
      if (!tc_wait(&aux->dfull[buf], ((uint32_t)it >> 1) & 1u, abort_flag)) { timeout_site = 4; break; }
      ptx::tc_fence_after();
      const uint32_t t_addr = tmem_base + (uint32_t)(buf * HTC_N + cq * 64) + ((uint32_t)(q * 32) << 16);
      const long long chunk0 = t * HTC_N + cq * 64;
      if (lc == 6) {                               // a row is 64 chunks: both groups at once, the top level first
        float v0[32], v1[32];
        ptx::tmem_ld32(t_addr, v0);
        ptx::tmem_ld32(t_addr + 32u, v1);
#pragma unroll
        for (int k = 0; k < 32; ++k) { const float a = v0[k], b = v1[k]; v0[k] = a + b; v1[k] = a - b; }
        finish32(v0, chunk0);
        finish32(v1, chunk0 + 32);
      } else {
#pragma unroll 1
        for (int gI = 0; gI < 2; ++gI) {
          float v[32];
          ptx::tmem_ld32(t_addr + (uint32_t)(gI * 32), v);
          finish32(v, chunk0 + gI * 32);
        }
      }
      ptx::tc_fence_before();
      __syncwarp();                                // one arrival per warp
      if (lane == 0) ptx::mbar_arrive(&aux->dempty[buf]);
    }
  }

  if (timeout_site != 0) atomicOr(&g_aux_status_flags, STATUS_FLAG_TIMEOUT);
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// n rows of d bf16 elements, contiguous (row stride d), 16-byte aligned base, n * d a multiple of 128.
template <typename TOut>
inline int hadamard_tc_launch(const __nv_bfloat16* X, TOut* Y, int64_t n, int logd, cudaStream_t s) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return CONQUR_ERR_CUDA;
  TcDevFacts f;
  if (tc_device_facts(dev, &f) != CONQUR_OK) return CONQUR_ERR_CUDA;
  auto kern = hadamard_tc_kernel<TOut>;
  if (f.major != 10) return CONQUR_ERR_UNSUPPORTED;
  static std::atomic<unsigned long long> attr_dev_mask{0};      // the attribute is per device
  const unsigned long long dev_bit = 1ull << (dev & 63);
  if (!(attr_dev_mask.load(std::memory_order_acquire) & dev_bit)) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, HTC_SMEM_BYTES) != cudaSuccess) return CONQUR_ERR_CUDA;
    attr_dev_mask.fetch_or(dev_bit, std::memory_order_release);
  }
  const long long NC = (long long)n * (1ll << logd) / 128;
  if (NC < 1 || NC > 0x7fffff00ll) return CONQUR_ERR_INVALID_ARG;
  CUtensorMap tm;
  int rc = tc_make_tmap(&tm, X, (uint64_t)NC, 128, 128, HTC_N);
  if (rc) return rc;
  const long long tiles = (NC + HTC_N - 1) / HTC_N;
  const int grid = (int)(tiles < f.sms ? tiles : f.sms);
  const float scale = (float)(1.0 / sqrt((double)(1 << logd)));
  kern<<<grid, HTC_THREADS, HTC_SMEM_BYTES, s>>>(tm, Y, NC, logd, scale);
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}

}  // namespace conqur
