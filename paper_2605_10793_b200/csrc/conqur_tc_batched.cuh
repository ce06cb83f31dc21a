// Tensor-core mode for many small problems (the per-head case, d = 128): one fused kernel per streamed batch.
//
// A CTA owns one problem at a time and walks its tokens in tiles of 128 rows.  Per tile
//   TMA            X tile (128 tokens x 128, bf16)              -> shared memory (read ONCE from HBM)
//   tcgen05.mma    Y = X_tile R                                 -> TMEM          (R: bf16, resident in shared memory)
//   epilogue       the rows' scales from a pass over Y (||x R~||, see the kernel), sign / fake-quant of Y,
//                  C' = sgn(.) * scale as bf16                   -> shared memory
//   tcgen05.mma    M += X_tile^T C'                              -> TMEM accumulator that lives for the whole problem
// and after the last tile the accumulator is added to the problem's fp32 M in global memory.  The X tile in
// shared memory serves twice: K-major operand of the first product, MN-major operand of the second.  Rows with a
// zero or non-finite scale are zeroed in shared memory before the second product so that they cannot reach M.
//
// Warp roles: 0 = TMA producer, 1 = issuer of the first product and TMEM owner, 2..17 = epilogue: two groups of
// eight warps (two per TMEM lane quarter, one per half of the 128 columns) that take alternate tiles, so that one
// group's waits and TMEM / shared-memory latencies overlap the other group's work; 18 = issuer of the second
// product.  The two products have their own issuing threads and Y has three TMEM buffers, so the first product runs
// up to three tiles ahead of the epilogue.  Shared-memory bandwidth sets the floor of a tile: both products read
// both operands from it (4 x 32 KB), TMA writes 32 KB and the targets 32 KB.  Every wait is bounded.
//
// Objective without fake-quantisation: sum_i ||y_i||_1 rnorm_i = <R, X_tilde^T S> = <R, M> while R is fixed (Section
// 3.2 with Eq. 2), so this kernel does not sum it: the update kernel forms it from M, and so does a read in between.
// At the end of a problem the accumulator leaves through the copy engine (tensor reduce-add into M), handed over by
// the epilogue group that owned the last tile while the other group goes on with the next problem.
#pragma once
#include <type_traits>

#include "conqur_tc.cuh"

namespace conqur {

constexpr int TCB_D = 128;                       // problem size this kernel is built for
constexpr int TCB_TILE_BYTES = 128 * 128 * 2;    // one 128 x 128 bf16 tile = two 64-column swizzled chunks of 16 KB
constexpr int TCB_XSTAGES = 4;                   // a stage is held from the copy's issue until the second product has read it
#ifndef TCB_EPI_GROUPS_N
#define TCB_EPI_GROUPS_N 2
#endif
constexpr int TCB_EPI_GROUPS = TCB_EPI_GROUPS_N; // groups of eight epilogue warps taking tiles in turn
constexpr int TCB_MMA2_WARP = 2 + 8 * TCB_EPI_GROUPS;    // issues the second product
constexpr int TCB_THREADS = (TCB_MMA2_WARP + 1) * 32;
constexpr int TCB_YBUF = 3;                      // Y accumulators in TMEM (128 columns each), then the M accumulator(s)
constexpr int TCB_MBUF = (TCB_YBUF == 2) ? 2 : 1;   // 512 columns in all: 3 + 1 or 2 + 2
constexpr int TCB_EPI_THREADS = 256;
constexpr int TCB_EPI_WARPS = TCB_EPI_THREADS / 32;
constexpr int TCB_PARTS = TCB_EPI_WARPS * TCB_EPI_GROUPS;   // objective partials per work item
constexpr int TCB_AUX_BYTES = 2048;
// Timeline hook (conqur_debug_trace_heads): per tile 16 slots of clock64() values, see TCB_EV_* for the events.
constexpr int TCB_TRACE_TILES = 96;
enum { TCB_EV_TMA = 0, TCB_EV_MMA1 = 1, TCB_EV_MMA2 = 2, TCB_EV_NORM_BEGIN = 3, TCB_EV_NORM_END = 4, TCB_EV_EPI_BEGIN = 5,
       TCB_EV_EPI_NORMS = 6, TCB_EV_EPI_CFREE = 7, TCB_EV_EPI_Y = 8, TCB_EV_EPI_END = 9, TCB_EV_OUT_WAIT = 10, TCB_EV_OUT_BEGIN = 11,
       TCB_EV_OUT_END = 12, TCB_EV_EPI_LD0 = 13, TCB_EV_EPI_ST0 = 14, TCB_EV_EPI_LD1 = 15 };
constexpr int TCB_SMEM_BYTES = TCB_TILE_BYTES * (1 + TCB_XSTAGES + 2) + TCB_AUX_BYTES + 1024;

struct TcbAux {
  uint64_t rfull, rempty, mfull[TCB_MBUF], mempty[TCB_MBUF];
  uint64_t pdone[2];         // [epilogue group]: every warp of the group has finished the problem (write-out, objective partial)
  uint64_t xfull[TCB_XSTAGES], xempty[TCB_XSTAGES];
  uint64_t yfull[TCB_YBUF], yempty[TCB_YBUF], cready[2], cfree[2];
  uint32_t tmem_base;
  int abort_flag;
};

static_assert(sizeof(TcbAux) <= TCB_AUX_BYTES, "the barrier / exchange block must fit its reserved shared memory");
static_assert(TCB_SMEM_BYTES <= 232448, "227 KB of dynamic shared memory per CTA");

struct TcbStepArgs {
  int n, P;                   // P problems; M, part_d, st point at the first of them
  int p0;                     // its index in the context (row block of the rotation map)
  int xp_outer_tokens;        // 1: the input map's dimensions are (column, problem, token) -- head-interleaved rows --
                              //    instead of (column, token, problem)
  QuantSpec qs;               // bits == 0: corner target of the rotated row; else per-token fake-quantisation first
  float* M;                   // P x 128 x 128 fp32 (without the 1/sqrt(d))
  int S;                      // token splits per problem: work item i = (problem i / S, tiles [T (i % S) / S, T (i % S + 1) / S))
  float* Mpart;               // S > 1: P * S partial cross-covariances (item order), summed into M by tcb_finish_kernel
  double* part_d;             // fake-quantisation only: P * S * TCB_PARTS objective partials (one per epilogue warp), item order
  DevState* st;               // P
  long long* trace;           // measurement hook: when set, CTA 0 records SM-clock timestamps of its first TCB_TRACE_TILES tiles
  int8_t* signs;              // test hook: when set, the sign decisions (-1/0/+1) of this call, (P * n) x 128 row-major
};

__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* tmap, uint64_t* bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(ptx::smem_u32(smem_dst)), "l"(tmap), "r"(ptx::smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}

// Byte offset of the 16-byte piece `c16` (0..15) of row `r` inside a 128 x 128 bf16 tile stored as two 64-column
// chunks with the 128-byte swizzle (what TMA writes and what the MMA descriptors expect).
__device__ __forceinline__ uint32_t tcb_piece(int r, int c16) {
  return (uint32_t)((c16 >> 3) * 16384 + r * 128 + (((c16 & 7) ^ (r & 7)) << 4));
}

// Work item -> problem and tile range [t_begin, t_end) of its T tiles (S items per problem).  T * S < 2^32: T <= 2^24
// tiles and S is at most the number of SMs.  The common case S = 1 needs no division.
__device__ __forceinline__ void tcb_item(int item, int T, int S, int& p, int& t_begin, int& t_end) {
  if (S == 1) { p = item; t_begin = 0; t_end = T; return; }
  p = item / S;
  const unsigned sp = (unsigned)(item - p * S);
  t_begin = (int)((unsigned)T * sp / (unsigned)S);
  t_end = (int)((unsigned)T * (sp + 1u) / (unsigned)S);
}

// One warp's share of a problem's write-out: 32 x 32 fp32 blocks of the accumulator (TMEM address t_addr + 32 c, a
// thread holds one row) for c = c0 .. c_end - 1.  Each block is laid into 4 KB of shared memory the way
// the copy engine expects a 32 x 32 fp32 box (128-byte rows, 128-byte swizzle) and handed to it: added element by
// element at the L2 (`add`; fire-and-forget, the warp only waits until the engine has read the staging area) or
// stored.  Box (column 32 c, row y0) of tmOut.  Waits for the accumulator first (`bar`, `parity`; false when that
// wait was abandoned) and arrives at `drained` once the warp's last block has left it.  Kept out of line: it runs once per problem and must not weigh on the tile loop.
__device__ __noinline__ bool tcb_write_out(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t t_addr, uint8_t* stg,
                                           int lane, const CUtensorMap* tmOut, int y0, bool add, int c0, int c_end, uint64_t* drained,
                                           long long* begun) {
  if (!tc_wait(bar, parity, abort_flag)) return false;
  ptx::tc_fence_after();
  if (begun) *begun = clock64();                   // timeline hook
#pragma unroll 1
  for (int c = c0; c < c_end; ++c) {
    float v[32];
    ptx::tmem_ld32(t_addr + (uint32_t)(c * 32), v);
    if (c == c_end - 1) {                          // this warp's part of the accumulator is in registers
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(drained);
    }
#pragma unroll
    for (int p = 0; p < 8; ++p)
      *reinterpret_cast<float4*>(stg + lane * 128 + ((p ^ (lane & 7)) << 4)) = make_float4(v[4 * p], v[4 * p + 1], v[4 * p + 2], v[4 * p + 3]);
    ptx::fence_proxy_async();                      // the staged rows must be visible to the copy engine
    __syncwarp();
    if (lane == 0) {
      if (add) ptx::tma_reduce_add_2d(tmOut, stg, c * 32, y0);
      else ptx::tma_store_2d(tmOut, stg, c * 32, y0);
      ptx::bulk_commit();
      ptx::bulk_wait_read_all();                   // the staging area may be overwritten after this
    }
    __syncwarp();
  }
  return true;
}

__global__ void __launch_bounds__(TCB_THREADS, 1)
tcb_step_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                const __grid_constant__ CUtensorMap tmOut, const TcbStepArgs g) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sR = smem;
  uint8_t* sX = smem + TCB_TILE_BYTES;
  uint8_t* sC = smem + TCB_TILE_BYTES * (1 + TCB_XSTAGES);
  TcbAux* aux = reinterpret_cast<TcbAux*>(smem + TCB_TILE_BYTES * (1 + TCB_XSTAGES + 2));
  volatile int* abort_flag = &aux->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int T = (g.n + 127) / 128;                 // token tiles per problem

  if (threadIdx.x == 0) {
    ptx::mbar_init(&aux->rfull, 1); ptx::mbar_init(&aux->rempty, 1);
    for (int b = 0; b < TCB_MBUF; ++b) { ptx::mbar_init(&aux->mfull[b], 1); ptx::mbar_init(&aux->mempty[b], TCB_EPI_WARPS); }
    for (int i = 0; i < TCB_EPI_GROUPS; ++i) ptx::mbar_init(&aux->pdone[i], TCB_EPI_WARPS);
    for (int s = 0; s < TCB_XSTAGES; ++s) { ptx::mbar_init(&aux->xfull[s], 1); ptx::mbar_init(&aux->xempty[s], 1); }
    for (int b = 0; b < TCB_YBUF; ++b) {
      ptx::mbar_init(&aux->yfull[b], 1); ptx::mbar_init(&aux->yempty[b], TCB_EPI_WARPS);
    }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&aux->cready[b], TCB_EPI_WARPS); ptx::mbar_init(&aux->cfree[b], 1); }
    aux->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmX);
    ptx::prefetch_tmap(&tmR);
    ptx::prefetch_tmap(&tmOut);
  }
  if (warp == 1) { ptx::tmem_alloc(&aux->tmem_base, 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // TMEM columns: the Y buffers, then the M accumulator(s) (with two, the next problem's second products can run
  // while this problem's accumulator is written out)
  const uint32_t tmem_base = aux->tmem_base;
  constexpr uint32_t TM_M = 128u * TCB_YBUF;
  int timeout_site = 0;
  // one thread per role of CTA 0 stamps its events of the first tiles (nothing is recorded unless a buffer was given)
  const bool tracing = g.trace != nullptr && blockIdx.x == 0 && lane == 0;
#define TCB_TR(tile, ev) do { if (tracing && (tile) < TCB_TRACE_TILES) g.trace[(tile) * 16 + (ev)] = clock64(); } while (0)

  if (warp == 0) {
    if (lane == 0) {
      int xs = 0; uint32_t xph = 0;
      int lp = 0, itp = 0;
      bool ok = true;
      int issued = 0;
      for (int item = blockIdx.x; item < g.P * g.S && ok; item += gridDim.x, ++lp) {
        int p, t_begin, t_end;
        tcb_item(item, T, g.S, p, t_begin, t_end);
        if (!tc_wait(&aux->rempty, ((uint32_t)lp & 1u) ^ 1u, abort_flag)) { ok = false; timeout_site = 11; break; }
        ptx::mbar_expect_tx(&aux->rfull, TCB_TILE_BYTES);
        ptx::tma_load_2d(sR, &tmR, &aux->rfull, 0, (g.p0 + p) * TCB_D);
        ptx::tma_load_2d(sR + 16384, &tmR, &aux->rfull, 64, (g.p0 + p) * TCB_D);
        for (int t = t_begin; t < t_end; ++t) {
          if (!tc_wait(&aux->xempty[xs], xph ^ 1u, abort_flag)) { ok = false; timeout_site = 12; break; }
          uint8_t* dst = sX + xs * TCB_TILE_BYTES;
          ptx::mbar_expect_tx(&aux->xfull[xs], TCB_TILE_BYTES);
          const int c1 = g.xp_outer_tokens ? p : t * 128, c2 = g.xp_outer_tokens ? t * 128 : p;
          tma_load_3d(dst, &tmX, &aux->xfull[xs], 0, c1, c2);
          tma_load_3d(dst + 16384, &tmX, &aux->xfull[xs], 64, c1, c2);
          TCB_TR(itp, TCB_EV_TMA); ++itp;
          ++issued;
          if (++xs == TCB_XSTAGES) { xs = 0; xph ^= 1u; }
        }
      }
      if (!ok && issued > 0) {                     // let the copies in flight land before the CTA exits
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- first product: Y = X_tile R
    if (lane == 0) {
      // instruction descriptor: bf16 x bf16 -> fp32, M = N = 128; A K-major, B MN-major
      const uint32_t idesc1 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24) | (1u << 16);
      const uint32_t sR_a = ptx::smem_u32(sR), sX_a = ptx::smem_u32(sX);
      int xs = 0; uint32_t xph = 0;
      int it = 0, lp = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < g.P * g.S && ok; item += gridDim.x, ++lp) {
        int p_item, tb_item, te_item;
        tcb_item(item, T, g.S, p_item, tb_item, te_item);
        const int T_item = te_item - tb_item;
        if (!tc_wait(&aux->rfull, (uint32_t)lp & 1u, abort_flag)) { ok = false; timeout_site = 20; break; }
        for (int t = 0; t < T_item && ok; ++t, ++it) {
          const int yb = it % TCB_YBUF;
          if (!tc_wait(&aux->xfull[xs], xph, abort_flag)) { ok = false; timeout_site = 22; break; }
          if (!tc_wait(&aux->yempty[yb], (((uint32_t)(it / TCB_YBUF)) & 1u) ^ 1u, abort_flag)) { ok = false; timeout_site = 24; break; }
          ptx::tc_fence_after();
          TCB_TR(it, TCB_EV_MMA1);
          const uint32_t xa = sX_a + xs * TCB_TILE_BYTES;
#pragma unroll
          for (int j = 0; j < 8; ++j)        // 16 features per instruction: chunk j/4, 32 bytes per step inside the swizzled row
            ptx::umma_bf16(tmem_base + yb * 128, tc_smem_desc(xa + (j >> 2) * 16384 + (j & 3) * 32, 16, 1024),
                           tc_smem_desc(sR_a + j * 2048, 16384, 1024), idesc1, j > 0 ? 1u : 0u);
          ptx::umma_commit(&aux->yfull[yb]);
          if (t == T_item - 1) ptx::umma_commit(&aux->rempty);     // R may be replaced once every first product has run
          if (++xs == TCB_XSTAGES) { xs = 0; xph ^= 1u; }
        }
      }
    }
  } else if (warp == TCB_MMA2_WARP) {
    // ---------------------------------------------------------------- second product: M += X_tile^T C'
    if (lane == 0) {
      // both operands MN-major (contraction over the tokens, the slow dimension of both tiles)
      const uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24) |
                              (1u << 15) | (1u << 16);
      const uint32_t sX_a = ptx::smem_u32(sX), sC_a = ptx::smem_u32(sC);
      int xs = 0; uint32_t xph = 0;
      int it = 0, lp = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < g.P * g.S && ok; item += gridDim.x, ++lp) {
        int p_item, tb_item, te_item;
        tcb_item(item, T, g.S, p_item, tb_item, te_item);
        const int T_item = te_item - tb_item;
        // the accumulator of the previous problem has been read out
        const int mb = lp % TCB_MBUF;
        if (!tc_wait(&aux->mempty[mb], (((uint32_t)(lp / TCB_MBUF)) & 1u) ^ 1u, abort_flag)) { ok = false; timeout_site = 21; break; }
        for (int t = 0; t < T_item && ok; ++t, ++it) {
          const int cb = it & 1;
          if (!tc_wait(&aux->xfull[xs], xph, abort_flag)) { ok = false; timeout_site = 25; break; }
          if (!tc_wait(&aux->cready[cb], ((uint32_t)it >> 1) & 1u, abort_flag)) { ok = false; timeout_site = 23; break; }
          ptx::tc_fence_after();
          TCB_TR(it, TCB_EV_MMA2);
          const uint32_t xa = sX_a + xs * TCB_TILE_BYTES, ca = sC_a + cb * TCB_TILE_BYTES;
#pragma unroll
          for (int j = 0; j < 8; ++j)          // 16 tokens per instruction: two 8-row groups, 2048 bytes per step
            ptx::umma_bf16(tmem_base + TM_M + mb * 128, tc_smem_desc(xa + j * 2048, 16384, 1024), tc_smem_desc(ca + j * 2048, 16384, 1024),
                           idesc2, (t > 0 || j > 0) ? 1u : 0u);
          ptx::umma_commit(&aux->xempty[xs]);
          ptx::umma_commit(&aux->cfree[cb]);
          if (++xs == TCB_XSTAGES) { xs = 0; xph ^= 1u; }
        }
        if (ok) ptx::umma_commit(&aux->mfull[mb]);
      }
    }
  } else {
    const int q = warp & 3;                        // TMEM lane quarter this warp may read
    const int grp = (warp - 2) >> 3;               // with two groups: group 0 takes the even tiles (and C' buffer 0), group 1 the odd ones
    const int ew = (warp - 2) & 7;                 // 0..7 inside the group
    const int half = ew >> 2;                      // which 64 of the 128 columns this warp handles
    const int r = q * 32 + lane;                   // token inside the tile; later: row of M
    int it = 0, lp = 0;
    uint32_t wo_count = 0;                         // write-outs this warp's group has done
    bool ok = true;
    for (int item = blockIdx.x; item < g.P * g.S && ok; item += gridDim.x, ++lp) {
      int p, t_begin, t_end;
      tcb_item(item, T, g.S, p, t_begin, t_end);
      double acc = 0.0;
      int skipped = 0, nonfinite = 0;
      for (int t = t_begin; t < t_end && ok; ++t, ++it) {
        if (TCB_EPI_GROUPS == 2 && (it & 1) != grp) continue;
        // the write-out's tensor map was last used a whole problem ago: fetch it again a few tiles before the end
        if (lane == 0 && t + 2 * TCB_EPI_GROUPS >= t_end && t + TCB_EPI_GROUPS < t_end) ptx::prefetch_tmap(&tmOut);
        const int yb = it % TCB_YBUF, cb = it & 1;
        const uint32_t par3 = ((uint32_t)(it / TCB_YBUF)) & 1u, par2 = ((uint32_t)it >> 1) & 1u;
        const bool tr_epi = ew == 0;                       // the first warp of the tile's group stamps the epilogue
        if (tr_epi) TCB_TR(it, TCB_EV_EPI_BEGIN);
        if (!tc_wait(&aux->yfull[yb], par3, abort_flag)) { ok = false; timeout_site = 32; break; }
        ptx::tc_fence_after();
        if (tr_epi) TCB_TR(it, TCB_EV_EPI_Y);
        const uint32_t t_addr = tmem_base + (uint32_t)(yb * 128) + ((uint32_t)(q * 32) << 16);
        uint8_t* crow = sC + cb * TCB_TILE_BYTES;
        // a1: the row's scale, taken from the rotated row: ||x R~|| with R~ the bf16 copy of the orthogonal R the
        // product uses.  It differs from ||x|| by at most ||R~ R~^T - I||_2 / 2 (about 1e-4 for a typical row at
        // d = 128), an order below the rounding of the scale itself to bf16 in the target tile, and costs no pass
        // over the input tile in shared memory, whose bandwidth bounds this kernel.  Every warp reads the whole
        // row (both warps of a row pair get the same sum); with fake-quantisation the same pass finds the row's range.
        if (tr_epi) TCB_TR(it, TCB_EV_NORM_BEGIN);
        float ss;
        float vmax = -3.0e38f, vmin = 3.0e38f;
        {
          float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;       // four chains; added in a fixed order
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            float v[32];
            ptx::tmem_ld32(t_addr + (uint32_t)(c * 32), v);
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              s0 = fmaf(v[i], v[i], s0); s1 = fmaf(v[i + 1], v[i + 1], s1);
              s2 = fmaf(v[i + 2], v[i + 2], s2); s3 = fmaf(v[i + 3], v[i + 3], s3);
            }
            if (g.qs.bits > 0) {
#pragma unroll
              for (int i = 0; i < 32; ++i) { vmax = fmaxf(vmax, v[i]); vmin = fminf(vmin, v[i]); }
            }
          }
          ss = (s0 + s1) + (s2 + s3);
        }
        if (tr_epi) TCB_TR(it, TCB_EV_NORM_END);
        const bool valid = (t * 128 + r) < g.n;
        const bool good = valid && (ss > 0.f) && (ss <= 3.0e38f);
        if (valid && !good) {
          // the row takes no part; a non-finite one is also zeroed in the input tile for the second product (this
          // warp's 64 columns; made visible to the tensor-core proxy by the fence before the tile is handed over)
          if (half == 0) { ++skipped; if (!(ss == 0.f)) nonfinite = 1; }
          uint8_t* xrow = sX + (it % TCB_XSTAGES) * TCB_TILE_BYTES;
#pragma unroll
          for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(xrow + tcb_piece(r, half * 8 + c)) = make_uint4(0, 0, 0, 0);
        }
        const float rn = good ? 1.0f / sqrtf(ss) : 0.f;
        const uint32_t rn_bits = bf16_bits(rn);
        if (tr_epi) TCB_TR(it, TCB_EV_EPI_NORMS);
        RowQuant rq{0.f, 0.f, 0.f, 0.f};
        if (g.qs.bits > 0) rq = row_quant(g.qs, vmax, vmin, good);
        // the target buffer is needed only now (the second product of the tile two back has read it)
        if (!tc_wait(&aux->cfree[cb], par2 ^ 1u, abort_flag)) { ok = false; timeout_site = 31; break; }
        if (tr_epi) TCB_TR(it, TCB_EV_EPI_CFREE);
        const bool live = (g.qs.bits == 0) ? good : (rq.inv > 0.f);
        float acc_t = 0.f;
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          const int c = half * 2 + cc;
          float v[32];
          ptx::tmem_ld32(t_addr + (uint32_t)(c * 32), v);
          if (tr_epi) TCB_TR(it, cc == 0 ? TCB_EV_EPI_LD0 : TCB_EV_EPI_LD1);
          uint32_t w[16];
          if (g.qs.bits > 0) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float a = fminf(fmaxf(rintf(v[2 * i] * rq.inv), rq.klo), rq.khi);
              const float b = fminf(fmaxf(rintf(v[2 * i + 1] * rq.inv), rq.klo), rq.khi);
              acc_t += fabsf(a) + fabsf(b);
              const uint32_t lo = (a == 0.f) ? 0u : (rn_bits | ((__float_as_uint(a) >> 16) & 0x8000u));
              const uint32_t hi = (b == 0.f) ? 0u : (rn_bits | ((__float_as_uint(b) >> 16) & 0x8000u));
              w[i] = live ? (lo | (hi << 16)) : 0u;
            }
          } else {
            // two elements per instruction: the sign bits and a non-zero mask (0xffff per half that is not +-0) of the
            // packed bf16 pair; the objective comes from the accumulator at the end of the problem
            const uint32_t rn2 = live ? (rn_bits | (rn_bits << 16)) : 0u;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const uint32_t pk = bf16x2_pack(v[2 * i], v[2 * i + 1]);
              uint32_t nz;
              asm("set.neu.u32.bf16x2 %0, %1, %2;" : "=r"(nz) : "r"(pk), "r"(0u));
              w[i] = (rn2 | (pk & 0x80008000u)) & nz;
            }
          }
#pragma unroll
          for (int k = 0; k < 4; ++k)
            *reinterpret_cast<uint4*>(crow + tcb_piece(r, c * 4 + k)) = make_uint4(w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]);
          if (g.signs != nullptr && valid) {
            // the decisions exactly as they enter the second product: sign bit and non-zero test of each bf16 half of C'
            uint32_t sb[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              uint32_t o = 0;
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const uint32_t pr = w[2 * k + e];
                const uint32_t lo = pr & 0xffffu, hi = pr >> 16;
                o |= ((lo & 0x7fffu) ? ((lo & 0x8000u) ? 0xffu : 1u) : 0u) << (16 * e);
                o |= ((hi & 0x7fffu) ? ((hi & 0x8000u) ? 0xffu : 1u) : 0u) << (16 * e + 8);
              }
              sb[k] = o;
            }
            uint4* so = reinterpret_cast<uint4*>(g.signs + ((long long)p * g.n + (long long)t * 128 + r) * TCB_D + c * 32);
            so[0] = make_uint4(sb[0], sb[1], sb[2], sb[3]);
            so[1] = make_uint4(sb[4], sb[5], sb[6], sb[7]);
          }
          if (tr_epi && cc == 0) TCB_TR(it, TCB_EV_EPI_ST0);
        }
        if (live && g.qs.bits > 0) acc += (double)(rn * rq.delta) * (double)acc_t;
        // hand the tile to the second product: shared-memory writes must be visible to the tensor-core proxy
        ptx::tc_fence_before();
        ptx::fence_proxy_async();
        __syncwarp();                              // one arrival per warp: every lane's fences precede it
        if (tr_epi) TCB_TR(it, TCB_EV_EPI_END);
        if (lane == 0) {
          ptx::mbar_arrive(&aux->cready[cb]);
          ptx::mbar_arrive(&aux->yempty[yb]);
        }
      }
      if (!ok) break;
      if (half == 0) {                               // rows skipped in this problem (counted once per row)
        int wsk = skipped, wnf = nonfinite;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { wsk += __shfl_xor_sync(0xffffffffu, wsk, o); wnf |= __shfl_xor_sync(0xffffffffu, wnf, o); }
        if (lane == 0) {
          if (wsk) atomicAdd(reinterpret_cast<unsigned long long*>(&g.st[p].step_skipped), (unsigned long long)wsk);
          if (wnf) atomicOr(&g.st[p].status_flags, STATUS_FLAG_NONFINITE);
        }
      }
      // The problem's cross-covariance: TMEM accumulator -> += global fp32 M (row r of M = feature r of X^T).  With two
      // groups, the one that owned the problem's last tile writes all of it out (each warp 32 rows x 64 columns) while
      // the other goes straight on to the next problem's first tile, so the second products resume as soon as the
      // accumulator has been read.
      const int wo_grp = (TCB_EPI_GROUPS == 2) ? ((it - 1) & 1) : 0;
      if (grp == wo_grp) {
        const int mb = lp % TCB_MBUF;
        if (ew == 0) TCB_TR(it - 1, TCB_EV_OUT_WAIT);
        // Every second product issued so far has finished once the accumulator is complete, and this group's next
        // target tile comes after the write-out, so its C' buffer is idle: each warp borrows 4 KB of it as staging
        // area.  One item per problem: added into M (one addition per element and launch, so the result does not
        // depend on any order); several: stored to the item's partial, summed in item order afterwards.
        const uint32_t t_addr = tmem_base + TM_M + (uint32_t)(mb * 128) + ((uint32_t)(q * 32) << 16);
        uint8_t* stg = sC + grp * TCB_TILE_BYTES + ew * 4096;
        const int y0 = ((g.S == 1) ? (g.p0 + p) : item) * TCB_D + q * 32;
        if (!tcb_write_out(&aux->mfull[mb], ((uint32_t)(lp / TCB_MBUF)) & 1u, abort_flag, t_addr, stg, lane, &tmOut, y0, g.S == 1,
                           half * 2, half * 2 + 2, &aux->mempty[mb],
                           (tracing && ew == 0 && it - 1 < TCB_TRACE_TILES) ? g.trace + (it - 1) * 16 + TCB_EV_OUT_BEGIN : nullptr)) {
          ok = false; timeout_site = 33; break;
        }
        if (ew == 0) TCB_TR(it - 1, TCB_EV_OUT_END);
        // the group's warps stay off their C' buffer until all of them have finished staging in it (bounded wait)
        if (lane == 0) ptx::mbar_arrive(&aux->pdone[grp]);
        if (!tc_wait(&aux->pdone[grp], wo_count & 1u, abort_flag)) { ok = false; timeout_site = 36; break; }
        ++wo_count;
      }
      // With fake-quantisation every warp leaves its objective partial of the problem (summed in a fixed order by the
      // kernel that follows); without, the objective is <R, M> / sqrt(d) and is formed from M when it is read.
      if (g.qs.bits > 0) {
        const double wsum = warp_sum_d(acc);
        if (lane == 0) g.part_d[(long long)item * TCB_PARTS + grp * 8 + ew] = wsum;
      }
    }
  }

  if (timeout_site != 0) {
    atomicOr(&g.st[0].status_flags, STATUS_FLAG_TIMEOUT);
    g.st[0].timeout_site = timeout_site;
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Per-head problems without fake-quantisation: between two updates R is fixed and M = sum of X~^T S, so the objective
// sum_rows <x~ R, s> / sqrt(d) equals <R, M> / sqrt(d) (Eq. 4 with the corner target); the step kernel does not
// accumulate it.  It is formed from M by the update kernel and, for a read in between, by tcb_objective_kernel.
inline bool tcb_objective_from_m(const TcHost& h) { return h.P > 1 && h.qs.bits == 0; }

// st[p].J = <R_p, M_p> / sqrt(d), summed in a fixed order.  grid P, 256 threads.
static __global__ void tcb_objective_kernel(DevState* st, const float* __restrict__ M, const float* __restrict__ R) {
  const int p = blockIdx.x;
  __shared__ double red[8];
  const float4* m4 = reinterpret_cast<const float4*>(M + (size_t)p * TCB_D * TCB_D);
  const float4* r4 = reinterpret_cast<const float4*>(R + (size_t)p * TCB_D * TCB_D);
  double v = 0.0;
  for (int i = threadIdx.x; i < TCB_D * TCB_D / 4; i += 256) {
    const float4 m = m4[i], q = r4[i];
    v += (double)m.x * q.x + (double)m.y * q.y + (double)m.z * q.z + (double)m.w * q.w;
  }
  const double tot = block_sum_d<256>(v, red);
  if (threadIdx.x == 0) st[p].J = tot / sqrt((double)TCB_D);
}

inline int tcb_refresh_objective(TcHost& h, cudaStream_t s) {
  if (!tcb_objective_from_m(h)) return CONQUR_OK;
  tcb_objective_kernel<<<h.P, 256, 0, s>>>(h.st, h.M, h.R);
  if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
  if (h.prof) h.prof->count(K_OTHER);
  return CONQUR_OK;
}

// M[p] += partial[p * S + 0] + ... + partial[p * S + S - 1], in that order.  grid (16, problems), 256 threads.
static __global__ void tcb_sum_partials_kernel(float* __restrict__ M, const float* __restrict__ part, int S) {
  const int p = blockIdx.y;
  const int i = (blockIdx.x * 256 + threadIdx.x) * 4;
  float4 m = *reinterpret_cast<const float4*>(M + (size_t)p * TCB_D * TCB_D + i);
  for (int sp = 0; sp < S; ++sp) {
    const float4 v = *reinterpret_cast<const float4*>(part + ((size_t)p * S + sp) * TCB_D * TCB_D + i);
    m.x += v.x; m.y += v.y; m.z += v.z; m.w += v.w;
  }
  *reinterpret_cast<float4*>(M + (size_t)p * TCB_D * TCB_D + i) = m;
}

// fp32 -> bf16 staging of a batched input (problem p, row i at X + p*pstride + i*ld) into a dense P x n x 128 copy
__global__ void tcb_stage_f32_kernel(const float* __restrict__ X, int64_t n, int64_t ld, int64_t pstride, int P,
                                     __nv_bfloat16* __restrict__ Xs) {
  const int64_t total4 = (int64_t)P * n * (TCB_D / 4);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total4; i += (int64_t)gridDim.x * blockDim.x) {
    const int c4 = (int)(i % (TCB_D / 4));
    const int64_t row = (i / (TCB_D / 4)) % n, p = i / ((TCB_D / 4) * n);
    const float* src = X + p * pstride + row * ld + c4 * 4;
    uint2 o;
    o.x = bf16_bits(src[0]) | (bf16_bits(src[1]) << 16);
    o.y = bf16_bits(src[2]) | (bf16_bits(src[3]) << 16);
    *reinterpret_cast<uint2*>(Xs + (p * n + row) * TCB_D + c4 * 4) = o;
  }
}

// 3-D view of a batched bf16 input: (128 features, n rows with stride ld, P problems with stride pstride); box 64 x 128 x 1.
// Dimensions are ordered by stride: (column, token, problem) when a problem's rows lie together, (column, problem,
// token) when the problems' columns are interleaved inside one row (problem stride < row stride).  Either way a box
// is 128 tokens x 64 columns of one problem and lands in shared memory row by row.
inline int tcb_make_x_tmap(CUtensorMap* tm, const void* ptr, uint64_t n, uint64_t ld, uint64_t pstride, uint64_t P,
                           int* outer_tokens) {
  PFN_encodeTiled fn = tc_encode_fn();
  if (!fn) return CONQUR_ERR_CUDA;
  const uint64_t ps = P > 1 ? pstride : ld * n;
  *outer_tokens = ps < ld ? 1 : 0;
  const cuuint64_t dims_tp[3] = {TCB_D, n, P}, dims_pt[3] = {TCB_D, P, n};
  const cuuint64_t strides_tp[2] = {ld * 2, ps * 2}, strides_pt[2] = {ps * 2, ld * 2};
  const cuuint32_t box_tp[3] = {64, 128, 1}, box_pt[3] = {64, 1, 128};
  const cuuint64_t* dims = *outer_tokens ? dims_pt : dims_tp;
  const cuuint64_t* strides = *outer_tokens ? strides_pt : strides_tp;
  const cuuint32_t* box = *outer_tokens ? box_pt : box_tp;
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::fprintf(stderr, "conqur: cuTensorMapEncodeTiled (batched input) failed (%d)\n", (int)r);
    return CONQUR_ERR_INVALID_ARG;
  }
  return CONQUR_OK;
}

// One streamed batch for all P problems.  X: device, bf16 or fp32 (fp32 is first rounded into the staging copy).
// Problems [p0, p0 + np) of the context; X holds those np problems.
inline int tcb_step(TcHost& h, cudaStream_t s, const void* X, int in_dtype, int64_t n, int64_t ld, int64_t pstride, int p0,
                    int np, int8_t* signs_out = nullptr, long long* trace = nullptr) {
  static std::atomic<unsigned long long> attr_dev_mask{0};      // the attribute is per device
  const unsigned long long dev_bit = 1ull << (h.device & 63);
  if (!(attr_dev_mask.load(std::memory_order_acquire) & dev_bit)) {
    if (cudaFuncSetAttribute(tcb_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TCB_SMEM_BYTES) != cudaSuccess)
      return CONQUR_ERR_CUDA;
    attr_dev_mask.fetch_or(dev_bit, std::memory_order_release);
  }
  const void* src = X;
  int64_t src_ld = ld, src_ps = pstride;
  if (in_dtype == CONQUR_F32) {
    __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Xs);
    tcb_stage_f32_kernel<<<tc_ew_blocks((int64_t)np * n * (TCB_D / 4)), 256, 0, s>>>(static_cast<const float*>(X), n, ld,
                                                                                    pstride, np, Xs);
    if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
    if (h.prof) h.prof->count(K_ROWNORM);
    src = Xs; src_ld = TCB_D; src_ps = n * TCB_D;
  } else if ((reinterpret_cast<uintptr_t>(X) & 15) || (ld % 8) || (pstride % 8)) {
    return CONQUR_ERR_INVALID_ARG;            // TMA needs 16-byte aligned rows and problem bases
  }
  CUtensorMap tmX;
  int outer_tokens = 0;
  int rc = tcb_make_x_tmap(&tmX, src, (uint64_t)n, (uint64_t)src_ld, (uint64_t)src_ps, (uint64_t)np, &outer_tokens);
  if (rc) return rc;
  TcbStepArgs g{};
  g.n = (int)n; g.P = np; g.p0 = p0; g.qs = h.qs; g.xp_outer_tokens = outer_tokens;
  g.M = h.M + (size_t)p0 * TCB_D * TCB_D; g.part_d = h.part_d; g.st = h.st + p0; g.signs = signs_out;
  g.trace = trace;
  // few problems: split each problem's tokens over several CTAs (partials land in the idle Newton-Schulz buffers,
  // 4 P matrices of 128 x 128 starting at Xa, and are summed in a fixed order)
  const int T = (int)((n + 127) / 128);
  int S = 1;
  if (np < h.num_sms) S = std::max(1, std::min(std::min(h.num_sms / np, T), 4 * h.P / np));
  g.S = S; g.Mpart = h.Xa;
  const int items = np * S;
  const int grid = items < h.num_sms ? items : h.num_sms;
  Prof::Rec rec{};
  const bool timed = h.prof && h.prof->enabled;
  if (timed) {
    rec.cls = K_ROTATE; rec.flops = 4.0 * (double)np * (double)n * TCB_D * TCB_D; rec.ns_k = -1; rec.nseg = 1;
    rec.e0 = h.prof->get_event(); rec.e1 = h.prof->get_event();
    cudaEventRecord(rec.e0, s);
  }
  tcb_step_kernel<<<grid, TCB_THREADS, TCB_SMEM_BYTES, s>>>(tmX, h.tmRb_mn, S == 1 ? h.tmM_blk : h.tmMpart_blk, g);
  if (timed) { cudaEventRecord(rec.e1, s); h.prof->open.push_back(rec); }
  if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
  if (h.prof) h.prof->count(K_ROTATE);
  if (S > 1) {
    tcb_sum_partials_kernel<<<dim3(16, np), 256, 0, s>>>(g.M, g.Mpart, S);
    if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
    if (h.prof) h.prof->count(K_OTHER);
  }
  finalize_step_kernel<<<np, 256, 0, s>>>(g.st, h.qs.bits > 0 ? h.part_d : nullptr, S * TCB_PARTS, n, 1.0 / std::sqrt((double)TCB_D));
  if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
  if (h.prof) h.prof->count(K_OTHER);
  return CONQUR_OK;
}

// ------------------------------------------------------------------ fused polar update of many 128 x 128 problems
// One CTA runs the whole Newton-Schulz iteration of one problem at a time with everything on chip: the iterate as
// a bf16 (hi, lo) pair in shared memory, G = X^T X and the products in TMEM, the scalar control in one thread.
// Per step (phases are strictly sequential; 128 threads = 128 rows):
//   G = X^T X (hi hi + hi lo + lo hi)      -> TMEM [0,128)
//   statistics of G - I, control decision, E = G - tau I as bf16           -> shared memory
//   E E                                     -> TMEM [128,256)
//   B = beta2 E E + beta1 E - kappa I as bf16                              -> shared memory (over E)
//   X B (hi, + lo while the schedule asks)  -> TMEM [0,128)
//   X <- (gamma + kappa) X + X B, tau = ||X||_F^2 / d, split into (hi, lo) -> shared memory
// Two CTAs fit one SM (96 KB of shared memory and 256 TMEM columns each), so one problem's element-wise phases
// overlap the other's products.
constexpr int TCBU_THREADS = 256;            // 128 rows x 2 column halves
constexpr int TCBU_SMEM_BYTES = 3 * TCB_TILE_BYTES + 4096 + 1024;

struct TcbUpdAux {
  uint64_t mbar;
  uint32_t tmem_base;
  int abort_flag;
  int done;
  float tau, x0s, lam;
  float coef[4];
  int seg_x;
  double red_d[8], red_t[8];
  float red_f[8];
  DevState state;                    // the problem's state while it is being iterated (written back once at the end)
  SchedEntry sched[NS_SCHED_MAX];    // the polynomial schedule (copied once per CTA)
};

static_assert(sizeof(TcbUpdAux) <= 4096, "the control block must fit its reserved shared memory");

struct TcbUpdArgs {
  int P;
  int objective_from_m;        // 1: the objective consumed by this update is <R, M> / sqrt(d), formed here
  float* M; float* R;          // P x 128 x 128 fp32
  __nv_bfloat16* Rb;           // P x 128 x 128: the rotations in bf16 (operand of the step kernel), rewritten with R
  DevState* st;
  NsControlParams ncp;
  float prior_rel, margin;
};

__device__ __forceinline__ double tcbu_block_sum(double v, double* red, int warp, int lane) {
  v = warp_sum_d(v);
  if (lane == 0) red[warp] = v;
  __syncthreads();
  const double t = ((red[0] + red[1]) + (red[2] + red[3])) + ((red[4] + red[5]) + (red[6] + red[7]));
  __syncthreads();
  return t;
}

__global__ void __launch_bounds__(TCBU_THREADS, 2) tcb_update_kernel(const TcbUpdArgs g) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sXh = smem;
  uint8_t* sXl = smem + TCB_TILE_BYTES;
  uint8_t* sEB = smem + 2 * TCB_TILE_BYTES;
  TcbUpdAux* aux = reinterpret_cast<TcbUpdAux*>(smem + 3 * TCB_TILE_BYTES);
  volatile int* abort_flag = &aux->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = threadIdx.x & 127;                 // the row this thread works on everywhere
  const int half = threadIdx.x >> 7;               // ... and which 64 of its 128 columns
  const int c_diag = r >> 5;                       // the 32-column chunk holding the row's diagonal element (one per warp)
  if (threadIdx.x == 0) {
    ptx::mbar_init(&aux->mbar, 1);
    aux->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 0) { ptx::tmem_alloc(&aux->tmem_base, 256); ptx::tmem_relinquish(); }
  for (int i = threadIdx.x; i < g.ncp.n_sched && i < NS_SCHED_MAX; i += TCBU_THREADS) aux->sched[i] = g.ncp.sched[i];
  NsControlParams ncp = g.ncp;
  ncp.sched = aux->sched;                          // control decisions read the shared-memory copy
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = aux->tmem_base;
  const uint32_t t_row = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);      // this warp's 32 TMEM lanes
  const uint32_t aXh = ptx::smem_u32(sXh), aXl = ptx::smem_u32(sXl), aEB = ptx::smem_u32(sEB);
  const uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  const uint32_t idesc_mm = idesc_base | (1u << 15) | (1u << 16);       // both operands read "transposed" (MN-major)
  const uint32_t idesc_km = idesc_base | (1u << 16);                    // A as stored (K-major), B MN-major
  uint32_t mph = 0;
  bool timed_out = false;
  const float isd = rsqrtf((float)TCB_D);

  // descriptor of k-step j (16 of the 128 contraction indices) of a 128 x 128 tile held as two swizzled 64-column chunks
  auto desc_k = [](uint32_t base, int j) { return tc_smem_desc(base + (j >> 2) * 16384 + (j & 3) * 32, 16, 1024); };   // contraction along columns
  auto desc_mn = [](uint32_t base, int j) { return tc_smem_desc(base + j * 2048, 16384, 1024); };                        // contraction along rows
  // all threads: make shared-memory writes visible to the tensor cores, then thread 0 issues `issue`; the block barrier
  // inside also publishes whatever the threads wrote to the control block before the call.  wait_products: everyone
  // waits for the products issued last.  Work placed between the two overlaps the products.
  auto issue_products = [&](auto issue) {
    ptx::fence_proxy_async();
    ptx::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) {
      ptx::tc_fence_after();
      issue();
      ptx::umma_commit(&aux->mbar);
    }
  };
  auto wait_products = [&]() -> bool {
    const bool okw = tc_wait(&aux->mbar, mph, abort_flag);
    mph ^= 1u;
    ptx::tc_fence_after();
    return okw;
  };
  auto issue_gram = [&] {                          // G = X^T X (hi hi + hi lo + lo hi)
    const uint32_t aa[3] = {aXh, aXh, aXl}, bb[3] = {aXh, aXl, aXh};
#pragma unroll
    for (int seg = 0; seg < 3; ++seg)
#pragma unroll
      for (int j = 0; j < 8; ++j)
        ptx::umma_bf16(tmem_base, desc_mn(aa[seg], j), desc_mn(bb[seg], j), idesc_mm, (seg > 0 || j > 0) ? 1u : 0u);
  };

  NsCtl ctl{};                                     // thread 0 only
  for (int p = blockIdx.x; p < g.P && !timed_out; p += gridDim.x) {
    DevState* const sg = g.st + p;                 // global copy: read once, written back once
    DevState* const s = &aux->state;
    if (threadIdx.x == 0) *s = *sg;
    const float4* M4 = reinterpret_cast<const float4*>(g.M + (long long)p * TCB_D * TCB_D);
    const float4* R4 = reinterpret_cast<const float4*>(g.R + (long long)p * TCB_D * TCB_D);
    // ---- scale: lam = prior_rel ||M||_F / sqrt(d), X_0 = (M + lam R) / (||M + lam R||_F (1 + margin)), with
    // ||M + lam R||^2 = ||M||^2 + 2 lam <M, R> + lam^2 ||R||^2; <R, M> / sqrt(d) is also the objective this update
    // consumes where the step kernel does not accumulate it.  One coalesced pass, sums in double in a fixed order.
    const bool need_r = g.objective_from_m || g.prior_rel > 0.f;
    double ssq = 0.0, dot = 0.0, rsq = 0.0;
#pragma unroll 8
    for (int k = 0; k < TCB_D * TCB_D / 4 / TCBU_THREADS; ++k) {
      const int i = k * TCBU_THREADS + threadIdx.x;
      const float4 m = M4[i];
      ssq += (double)m.x * m.x + (double)m.y * m.y + (double)m.z * m.z + (double)m.w * m.w;
      if (need_r) {
        const float4 q = R4[i];
        dot += (double)m.x * q.x + (double)m.y * q.y + (double)m.z * q.z + (double)m.w * q.w;
        rsq += (double)q.x * q.x + (double)q.y * q.y + (double)q.z * q.z + (double)q.w * q.w;
      }
    }
    const double m2 = tcbu_block_sum(ssq, aux->red_d, warp, lane);
    if (need_r) {
      dot = tcbu_block_sum(dot, aux->red_d, warp, lane);
      rsq = tcbu_block_sum(rsq, aux->red_d, warp, lane);
    }
    if (g.objective_from_m && threadIdx.x == 0) s->J = dot / sqrt((double)TCB_D);
    const float lam = g.prior_rel * (float)sqrt(m2) * isd;
    double fro2 = m2;
    if (g.prior_rel > 0.f) fro2 = fmax(m2 + 2.0 * (double)lam * dot + (double)lam * (double)lam * rsq, 0.0);
    if (threadIdx.x == 0) {
      const float fro = (float)sqrt(fro2);
      const bool ok = (fro > 0.f) && (fro <= 3.0e38f) && (s->N > 0);
      s->lam = lam; s->scale = fro;
      s->x0_scale = ok ? 1.0f / (fro * (1.0f + g.margin)) : 0.f;
      s->ns_done = ok ? 0 : NS_DONE_FAILED;
      s->ns_steps_used = 0; s->ns_final_buf = 0; s->seg_x = 2;
      ns_arm_lifting(s, g.ncp.n_lift_init);
      s->tau = 1.0f / ((1.0f + g.margin) * (1.0f + g.margin) * (float)TCB_D);
      aux->done = s->ns_done; aux->tau = s->tau; aux->x0s = s->x0_scale; aux->lam = lam;
      ns_ctl_load(ctl, s);                          // thread 0 keeps the decision's state in registers from here on
    }
    __syncthreads();
    if (!aux->done) {
      const float x0s = aux->x0s;
#pragma unroll 4
      for (int k = 0; k < TCB_D * TCB_D / 4 / TCBU_THREADS; ++k) {
        const int i = k * TCBU_THREADS + threadIdx.x;             // float4 i: row i / 32, columns 4 (i % 32)..+3
        float4 a = M4[i];
        if (lam != 0.f) {
          const float4 q = R4[i];
          a.x = fmaf(lam, q.x, a.x); a.y = fmaf(lam, q.y, a.y); a.z = fmaf(lam, q.z, a.z); a.w = fmaf(lam, q.w, a.w);
        }
        uint32_t h0, h1, l0, l1;
        bf16x2_split(a.x * x0s, a.y * x0s, h0, l0);
        bf16x2_split(a.z * x0s, a.w * x0s, h1, l1);
        const uint32_t off = tcb_piece(i >> 5, (i & 31) >> 1) + (uint32_t)(i & 1) * 8u;
        *reinterpret_cast<uint2*>(sXh + off) = make_uint2(h0, h1);
        *reinterpret_cast<uint2*>(sXl + off) = make_uint2(l0, l1);
      }
      issue_products(issue_gram);
      bool gram_in_flight = true;
      for (int k = 0; k <= ncp.max_steps; ++k) {
        // ---- G = X^T X (issued before the loop / at the end of the previous step)
        gram_in_flight = false;
        if (!wait_products()) { timed_out = true; break; }
        // ---- statistics of G - I; E = G - tau I
        const float tau = aux->tau;
        float mx = 0.f, tr = 0.f;
        double sq = 0.0;
        // (the diagonal lies in one 32-column chunk per warp, c_diag: only that chunk pays for finding it)
        auto resid_chunk = [&](int c, auto has_diag) {
          float v[32];
          ptx::tmem_ld32(t_row + (uint32_t)(c * 32), v);
          const int dcol = r - c * 32;
          uint32_t w[16];
          float sq32 = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float e1 = v[i];
            if (decltype(has_diag)::value && i == dcol) { tr += v[i]; e1 -= 1.f; v[i] -= tau; }
            mx = fmaxf(mx, fabsf(e1));
            sq32 = fmaf(e1, e1, sq32);
          }
          sq += (double)sq32;
#pragma unroll
          for (int i = 0; i < 16; ++i) w[i] = bf16x2_pack(v[2 * i], v[2 * i + 1]);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            *reinterpret_cast<uint4*>(sEB + tcb_piece(r, c * 4 + q4)) = make_uint4(w[4 * q4], w[4 * q4 + 1], w[4 * q4 + 2], w[4 * q4 + 3]);
        };
#pragma unroll 1
        for (int c = half * 2; c < half * 2 + 2; ++c) {
          if (c == c_diag) resid_chunk(c, std::true_type{}); else resid_chunk(c, std::false_type{});
        }
        {
          const double wsq = warp_sum_d(sq), wtr = warp_sum_d((double)tr);
          const float wmx = warp_max(mx);
          if (lane == 0) { aux->red_d[warp] = wsq; aux->red_t[warp] = wtr; aux->red_f[warp] = wmx; }
        }
        // ---- E E, which does not depend on the control decision: issued first, the decision is taken while it runs
        // (a step that turns out to be the last one throws the product away)
        issue_products([&] {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            ptx::umma_bf16(tmem_base + 128, desc_k(aEB, j), desc_mn(aEB, j), idesc_km, j > 0 ? 1u : 0u);
        });
        if (threadIdx.x == 0) {
          double tsq = 0.0, ttr = 0.0;
          float tmx = 0.f;
          for (int i = 0; i < 8; ++i) { tsq += aux->red_d[i]; ttr += aux->red_t[i]; tmx = fmaxf(tmx, aux->red_f[i]); }
          const unsigned char log_entry = ns_control_decide(&ctl, tmx, tsq, ttr, k, 0, ncp);
          if (log_entry && k < 128) s->seg_log[k] = log_entry;
          aux->done = ctl.ns_done;
          aux->coef[0] = ctl.coef[0]; aux->coef[1] = ctl.coef[1]; aux->coef[2] = ctl.coef[2]; aux->coef[3] = ctl.coef[3];
          aux->seg_x = ctl.seg_x;
        }
        __syncthreads();
        if (!wait_products()) { timed_out = true; break; }
        if (aux->done) break;
        const float cg = aux->coef[0], cb1 = aux->coef[1], cb2 = aux->coef[2], ck = aux->coef[3];
        const int seg_x = aux->seg_x;
        // ---- B = beta2 E E + beta1 E - kappa I (over E: the product that read it has finished)
        auto poly_chunk = [&](int c, auto has_diag) {
          float gq[32], ee[32];
          ptx::tmem_ld32(t_row + (uint32_t)(c * 32), gq);
          ptx::tmem_ld32(t_row + 128u + (uint32_t)(c * 32), ee);
          const int dcol = r - c * 32;
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const bool on_diag = decltype(has_diag)::value && i == dcol;
            const float e = on_diag ? gq[i] - tau : gq[i];
            float b = fmaf(cb2, ee[i], cb1 * e);
            if (on_diag) b -= ck;
            ee[i] = b;
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) w[i] = bf16x2_pack(ee[2 * i], ee[2 * i + 1]);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            *reinterpret_cast<uint4*>(sEB + tcb_piece(r, c * 4 + q4)) = make_uint4(w[4 * q4], w[4 * q4 + 1], w[4 * q4 + 2], w[4 * q4 + 3]);
        };
#pragma unroll 1
        for (int c = half * 2; c < half * 2 + 2; ++c) {
          if (c == c_diag) poly_chunk(c, std::true_type{}); else poly_chunk(c, std::false_type{});
        }
        // ---- X B
        issue_products([&] {
#pragma unroll
          for (int j = 0; j < 8; ++j) ptx::umma_bf16(tmem_base, desc_k(aXh, j), desc_mn(aEB, j), idesc_km, j > 0 ? 1u : 0u);
          if (seg_x > 1) {
#pragma unroll
            for (int j = 0; j < 8; ++j) ptx::umma_bf16(tmem_base, desc_k(aXl, j), desc_mn(aEB, j), idesc_km, 1u);
          }
        });
        if (!wait_products()) { timed_out = true; break; }
        // ---- X <- (gamma + kappa) X + X B; tau of the next step
        double x2 = 0.0;
#pragma unroll 1
        for (int c = half * 2; c < half * 2 + 2; ++c) {
          float v[32];
          ptx::tmem_ld32(t_row + (uint32_t)(c * 32), v);
          float x2f = 0.f;
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const uint32_t off = tcb_piece(r, c * 4 + q4);
            const uint4 h4 = *reinterpret_cast<const uint4*>(sXh + off), l4 = *reinterpret_cast<const uint4*>(sXl + off);
            const uint32_t hh[4] = {h4.x, h4.y, h4.z, h4.w}, ll[4] = {l4.x, l4.y, l4.z, l4.w};
            uint32_t wh[4], wl[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float xa = __uint_as_float(hh[e] << 16) + __uint_as_float(ll[e] << 16);
              const float xb = __uint_as_float(hh[e] & 0xffff0000u) + __uint_as_float(ll[e] & 0xffff0000u);
              const float a = fmaf(cg, xa, v[q4 * 8 + 2 * e]), b = fmaf(cg, xb, v[q4 * 8 + 2 * e + 1]);
              x2f = fmaf(a, a, fmaf(b, b, x2f));
              bf16x2_split(a, b, wh[e], wl[e]);
            }
            *reinterpret_cast<uint4*>(sXh + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
            *reinterpret_cast<uint4*>(sXl + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
          }
          x2 += (double)x2f;
        }
        {
          const double wx2 = warp_sum_d(x2);
          if (lane == 0) aux->red_d[warp] = wx2;
        }
        // ---- the next step's G needs the new iterate but not its tau: issued now, tau is summed while it runs
        if (k < ncp.max_steps) { issue_products(issue_gram); gram_in_flight = true; } else { __syncthreads(); }
        if (threadIdx.x == 0) {
          const double tx2 = ((aux->red_d[0] + aux->red_d[1]) + (aux->red_d[2] + aux->red_d[3])) +
                             ((aux->red_d[4] + aux->red_d[5]) + (aux->red_d[6] + aux->red_d[7]));
          ctl.tau = (float)(tx2 * (1.0 / (double)TCB_D)); aux->tau = ctl.tau;
        }
        __syncthreads();
      }
      if (gram_in_flight && !timed_out) {          // nothing may be in flight when the tiles are reused
        if (!wait_products()) timed_out = true;
      }
    }
    if (timed_out) break;
    // ---- commit: R <- X, M <- 0, sums <- 0; or keep everything and latch the failure
    const bool converged = (aux->done == NS_DONE_CONVERGED);
    if (converged) {
      // coalesced: float4 i = row i / 32, columns 4 (i % 32)..+3; the bf16 copy the step kernel multiplies with is
      // the round-to-nearest of the fp32 rotation
      float4* Ro = reinterpret_cast<float4*>(g.R + (long long)p * TCB_D * TCB_D);
      float4* Mo = reinterpret_cast<float4*>(g.M + (long long)p * TCB_D * TCB_D);
      uint2* Rbo = reinterpret_cast<uint2*>(g.Rb + (long long)p * TCB_D * TCB_D);
#pragma unroll 4
      for (int k = 0; k < TCB_D * TCB_D / 4 / TCBU_THREADS; ++k) {
        const int i = k * TCBU_THREADS + threadIdx.x;
        const uint32_t off = tcb_piece(i >> 5, (i & 31) >> 1) + (uint32_t)(i & 1) * 8u;
        const uint2 h2 = *reinterpret_cast<const uint2*>(sXh + off), l2 = *reinterpret_cast<const uint2*>(sXl + off);
        float4 o;
        o.x = __uint_as_float(h2.x << 16) + __uint_as_float(l2.x << 16);
        o.y = __uint_as_float(h2.x & 0xffff0000u) + __uint_as_float(l2.x & 0xffff0000u);
        o.z = __uint_as_float(h2.y << 16) + __uint_as_float(l2.y << 16);
        o.w = __uint_as_float(h2.y & 0xffff0000u) + __uint_as_float(l2.y & 0xffff0000u);
        Ro[i] = o;
        Rbo[i] = make_uint2(bf16x2_pack(o.x, o.y), bf16x2_pack(o.z, o.w));
        Mo[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (threadIdx.x == 0) {
      ns_ctl_store(ctl, s);
      ns_adapt_lift_plan(s, ncp.n_sched - 1, converged ? 1 : 0);
      if (converged) {
        s->last_J = s->J; s->last_N = s->N; s->J = 0.0; s->N = 0; s->updates += 1;
        s->diag_pr = s->diag_rho = s->diag_qnum = s->diag_qden = 0.0;
        s->last_orth = s->e_max; s->last_fro = s->e_fro;
      } else {
        s->status_flags |= STATUS_FLAG_NS_FAILED;
      }
      *sg = *s;                                     // this CTA is the only writer of problem p's state during the update
    }
    __syncthreads();                                // aux->done is rewritten by the next problem
  }
  if (timed_out && threadIdx.x == 0) {
    atomicOr(&g.st[0].status_flags, STATUS_FLAG_TIMEOUT);
    g.st[0].timeout_site = 40;
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 256);
  }
}

inline int tcb_update(TcHost& h, cudaStream_t s, const NsControlParams& ncp, float prior_rel, float margin) {
  static std::atomic<unsigned long long> attr_dev_mask{0};      // the attribute is per device
  const unsigned long long dev_bit = 1ull << (h.device & 63);
  if (!(attr_dev_mask.load(std::memory_order_acquire) & dev_bit)) {
    if (cudaFuncSetAttribute(tcb_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TCBU_SMEM_BYTES) != cudaSuccess)
      return CONQUR_ERR_CUDA;
    attr_dev_mask.fetch_or(dev_bit, std::memory_order_release);
  }
  TcbUpdArgs g{};
  g.P = h.P; g.M = h.M; g.R = h.R; g.st = h.st; g.ncp = ncp; g.prior_rel = prior_rel; g.margin = margin;
  g.objective_from_m = tcb_objective_from_m(h) ? 1 : 0;
  g.Rb = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Rb);
  const int grid = h.P < 2 * h.num_sms ? h.P : 2 * h.num_sms;
  tcb_update_kernel<<<grid, TCBU_THREADS, TCBU_SMEM_BYTES, s>>>(g);
  if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
  if (h.prof) h.prof->count(K_NS_RESID);
  return CONQUR_OK;
}

}  // namespace conqur
