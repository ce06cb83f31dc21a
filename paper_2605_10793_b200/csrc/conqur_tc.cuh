// Tensor-core mode: one persistent, warp-specialised tcgen05 GEMM kernel (TMA -> 128B-swizzled
// shared memory ring -> tcgen05.mma with fp32 accumulators in TMEM -> tcgen05.ld epilogue) with the
// path's steps fused into its epilogues, plus the small element-wise kernels around it.
//
//   D[m][n] = sum_k A(m,k) * B(n,k),  BK = 64, bf16 operands, fp32 accumulation.  Default variant: clusters of two
//   CTAs work on one 256 x 256 tile with cta_group::2 instructions (each CTA loads half of the operands, CTA 0 issues
//   the products for both, each CTA's epilogue warps read their own 128 rows of the accumulator); a single-CTA
//   128 x BN variant remains for devices where such clusters cannot be resident.
//
// Each operand is a row-major bf16 matrix read in place in either orientation:
//   K-major : rows are m (or n), k contiguous      -> TMA box 64(k) x 128|BN rows
//   MN-major: rows are k, m (or n) contiguous      -> TMA boxes 64(m|n) x 64(k rows)
// so X^T C', X^T X and X B need no transposed copies.
//
// Split precision: an operand may be a stacked pair [hi; lo] of bf16 matrices (value = hi + lo).  With
// nseg = 3 the k loop runs three times over (hi,hi), (hi,lo), (lo,hi), accumulating into the same TMEM tile.
//
// Copies are never multicast (every CTA fetches its own operand tiles; the only cluster-wide signal is the commit
// that releases a stage in both CTAs of a pair).  Every mbarrier wait is bounded: on expiry
// the CTA raises a shared abort flag, latches STATUS_FLAG_TIMEOUT in the device state, drains its own
// copies with a bounded wait, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "../../include/conqur.h"
#include "conqur_internal.h"
#include "conqur_simt.cuh"

namespace conqur {

// ------------------------------------------------------------------ PTX wrappers
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* tmap, uint64_t* bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
// Shared memory -> global through the copy engine (a box of the tensor map, whole), stored or added element by
// element at the L2.  Asynchronous: the issuing thread commits the group and only waits until the source has been read.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tmap, const void* smem_src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tmap), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* tmap, const void* smem_src, int x, int y) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tmap), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D(tmem) (+)= A(smem desc) * B(smem desc); accumulate == 0 overwrites D.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier once every previously issued MMA of this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread t of the warp receives row (lane base + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// ---- CTA-pair (cta_group::2) forms: two CTAs of a cluster share one 256-row MMA
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory; the bytes are counted on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* tmap, uint32_t bar_cluster_addr,
                                                 int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far retire.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(mask)
               : "memory");
}

}  // namespace ptx

// ------------------------------------------------------------------ kernel configuration
constexpr int TC_BM = 128;
constexpr int TC_BK = 64;                   // one 128-byte swizzle row of bf16
constexpr int TC_THREADS = 320;             // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-9: epilogue
constexpr int TC_EPI_THREADS = 256;         // two warps per TMEM lane quarter, one per half of the tile's columns
constexpr long long TC_WAIT_LIMIT = 4000000000ll;   // ~2 s of SM clocks
constexpr int TC_BAND = 8;                  // row tiles per band of the tile order

enum { TC_EPI_ROTATE = 0, TC_EPI_ROTATE_Q = 1, TC_EPI_ACCUM = 2, TC_EPI_RESID = 3, TC_EPI_POLY = 4, TC_EPI_NEXT = 5,
       TC_EPI_PLAIN = 6 };

// PAIR: two CTAs of a cluster work on one 256 x 256 tile (each holds 128 rows of A and of the accumulator and
// 128 of the 256 columns of B in its own shared memory); otherwise one CTA works on a 128 x BN tile.
template <int BN, bool PAIR, int NA = 1, int NB = 1> struct TcCfg {
  static_assert(!PAIR || BN == 256, "a CTA pair always computes 256 x 256 tiles");
  static_assert(PAIR || (NA == 1 && NB == 1), "only the pair kernel keeps several operand tiles per stage");
  static constexpr int TILE_M = PAIR ? 256 : TC_BM;
  static constexpr int A_BYTES = TC_BM * TC_BK * 2;
  static constexpr int B_ROWS = PAIR ? 128 : BN;      // rows (n) of B this CTA loads per stage
  static constexpr int B_BYTES = B_ROWS * TC_BK * 2;
  // A pair's stage holds every distinct operand tile the passes of a split product need (e.g. A_hi, A_lo, B_hi, B_lo),
  // so the three passes hi hi + hi lo + lo hi cost four tile loads per k block instead of six.
  static constexpr int STAGE_BYTES = NA * A_BYTES + NB * B_BYTES;
  static constexpr int STAGES = PAIR ? (12 / (NA + NB)) : ((BN == 256) ? 4 : 6);
  static constexpr int TMEM_COLS = 2 * BN;          // two accumulators: the epilogue of tile i overlaps tile i+1
  static constexpr int AUX_BYTES = 1024;
  static constexpr int EPI_STAGE_BYTES = 8 * 4096;   // one 32 x 32 fp32 transposition buffer per epilogue warp
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + AUX_BYTES + EPI_STAGE_BYTES + 1024 /* alignment slack */;
};

struct TcGemmArgs {
  int M, N, K;                  // output rows, cols; contraction length of one segment
  int nseg;                     // k-loop passes: 1, or up to 3 for split-precision products
  int nseg_from_state;          // passes chosen on the device per step: 1 = st->seg_x, 2 = st->seg_e (else nseg)
  int a_off[3], b_off[3];       // outer-coordinate offset of each pass's operand inside a stacked [hi; lo] pair
  // the same passes as (distinct operand tiles, which tile each pass reads): filled by tc_fuse_passes for the pair kernel
  int na, nb;                   // distinct A / B tiles over all passes
  int a_toff[2], b_toff[2];     // their outer-coordinate offsets
  int a_tile[3], b_tile[3];     // tile index each pass reads (tiles appear in order of first use)
  int full_tiles;               // pair kernel: tiles [0, full_tiles) are worked on whole, the
                                //   remaining ones as two half-width items each (fills the last, partial wave)
  int sym;                      // 1: the output is symmetric (M == N): only tiles that touch the upper triangle are
                                //    computed; tiles strictly above the diagonal also write their transpose
  float* outF; long long ldo;   // fp32 output (M read-modify-write, E, X_next, Y)
  __nv_bfloat16* outH; long long ldh; long long lo_elems;   // bf16 output hi part (+ lo part at +lo_elems)
  const __nv_bfloat16* inH;                                 // bf16 pair epilogue input (the old iterate; same ld / lo_elems as outH)
  const float* rnorm;
  unsigned* rowmax; unsigned* rowmin;   // per-row ordered max / min of the raw products (quant modes)
  double* part_d; float* part_f;
  double* part_t;               // per-tile trace (residual) or sum of squares (next iterate)
  DevState* st;
  int check_done;
};

// Tiles (TM x BN) of a symmetric product, column by column: column tn holds the row tiles 0 .. (tn+1)*BN/TM - 1.
__host__ __device__ inline int tc_sym_tiles(int tiles_n, int r /* BN / TM */) { return r * tiles_n * (tiles_n + 1) / 2; }
template <int R>
__device__ __forceinline__ void tc_tile_coords(int t, int tiles_m, int tiles_n, int sym, int& tm, int& tn) {
  if (!sym) {
    // bands of TC_BAND row tiles, column by column inside a band: the tiles in flight at any time cover a roughly
    // square patch of the output, which keeps the operand blocks they share resident in L2
    const int per_band = TC_BAND * tiles_n;
    const int band = t / per_band, within = t - band * per_band;
    const int rows = min(TC_BAND, tiles_m - band * TC_BAND);
    tn = within / rows;
    tm = band * TC_BAND + (within - tn * rows);
    return;
  }
  int j = (int)((sqrtf(1.0f + 8.0f * (float)t / (float)R) - 1.0f) * 0.5f);
  while (R * (j + 1) * (j + 2) / 2 <= t) ++j;
  while (R * j * (j + 1) / 2 > t) --j;
  tn = j;
  tm = t - R * j * (j + 1) / 2;
}

struct TcAux {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint32_t tmem_base;
  int abort_flag;
  double red_d[8];
  float red_f[8];
  float red_t[8];
};

static_assert(sizeof(TcAux) <= 1024, "TcCfg::AUX_BYTES");

// Bounded wait.  Returns false when the wait was abandoned (timeout here, or another role aborted).
__device__ __forceinline__ bool tc_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                        long long limit = TC_WAIT_LIMIT) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) {
        *abort_flag = 1;
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // start address, leading / stride byte offsets (16-byte units), descriptor version 1, 128-byte swizzle
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ uint32_t bf16_bits(float v) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16(v)); }
__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16(v)); }
// Two floats -> packed bf16 pair (first in the low half) with one conversion instruction.
__device__ __forceinline__ uint32_t bf16x2_pack(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// Two-term split of a pair of floats: wh = packed round-to-nearest bf16, wl = packed bf16 of the remainders.
__device__ __forceinline__ void bf16x2_split(float a, float b, uint32_t& wh, uint32_t& wl) {
  wh = bf16x2_pack(a, b);
  wl = bf16x2_pack(a - __uint_as_float(wh << 16), b - __uint_as_float(wh & 0xffff0000u));
}

// Epilogue stores.  A thread holds 32 consecutive columns of ONE row (TMEM lane = row), so a direct 16-byte store
// per thread touches 32 different lines per instruction and only half a sector of each.  The warp's 32 x 32 block
// goes through a private, swizzled shared-memory buffer instead and leaves as full 128-byte (fp32) or 64-byte (bf16)
// row segments.  All 32 lanes must call these; rows >= rows_ok are not written.
__device__ __forceinline__ void tc_store_block_f32(uint8_t* stg, int lane, const float (&v)[32], float* out, long long ld,
                                                   int rows_ok) {
#pragma unroll
  for (int p = 0; p < 8; ++p)
    *reinterpret_cast<float4*>(stg + lane * 128 + ((p ^ (lane & 7)) << 4)) = make_float4(v[4 * p], v[4 * p + 1], v[4 * p + 2], v[4 * p + 3]);
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = i * 4 + (lane >> 3), c = lane & 7;
    const float4 t = *reinterpret_cast<const float4*>(stg + r * 128 + ((c ^ (r & 7)) << 4));
    if (r < rows_ok) __stcs(reinterpret_cast<float4*>(out + (long long)r * ld + c * 4), t);   // streaming: keep operand tiles in L2
  }
  __syncwarp();
}
// The same block added into `out` with vector reductions (fire-and-forget, performed at the L2).
__device__ __forceinline__ void tc_red_block_f32(uint8_t* stg, int lane, const float (&v)[32], float* out, long long ld,
                                                 int rows_ok) {
#pragma unroll
  for (int p = 0; p < 8; ++p)
    *reinterpret_cast<float4*>(stg + lane * 128 + ((p ^ (lane & 7)) << 4)) = make_float4(v[4 * p], v[4 * p + 1], v[4 * p + 2], v[4 * p + 3]);
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = i * 4 + (lane >> 3), c = lane & 7;
    const float4 t = *reinterpret_cast<const float4*>(stg + r * 128 + ((c ^ (r & 7)) << 4));
    if (r < rows_ok)
      asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(out + (long long)r * ld + c * 4), "f"(t.x), "f"(t.y),
                   "f"(t.z), "f"(t.w)
                   : "memory");
  }
  __syncwarp();
}
// 32 rows x 32 bf16 (w[16] = the thread's row as packed pairs) -> 64-byte row segments.
__device__ __forceinline__ void tc_store_block_bf16(uint8_t* stg, int lane, const uint32_t (&w)[16], __nv_bfloat16* out,
                                                    long long ld, int rows_ok) {
#pragma unroll
  for (int p = 0; p < 4; ++p)
    *reinterpret_cast<uint4*>(stg + lane * 64 + ((p ^ ((lane >> 1) & 3)) << 4)) = make_uint4(w[4 * p], w[4 * p + 1], w[4 * p + 2], w[4 * p + 3]);
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = i * 8 + (lane >> 2), c = lane & 3;
    const uint4 t = *reinterpret_cast<const uint4*>(stg + r * 64 + ((c ^ ((r >> 1) & 3)) << 4));
    if (r < rows_ok) __stcs(reinterpret_cast<uint4*>(out + (long long)r * ld + c * 8), t);
  }
  __syncwarp();
}

// Exercises the bounded wait on purpose: one thread waits on a barrier that nothing will ever arrive at, gives up after
// `limit_cycles`, and latches TIMEOUT exactly as the product kernels do.  The kernel then ends normally.
static __global__ void tc_wait_probe_kernel(DevState* st, long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0 && !tc_wait(&bar, 0u, &abort_flag, limit_cycles)) {
    atomicOr(&st->status_flags, STATUS_FLAG_TIMEOUT);
    st->timeout_site = 99;
  }
}

template <int BN, bool A_MN, bool B_MN, int EPI, bool PAIR, int NA = 1, int NB = 1>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TcGemmArgs g) {
  using Cfg = TcCfg<BN, PAIR, NA, NB>;
  constexpr int TM = Cfg::TILE_M;
  constexpr int R = BN / TM;                        // tiles per column step of a symmetric product
  if (g.check_done && g.st->ns_done) return;      // uniform over the grid: the iteration already finished

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  TcAux* aux = reinterpret_cast<TcAux*>(smem + Cfg::STAGES * Cfg::STAGE_BYTES);
  volatile int* abort_flag = &aux->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;        // 0: the CTA that issues the pair's MMAs
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int tiles_m = (g.M + TM - 1) / TM, tiles_n = (g.N + BN - 1) / BN;
  const int num_tiles = g.sym ? tc_sym_tiles(tiles_n, R) : tiles_m * tiles_n;
  // work items: whole tiles, then (pair kernel only) the tail tiles as two half-width items each
  const int full_tiles = (PAIR && B_MN) ? min(max(g.full_tiles, 0), num_tiles) : num_tiles;
  const int num_items = full_tiles + 2 * (num_tiles - full_tiles);
  auto decode_item = [&](int item, int& tm, int& tn, int& nt, int& ncol0) {
    int tile = item; nt = BN; ncol0 = 0;
    if (item >= full_tiles) { const int hh = item - full_tiles; tile = full_tiles + (hh >> 1); nt = BN / 2; ncol0 = (hh & 1) * (BN / 2); }
    tc_tile_coords<R>(tile, tiles_m, tiles_n, g.sym, tm, tn);
  };
  const int num_kb = (g.K + TC_BK - 1) / TC_BK;
  const int nseg = g.nseg_from_state ? max(1, min(g.nseg, g.nseg_from_state == 2 ? g.st->seg_e : g.st->seg_x)) : g.nseg;
  const int k_iters = PAIR ? num_kb : num_kb * nseg;     // a pair runs all passes of a k block from one stage

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::STAGES; ++s) { ptx::mbar_init(&aux->full[s], 1); ptx::mbar_init(&aux->empty[s], 1); }
    // the accumulator is handed back by every epilogue thread (of both CTAs of a pair)
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&aux->tfull[b], 1); ptx::mbar_init(&aux->tempty[b], PAIR ? 2 * TC_EPI_THREADS : TC_EPI_THREADS); }
    aux->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    if (PAIR) { ptx::tmem_alloc_pair(&aux->tmem_base, Cfg::TMEM_COLS); ptx::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(&aux->tmem_base, Cfg::TMEM_COLS); ptx::tmem_relinquish(); }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (PAIR) ptx::cluster_sync_all();                // the peer's barriers exist before anything is sent to them
  ptx::tc_fence_after();
  const uint32_t tmem_base = aux->tmem_base;
  int timeout_site = 0;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int tile = worker; tile < num_items && ok; tile += n_workers) {
        int tm, tn, nt, ncol0;
        decode_item(tile, tm, tn, nt, ncol0);
        // a pair splits the item: this CTA loads 128 of the 256 rows of A and half of the item's columns of B
        const int b_rows = PAIR ? nt / 2 : BN;
        const int m0 = tm * TM + (PAIR ? (int)rank * TC_BM : 0), n0 = tn * BN + ncol0 + (PAIR ? (int)rank * b_rows : 0);
        for (int it = 0; it < k_iters; ++it) {
          const int seg = it / num_kb, k0 = (it - seg * num_kb) * TC_BK;
          const int a_off = g.a_off[seg], b_off = g.b_off[seg];
          if (!tc_wait(&aux->empty[stage], phase ^ 1u, abort_flag)) { ok = false; timeout_site = 1; break; }
          uint8_t* sa = smem + stage * Cfg::STAGE_BYTES;
          uint8_t* sb = sa + Cfg::A_BYTES;
          if (PAIR) {
            // both CTAs' copies are counted on the barrier of CTA 0, whose MMA thread consumes the stage
            const uint32_t bar = ptx::mapa_u32(ptx::smem_u32(&aux->full[stage]), 0);
            int na = 1, nb = 1;                          // tiles the passes in use need
            for (int sg = 0; sg < nseg; ++sg) { na = max(na, g.a_tile[sg] + 1); nb = max(nb, g.b_tile[sg] + 1); }
            na = min(na, NA); nb = min(nb, NB);
            if (rank == 0) ptx::mbar_expect_tx(&aux->full[stage], 2 * (na * Cfg::A_BYTES + nb * b_rows * TC_BK * 2));
            const int kk = it * TC_BK;
#pragma unroll
            for (int ia = 0; ia < NA; ++ia) {
              if (ia >= na) break;
              uint8_t* ta = sa + ia * Cfg::A_BYTES;
              if (A_MN) {
#pragma unroll
                for (int h = 0; h < TC_BM / 64; ++h) ptx::tma_load_2d_pair(ta + h * 8192, &tmA, bar, m0 + 64 * h, kk + g.a_toff[ia]);
              } else {
                ptx::tma_load_2d_pair(ta, &tmA, bar, kk, m0 + g.a_toff[ia]);
              }
            }
#pragma unroll
            for (int ib = 0; ib < NB; ++ib) {
              if (ib >= nb) break;
              uint8_t* tb = sa + NA * Cfg::A_BYTES + ib * Cfg::B_BYTES;
              if (B_MN) {
#pragma unroll
                for (int h = 0; h < Cfg::B_ROWS / 64; ++h) {
                  if (h * 64 >= b_rows) break;
                  ptx::tma_load_2d_pair(tb + h * 8192, &tmB, bar, n0 + 64 * h, kk + g.b_toff[ib]);
                }
              } else {
                ptx::tma_load_2d_pair(tb, &tmB, bar, kk, n0 + g.b_toff[ib]);
              }
            }
          } else {
            ptx::mbar_expect_tx(&aux->full[stage], Cfg::STAGE_BYTES);
            if (A_MN) {
#pragma unroll
              for (int h = 0; h < TC_BM / 64; ++h)
                ptx::tma_load_2d(sa + h * 8192, &tmA, &aux->full[stage], m0 + 64 * h, k0 + a_off);
            } else {
              ptx::tma_load_2d(sa, &tmA, &aux->full[stage], k0, m0 + a_off);
            }
            if (B_MN) {
#pragma unroll
              for (int h = 0; h < BN / 64; ++h)
                ptx::tma_load_2d(sb + h * 8192, &tmB, &aux->full[stage], n0 + 64 * h, k0 + b_off);
            } else {
              ptx::tma_load_2d(sb, &tmB, &aux->full[stage], k0, n0 + b_off);
            }
          }
          ++issued;
          if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // drain: the copies already issued must have landed before the CTA may exit
        if (PAIR) {
          // their completion is counted in the other CTA: give them a fixed time (far beyond any copy latency)
          const long long t0 = clock64();
          while (clock64() - t0 < 4000000ll) {}
        } else {
          const int pending = issued < Cfg::STAGES ? issued : Cfg::STAGES;
          int s = stage;
          uint32_t ph = phase;
          for (int i = 0; i < pending; ++i) {
            if (--s < 0) { s = Cfg::STAGES - 1; ph ^= 1u; }
            const long long t0 = clock64();
            while (!ptx::mbar_try_wait(&aux->full[s], ph) && clock64() - t0 < TC_WAIT_LIMIT) {}
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (CTA 0 of a pair issues for both)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      const uint32_t idesc_half = (idesc & ~(0x3fu << 17)) | ((uint32_t)((BN / 2) >> 3) << 17);   // N = BN / 2
      for (int tile = worker; tile < num_items && ok; tile += n_workers, ++local) {
        const int buf = local & 1;
        const uint32_t idesc_t = (tile >= full_tiles) ? idesc_half : idesc;
        if (!tc_wait(&aux->tempty[buf], ((uint32_t)(local >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; timeout_site = 2; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int it = 0; it < k_iters; ++it) {
          if (!tc_wait(&aux->full[stage], phase, abort_flag)) { ok = false; timeout_site = 3; break; }
          ptx::tc_fence_after();
          const uint32_t sa = ptx::smem_u32(smem + stage * Cfg::STAGE_BYTES);
          // K-major: 16 k = 32 bytes inside the swizzled 128-byte row; 8-row groups 1024 bytes apart.
          // MN-major: 16 k = two 8-row groups of 1024 bytes; 64-wide m|n chunks 8192 bytes apart.
          // For a pair the descriptors name this CTA's tiles; the peer's halves sit at the same offsets in its memory.
          if (PAIR) {
            for (int sg = 0; sg < nseg; ++sg) {
              const uint32_t ta = sa + (uint32_t)(g.a_tile[sg] * Cfg::A_BYTES);
              const uint32_t tb = sa + (uint32_t)(NA * Cfg::A_BYTES + g.b_tile[sg] * Cfg::B_BYTES);
#pragma unroll
              for (int j = 0; j < TC_BK / 16; ++j) {
                const uint64_t ad = A_MN ? tc_smem_desc(ta + j * 2048, 8192, 1024) : tc_smem_desc(ta + j * 32, 16, 1024);
                const uint64_t bd = B_MN ? tc_smem_desc(tb + j * 2048, 8192, 1024) : tc_smem_desc(tb + j * 32, 16, 1024);
                ptx::umma_bf16_pair(d_tmem, ad, bd, idesc_t, (it > 0 || sg > 0 || j > 0) ? 1u : 0u);
              }
            }
          } else {
            const uint32_t sb = sa + Cfg::A_BYTES;
#pragma unroll
            for (int j = 0; j < TC_BK / 16; ++j) {
              const uint64_t ad = A_MN ? tc_smem_desc(sa + j * 2048, 8192, 1024) : tc_smem_desc(sa + j * 32, 16, 1024);
              const uint64_t bd = B_MN ? tc_smem_desc(sb + j * 2048, 8192, 1024) : tc_smem_desc(sb + j * 32, 16, 1024);
              ptx::umma_bf16(d_tmem, ad, bd, idesc, (it > 0 || j > 0) ? 1u : 0u);
            }
          }
          // frees the shared-memory stage (in both CTAs of a pair) once these MMAs retire
          if (PAIR) ptx::umma_commit_pair(&aux->empty[stage]); else ptx::umma_commit(&aux->empty[stage]);
          if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) {                                         // accumulator complete
          if (PAIR) ptx::umma_commit_pair(&aux->tfull[buf]); else ptx::umma_commit(&aux->tfull[buf]);
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue (8 warps: 128 TMEM lanes x 2 column halves)
    const int q = warp & 3;                               // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;                     // which half of the tile's columns this warp handles
    const int ew = warp - 2;                              // 0..7
    const int et = q * 32 + lane;                         // row inside the tile
    uint8_t* stg = smem + Cfg::STAGES * Cfg::STAGE_BYTES + Cfg::AUX_BYTES + ew * 4096;   // this warp's transposition buffer
    float c_gamma = 0.f, c_b1 = 0.f, c_b2 = 0.f, c_kappa = 0.f, c_tau = 1.f;
    if (EPI == TC_EPI_POLY || EPI == TC_EPI_NEXT) {
      c_gamma = g.st->coef[0]; c_b1 = g.st->coef[1]; c_b2 = g.st->coef[2]; c_kappa = g.st->coef[3];
    }
    if (EPI == TC_EPI_RESID) c_tau = g.st->tau;
    int local = 0;
    bool ok = true;
    const uint32_t tempty_addr0 = PAIR ? ptx::mapa_u32(ptx::smem_u32(&aux->tempty[0]), 0) : 0u;
    for (int tile = worker; tile < num_items && ok; tile += n_workers, ++local) {
      const int buf = local & 1;
      int tm, tn, nt, ncol0;
      decode_item(tile, tm, tn, nt, ncol0);
      const int m0 = tm * TM + (PAIR ? (int)rank * TC_BM : 0), n0 = tn * BN + ncol0;   // this CTA's 128 rows, all nt columns
      const bool mirror = g.sym && ((tm + 1) * TM <= tn * BN);        // strictly above the diagonal
      const int slot = PAIR ? 2 * tile + (int)rank : tile;            // where this CTA's per-tile partials go
      if (!tc_wait(&aux->tfull[buf], (uint32_t)(local >> 1) & 1u, abort_flag)) { ok = false; timeout_site = 4; break; }
      ptx::tc_fence_after();
      const int row = m0 + et;
      const bool row_ok = row < g.M;
      const uint32_t t_addr = tmem_base + (uint32_t)(buf * BN) + ((uint32_t)(q * 32) << 16);
      float rn = 0.f;
      uint32_t rn_bits = 0;
      if (EPI == TC_EPI_ROTATE || EPI == TC_EPI_ROTATE_Q) {
        rn = row_ok ? g.rnorm[row] : 0.f;
        rn_bits = bf16_bits(rn);
      }
      float acc_abs = 0.f, acc_max = 0.f, acc_tr = 0.f, acc_vmax = -3.0e38f, acc_vmin = 3.0e38f;
      double acc_sq = 0.0;
#pragma unroll 1
      for (int c = half * (nt / 64); c < (half + 1) * (nt / 64); ++c) {
        float v[32];
        ptx::tmem_ld32(t_addr + (uint32_t)(c * 32), v);
        const int col0 = n0 + c * 32;
        if (col0 >= g.N) continue;                         // N is a multiple of 32 in every use (uniform over the warp)
        const int wrow0 = m0 + q * 32;                     // first row of this warp's 32 x 32 block
        const int rows_ok = min(32, max(0, g.M - wrow0));  // rows of it inside the matrix
        if (rows_ok == 0) continue;
        if (!row_ok) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0.f;         // rows past the end take part in the stores with nothing to say
        }
        if (EPI == TC_EPI_ROTATE) {
          // C' = sgn(y) * rnorm as bf16 (sign bit or-ed in; exact zeros stay zero); objective partial sum |y|
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float a = v[2 * i], b = v[2 * i + 1];
            acc_abs += fabsf(a) + fabsf(b);
            const uint32_t lo = (a == 0.f) ? 0u : (rn_bits | ((__float_as_uint(a) >> 16) & 0x8000u));
            const uint32_t hi = (b == 0.f) ? 0u : (rn_bits | ((__float_as_uint(b) >> 16) & 0x8000u));
            w[i] = lo | (hi << 16);
          }
          tc_store_block_bf16(stg, lane, w, g.outH + (long long)wrow0 * g.ldh + col0, g.ldh, rows_ok);
        } else if (EPI == TC_EPI_ROTATE_Q) {
#pragma unroll
          for (int i = 0; i < 32; ++i) { acc_vmax = fmaxf(acc_vmax, v[i]); acc_vmin = fminf(acc_vmin, v[i]); }
          tc_store_block_f32(stg, lane, v, g.outF + (long long)wrow0 * g.ldo + col0, g.ldo, rows_ok);
        } else if (EPI == TC_EPI_ACCUM) {
          // M += acc as fire-and-forget vector reductions performed at the L2: the epilogue never waits for M to
          // arrive.  Each element of M receives exactly one addition per launch, so the result does not depend on
          // any ordering inside the launch.
          tc_red_block_f32(stg, lane, v, g.outF + (long long)wrow0 * g.ldo + col0, g.ldo, rows_ok);
        } else if (EPI == TC_EPI_PLAIN) {
          tc_store_block_f32(stg, lane, v, g.outF + (long long)wrow0 * g.ldo + col0, g.ldo, rows_ok);
        } else {
          // Newton-Schulz epilogues
          const int dcol = row - col0;                      // position of the diagonal inside this chunk, if any
          if (EPI == TC_EPI_RESID) {
            // statistics of G - I and of tr G; the stored residual is E = G - tau I
            float sq32 = 0.f;                              // 32 terms in fp32, then one double add per chunk
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              float e1 = v[i];
              if (i == dcol) { acc_tr += v[i]; e1 -= 1.f; v[i] -= c_tau; }
              acc_max = fmaxf(acc_max, fabsf(e1));
              sq32 = fmaf(e1, e1, sq32);
            }
            acc_sq += (double)sq32;
          } else {
            if (EPI == TC_EPI_POLY) {
              // beta1 E from the bf16 copy of E this product streams as its operands: the difference to fp32 E is a
              // symmetric relative perturbation of the size of B's own rounding to bf16
              const uint4* se = reinterpret_cast<const uint4*>(g.inH + (long long)(row_ok ? row : wrow0) * g.ldh + col0);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const uint4 e4 = se[i];
                const uint32_t ee[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  v[8 * i + 2 * e] = fmaf(c_b2, v[8 * i + 2 * e], c_b1 * __uint_as_float(ee[e] << 16));
                  v[8 * i + 2 * e + 1] = fmaf(c_b2, v[8 * i + 2 * e + 1], c_b1 * __uint_as_float(ee[e] & 0xffff0000u));
                }
              }
            } else {
              // the old iterate is its bf16 pair hi + lo (the same tiles this product streams as operand A)
              const long long at = (long long)(row_ok ? row : wrow0) * g.ldh + col0;
              const uint4* sh = reinterpret_cast<const uint4*>(g.inH + at);
              const uint4* sl = reinterpret_cast<const uint4*>(g.inH + g.lo_elems + at);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const uint4 h4 = sh[i], l4 = sl[i];
                const uint32_t hh[4] = {h4.x, h4.y, h4.z, h4.w}, ll[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float xa = __uint_as_float(hh[e] << 16) + __uint_as_float(ll[e] << 16);
                  const float xb = __uint_as_float(hh[e] & 0xffff0000u) + __uint_as_float(ll[e] & 0xffff0000u);
                  v[8 * i + 2 * e] = fmaf(c_gamma, xa, v[8 * i + 2 * e]);
                  v[8 * i + 2 * e + 1] = fmaf(c_gamma, xb, v[8 * i + 2 * e + 1]);
                }
              }
            }
            if (EPI == TC_EPI_POLY) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (i == dcol) v[i] -= c_kappa;
            } else {
              float sq32 = 0.f;
#pragma unroll
              for (int i = 0; i < 32; ++i) sq32 = fmaf(v[i], v[i], sq32);
              acc_sq += (double)sq32;
            }
          }
          uint32_t wh[16], wl[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            if (EPI == TC_EPI_NEXT) bf16x2_split(v[2 * i], v[2 * i + 1], wh[i], wl[i]);
            else wh[i] = bf16x2_pack(v[2 * i], v[2 * i + 1]);
          }
          tc_store_block_bf16(stg, lane, wh, g.outH + (long long)wrow0 * g.ldh + col0, g.ldh, rows_ok);
          if (EPI == TC_EPI_NEXT)
            tc_store_block_bf16(stg, lane, wl, g.outH + g.lo_elems + (long long)wrow0 * g.ldh + col0, g.ldh, rows_ok);
          if (EPI != TC_EPI_NEXT && mirror && row_ok) {
            // transpose of the tile: lane t holds row (m0 + 32 q + t), so for a fixed column the 32 lanes write
            // 32 consecutive elements of one output row
            unsigned short* oh = reinterpret_cast<unsigned short*>(g.outH);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const long long at = (long long)(col0 + i) * g.ldh + row;
              oh[at] = (unsigned short)((i & 1) ? (wh[i >> 1] >> 16) : (wh[i >> 1] & 0xffffu));
            }
          }
        }
      }
      // release the accumulator to the MMA thread before the (slower) reductions
      ptx::tc_fence_before();
      if (PAIR) ptx::mbar_arrive_cluster(tempty_addr0 + (uint32_t)(buf * sizeof(uint64_t)));
      else ptx::mbar_arrive(&aux->tempty[buf]);

      if (EPI == TC_EPI_ROTATE_Q) {
        if (row_ok && rn > 0.f) { atomicMax(g.rowmax + row, f2ord(acc_vmax)); atomicMin(g.rowmin + row, f2ord(acc_vmin)); }
      }
      if (EPI == TC_EPI_ROTATE || EPI == TC_EPI_RESID || EPI == TC_EPI_NEXT) {
        // per-tile partials, fixed reduction order; named barrier 1 synchronises the 8 epilogue warps only
        double dsum = (EPI == TC_EPI_ROTATE) ? (double)(acc_abs * rn) : acc_sq;
        dsum = warp_sum_d(dsum);
        float fmx = warp_max(acc_max);
        float ftr = warp_sum(acc_tr);
        if (lane == 0) { aux->red_d[ew] = dsum; aux->red_f[ew] = fmx; aux->red_t[ew] = ftr; }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (ew == 0 && lane == 0) {
          double tot = 0.0, ttr = 0.0;
          float tmx = 0.f;
#pragma unroll
          for (int i = 0; i < 8; ++i) { tot += aux->red_d[i]; ttr += (double)aux->red_t[i]; tmx = fmaxf(tmx, aux->red_f[i]); }
          if (EPI == TC_EPI_NEXT) {
            g.part_t[slot] = tot;
          } else {
            g.part_d[slot] = mirror ? 2.0 * tot : tot;       // a mirrored tile stands for two
          }
          if (EPI == TC_EPI_RESID) {
            g.part_f[slot] = tmx;
            g.part_t[slot] = ttr;
          }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
      }
    }
  }

  if (timeout_site != 0) {
    atomicOr(&g.st->status_flags, STATUS_FLAG_TIMEOUT);
    g.st->timeout_site = timeout_site;
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (PAIR) ptx::cluster_sync_all();                // neither CTA leaves while the other may still reach into it
  if (warp == 1) {
    ptx::tc_fence_after();
    if (PAIR) ptx::tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS); else ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

// ------------------------------------------------------------------ element-wise kernels of the mode

// a1 for the tensor-core mode: one warp per row.  rnorm_i = 1/||x_i||_2 (fp32, from the bf16-rounded values the
// MMA will see) and a bf16 copy of the row in the workspace; skipped rows are written as zeros so that they
// cannot reach the accumulators.
template <typename TIn>
__global__ void __launch_bounds__(256) rownorm_stage_kernel(const TIn* __restrict__ X, int64_t n, int d, int64_t ld,
                                                            float* __restrict__ rnorm,
                                                            __nv_bfloat16* __restrict__ Xs, DevState* st) {
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= n) return;
  const TIn* x = X + row * ld;
  __nv_bfloat16* dst = Xs + row * (int64_t)d;
  if (sizeof(TIn) == 2 && d <= 4096 && (d & 255) == 0 && (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
    // bf16 rows of up to 4096 elements: the whole row sits in the warp's registers (16-byte pieces, all loads in
    // flight at once), is read from memory once and written out from the registers
    const int nchunk = d >> 8;                          // 256 elements = 32 lanes x 16 bytes
    uint4 buf[16];
#pragma unroll
    for (int c = 0; c < 16; ++c)
      buf[c] = (c < nchunk) ? __ldg(reinterpret_cast<const uint4*>(x + c * 256 + lane * 8)) : make_uint4(0u, 0u, 0u, 0u);
    float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const uint32_t u[4] = {buf[c].x, buf[c].y, buf[c].z, buf[c].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a = __uint_as_float(u[e] << 16), b = __uint_as_float(u[e] & 0xffff0000u);
        s4[e] = fmaf(a, a, s4[e]); s4[e] = fmaf(b, b, s4[e]);
      }
    }
    const float ssr = warp_sum((s4[0] + s4[1]) + (s4[2] + s4[3]));
    const bool goodr = (ssr > 0.f) && (ssr <= 3.0e38f);
#pragma unroll
    for (int c = 0; c < 16; ++c)
      if (c < nchunk) *reinterpret_cast<uint4*>(dst + c * 256 + lane * 8) = goodr ? buf[c] : make_uint4(0u, 0u, 0u, 0u);
    if (lane == 0) {
      if (!goodr) {
        atomicAdd(reinterpret_cast<unsigned long long*>(&st->step_skipped), 1ull);
        if (!(ssr == 0.f)) atomicOr(&st->status_flags, STATUS_FLAG_NONFINITE);
      }
      rnorm[row] = goodr ? 1.0f / sqrtf(ssr) : 0.f;
    }
    return;
  }
  const bool vec = (reinterpret_cast<uintptr_t>(x) & (sizeof(TIn) * 4 - 1)) == 0;    // d is a multiple of 128
  float ss = 0.f;
  for (int k = lane * 4; k < d; k += 128) {
    float v[4];
    if (vec) {
      ld4_as_float(x + k, v);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = ld_as_float(x + k + j);
    }
    if (sizeof(TIn) == 4) {                            // fp32 input: the norm of what the MMA will see (bf16 values are exact already)
      const uint32_t p0 = bf16x2_pack(v[0], v[1]), p1 = bf16x2_pack(v[2], v[3]);
      v[0] = __uint_as_float(p0 << 16); v[1] = __uint_as_float(p0 & 0xffff0000u);
      v[2] = __uint_as_float(p1 << 16); v[3] = __uint_as_float(p1 & 0xffff0000u);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) ss = fmaf(v[j], v[j], ss);
  }
  ss = warp_sum(ss);
  const bool good = (ss > 0.f) && (ss <= 3.0e38f);
  for (int k = lane * 4; k < d; k += 128) {
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (good) {
      if (vec) {
        ld4_as_float(x + k, v);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = ld_as_float(x + k + j);
      }
    }
    uint2 o;
    o.x = bf16x2_pack(v[0], v[1]);
    o.y = bf16x2_pack(v[2], v[3]);
    *reinterpret_cast<uint2*>(dst + k) = o;
  }
  if (lane == 0) {
    if (!good) {
      atomicAdd(reinterpret_cast<unsigned long long*>(&st->step_skipped), 1ull);
      if (!(ss == 0.f)) atomicOr(&st->status_flags, STATUS_FLAG_NONFINITE);
    }
    rnorm[row] = good ? 1.0f / sqrtf(ss) : 0.f;
  }
}

// fp32 -> bf16 (hi only, lo_elems == 0) or the two-term split [hi; lo]
__global__ void split_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t count,
                                  int64_t lo_elems) {
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < count;
       i += (int64_t)gridDim.x * blockDim.x * 4) {
    const float4 t = *reinterpret_cast<const float4*>(src + i);
    uint2 o, l;
    bf16x2_split(t.x, t.y, o.x, l.x);
    bf16x2_split(t.z, t.w, o.y, l.y);
    *reinterpret_cast<uint2*>(dst + i) = o;
    if (lo_elems) *reinterpret_cast<uint2*>(dst + lo_elems + i) = l;
  }
}

// Second pass of the two-pass step in tensor-core mode (quant modes, or diagnostics): Y (fp32, row-major) ->
// C' (bf16, row-major) + objective partials (+ diagnostics partials).
__global__ void __launch_bounds__(256) quant_target_bf16_kernel(const float* __restrict__ Y, int64_t n, int d,
                                                                const float* __restrict__ rnorm,
                                                                const unsigned int* __restrict__ rowmax_ord,
                                                                const unsigned int* __restrict__ rowmin_ord,
                                                                QuantSpec qs, double* __restrict__ partials,
                                                                __nv_bfloat16* __restrict__ Cp, double* __restrict__ part_diag) {
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const bool diag = part_diag != nullptr;
  double contrib = 0.0, dterm[4] = {0.0, 0.0, 0.0, 0.0};
  if (row < n) {
    const float r = rnorm[row];
    RowQuant rq{0.f, 1.f, 0.f, 0.f};
    if (qs.bits) rq = row_quant(qs, ord2f(rowmax_ord[row]), ord2f(rowmin_ord[row]), r > 0.f);
    const bool live = qs.bits ? (rq.inv > 0.f) : (r > 0.f);
    const float* y = Y + row * (int64_t)d;
    __nv_bfloat16* c = Cp + row * (int64_t)d;
    float qsum = 0.f;
    RowDiag dg{0.f, 0.f, 0.f, 0.f};
    for (int j0 = lane * 4; j0 < d; j0 += 1024) {              // eight 16-byte loads in flight per lane (Y is read once)
      float4 t8[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = j0 + 128 * u;
        t8[u] = (j < d) ? __ldcs(reinterpret_cast<const float4*>(y + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = j0 + 128 * u;
        if (j >= d) break;
        const float in[4] = {t8[u].x, t8[u].y, t8[u].z, t8[u].w};
        float sg[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) sg[e] = live ? second_pass_elem(in[e], r, qs, rq, qsum, diag, dg) * r : 0.f;
        uint2 o;
        o.x = bf16x2_pack(sg[0], sg[1]);
        o.y = bf16x2_pack(sg[2], sg[3]);
        *reinterpret_cast<uint2*>(c + j) = o;
      }
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
    if (threadIdx.x == 0) partials[blockIdx.x] = t;
    else if (diag) part_diag[(int64_t)(threadIdx.x - 1) * gridDim.x + blockIdx.x] = t;
  }
}

// ------------------------------------------------------------------ host side
struct TcLayout {
  size_t Xs, Cp, Rb, Xh[2], Eh, Bh;
};

struct TcHost {
  int d, P, quant_bits, num_sms;
  int device;                                // CUDA device the context was created on
  int pair_clusters;                         // CTA pairs that can be co-resident (0: single-CTA kernels only)
  float e1_tau;                              // residual product runs one pass while mean sigma^2 of the iterate is below this
  float lo_budget;                           // ... and in mid-iteration, see ns_tau_kernel
  int64_t n_max;
  char* ws;
  TcLayout L;
  float *R, *M, *Xa, *Xb, *E, *B, *rnorm, *Y;
  unsigned* rowmax;
  QuantSpec qs;
  int diagnostics;                           // 1: every step takes the two-pass route and gathers the Section-4 diagnostics
  double* part_diag;
  DevState* st;
  double* part_d;
  float* part_f;
  // static tensor maps (d x d operands)
  CUtensorMap tmRb_mn;                       // R bf16 as MN-major B of the rotate product
  CUtensorMap tmM_blk, tmMpart_blk;          // per-head case: fp32 M of all problems / the partials, 32 x 32 boxes
  CUtensorMap tmXh_mn[2], tmXh_k[2];         // iterate, stacked [hi; lo]
  CUtensorMap tmEh_k, tmEh_mn, tmBh_mn;
  Prof* prof;
  int ns_k;                                  // Newton-Schulz step index of the launches being enqueued (-1 outside)
};

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline PFN_encodeTiled tc_encode_fn() {
  static PFN_encodeTiled fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_encodeTiled>(p);
  }
  return fn;
}

// 2-D bf16 row-major tensor (rows x cols, row stride ld elements); box = box_rows x 64 columns, 128-byte swizzle,
// out-of-range elements read as zero.
inline int tc_make_tmap(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
  PFN_encodeTiled fn = tc_encode_fn();
  if (!fn) return CONQUR_ERR_CUDA;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::fprintf(stderr, "conqur: cuTensorMapEncodeTiled failed (%d)\n", (int)r);
    return CONQUR_ERR_CUDA;
  }
  return CONQUR_OK;
}

// 2-D fp32 row-major tensor of 128 columns (rows x 128, contiguous rows); box = 32 rows x 32 columns, 128-byte swizzle.
inline int tc_make_tmap_f32_blocks(CUtensorMap* tm, const void* ptr, uint64_t rows) {
  PFN_encodeTiled fn = tc_encode_fn();
  if (!fn) return CONQUR_ERR_CUDA;
  const cuuint64_t dims[2] = {128, rows};
  const cuuint64_t strides[1] = {128 * 4};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::fprintf(stderr, "conqur: cuTensorMapEncodeTiled (fp32 blocks) failed (%d)\n", (int)r);
    return CONQUR_ERR_CUDA;
  }
  return CONQUR_OK;
}

// one problem of any d that is a multiple of 128, or many problems of d = 128 (the per-head case)
inline bool tc_supported_shape(int d, int batch) { return d >= 128 && (d % 128) == 0 && (batch == 1 || d == 128); }

template <typename Take>
inline void tc_make_layout(int d, int P, int64_t n_max, int quant_bits, int in_dtype, TcLayout* L, Take&& take) {
  (void)quant_bits;
  const size_t dd = (size_t)d * d;
  *L = TcLayout{};
  if (P > 1) {
    // batched (d = 128): the fused kernel keeps everything else on chip
    if (in_dtype == CONQUR_F32) L->Xs = take(2 * (size_t)n_max * d * P);
    L->Rb = take(2 * dd * P);
    return;
  }
  L->Xs = take(2 * (size_t)n_max * d);
  L->Cp = take(2 * (size_t)n_max * d);
  L->Rb = take(2 * dd);
  L->Xh[0] = take(4 * dd);
  L->Xh[1] = take(4 * dd);
  L->Eh = take(2 * dd);
  L->Bh = take(2 * dd);
}

inline int tc_epi_class(int epi) {
  switch (epi) {
    case TC_EPI_ROTATE: case TC_EPI_ROTATE_Q: return K_ROTATE;
    case TC_EPI_ACCUM: return K_ACCUM;
    case TC_EPI_RESID: return K_NS_RESID;
    case TC_EPI_POLY: return K_NS_POLY;
    case TC_EPI_NEXT: return K_NS_NEXT;
    default: return K_OTHER;
  }
}

// Which kernel variant a product of output width N runs with.
//   pair : CTA pairs on 256 x 256 tiles (needs N % 256 == 0 and a device that can co-schedule the pairs)
//   else : single CTAs on 128 x 256 (N % 256 == 0) or 128 x 128 tiles
struct TcVariant { bool pair; int tile_m, tile_n; };
inline TcVariant tc_variant(const TcHost& h, int N) {
  if (N % 256 == 0) return h.pair_clusters > 0 ? TcVariant{true, 256, 256} : TcVariant{false, 128, 256};
  return TcVariant{false, 128, 128};
}
// tiles the kernel computes
inline int tc_tiles(const TcVariant& v, int M, int N, int sym) {
  const int tn = (N + v.tile_n - 1) / v.tile_n, tm = (M + v.tile_m - 1) / v.tile_m;
  return sym ? tc_sym_tiles(tn, v.tile_n / v.tile_m) : tm * tn;
}
// Work items of a launch (B operand MN-major): the pair kernel works on the tiles of its last, partial wave as two
// half-width items each when that lets them all run at once (e.g. 256 tiles on 74 pairs: 3 waves + 34 tiles ->
// 3 waves + 68 half tiles, i.e. 3.5 instead of 4 tile times).  *full_tiles: tiles worked on whole.
inline int tc_items(const TcHost& h, const TcVariant& v, int M, int N, int sym, int* full_tiles = nullptr) {
  const int tiles = tc_tiles(v, M, N, sym);
  int full = tiles;
  if (v.pair && h.pair_clusters > 0) {
    const int r = tiles % h.pair_clusters;
    if (r > 0 && 2 * r <= h.pair_clusters) full = tiles - r;
  }
  if (full_tiles) *full_tiles = full;
  return full + 2 * (tiles - full);
}
// per-item partial slots a launch writes (a pair writes one per CTA)
inline int tc_part_slots(const TcHost& h, const TcVariant& v, int M, int N, int sym) {
  return tc_items(h, v, M, N, sym) * (v.pair ? 2 : 1);
}

// Rewrite the passes (a_off[s], b_off[s]) as distinct operand tiles + which tile each pass reads.
inline void tc_fuse_passes(TcGemmArgs* g) {
  g->na = g->nb = 0;
  for (int s = 0; s < g->nseg && s < 3; ++s) {
    int ia = -1, ib = -1;
    for (int i = 0; i < g->na; ++i) if (g->a_toff[i] == g->a_off[s]) ia = i;
    for (int i = 0; i < g->nb; ++i) if (g->b_toff[i] == g->b_off[s]) ib = i;
    if (ia < 0 && g->na < 2) { ia = g->na; g->a_toff[g->na++] = g->a_off[s]; }
    if (ib < 0 && g->nb < 2) { ib = g->nb; g->b_toff[g->nb++] = g->b_off[s]; }
    g->a_tile[s] = ia < 0 ? 0 : ia;
    g->b_tile[s] = ib < 0 ? 0 : ib;
  }
}

template <int BN, bool A_MN, bool B_MN, int EPI, bool PAIR, int NA = 1, int NB = 1>
inline int tc_launch(TcHost& h, cudaStream_t s, const CUtensorMap& a, const CUtensorMap& b, const TcGemmArgs& g) {
  using Cfg = TcCfg<BN, PAIR, NA, NB>;
  auto kern = tc_gemm_kernel<BN, A_MN, B_MN, EPI, PAIR, NA, NB>;
  // the attribute is per device; setting it twice from two threads is harmless, so an atomic mask is enough
  static std::atomic<unsigned long long> attr_dev_mask{0};
  const unsigned long long dev_bit = 1ull << (h.device & 63);
  if (!(attr_dev_mask.load(std::memory_order_acquire) & dev_bit)) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES) != cudaSuccess)
      return CONQUR_ERR_CUDA;
    attr_dev_mask.fetch_or(dev_bit, std::memory_order_release);
  }
  const TcVariant v{PAIR, Cfg::TILE_M, BN};
  const int tiles = tc_tiles(v, g.M, g.N, g.sym);
  TcGemmArgs gl = g;
  gl.full_tiles = tiles;
  const int items = B_MN ? tc_items(h, v, g.M, g.N, g.sym, &gl.full_tiles) : tiles;
  const int workers = PAIR ? h.pair_clusters : h.num_sms;
  const int grid = (items < workers ? items : workers) * (PAIR ? 2 : 1);
  const int cls = tc_epi_class(EPI);
  Prof::Rec rec{};
  const bool timed = h.prof && h.prof->enabled;
  if (timed) {
    // flops the tensor cores execute: computed tiles only, one pass (scaled by the passes taken when folded)
    rec.cls = cls; rec.flops = 2.0 * (double)tiles * Cfg::TILE_M * BN * (double)g.K; rec.ns_k = h.ns_k;
    rec.nseg = g.nseg_from_state == 1 ? 0 : (g.nseg_from_state == 2 ? -1 : g.nseg);
    rec.e0 = h.prof->get_event(); rec.e1 = h.prof->get_event();
    cudaEventRecord(rec.e0, s);
  }
  cudaError_t err;
  if (PAIR) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = Cfg::SMEM_BYTES; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    err = cudaLaunchKernelEx(&cfg, kern, a, b, gl);
  } else {
    kern<<<grid, TC_THREADS, Cfg::SMEM_BYTES, s>>>(a, b, gl);
    err = cudaGetLastError();
  }
  if (timed) { cudaEventRecord(rec.e1, s); h.prof->open.push_back(rec); }
  if (h.prof) h.prof->count(cls);
  return err == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}

// dispatch on the kernel variant (see tc_variant)
template <bool A_MN, bool B_MN, int EPI>
inline int tc_launch_n(TcHost& h, cudaStream_t s, const CUtensorMap& a, const CUtensorMap& b, const TcGemmArgs& g) {
  const TcVariant v = tc_variant(h, g.N);
  if (v.pair) {
    TcGemmArgs gg = g;
    tc_fuse_passes(&gg);
    if constexpr (EPI == TC_EPI_RESID || EPI == TC_EPI_PLAIN) {
      if (gg.na + gg.nb > 2) return tc_launch<256, A_MN, B_MN, EPI, true, 2, 2>(h, s, a, b, gg);
    }
    if constexpr (EPI == TC_EPI_NEXT) return tc_launch<256, A_MN, B_MN, EPI, true, 2, 1>(h, s, a, b, gg);
    return tc_launch<256, A_MN, B_MN, EPI, true>(h, s, a, b, gg);
  }
  if (v.tile_n == 256) return tc_launch<256, A_MN, B_MN, EPI, false>(h, s, a, b, g);
  return tc_launch<128, A_MN, B_MN, EPI, false>(h, s, a, b, g);
}

// How many CTA pairs of the 256 x 256 kernel can be resident at once on the current device (0: use single CTAs).
inline int tc_query_pair_clusters() {
  using Cfg = TcCfg<256, true>;
  auto kern = tc_gemm_kernel<256, false, true, TC_EPI_PLAIN, true>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES) != cudaSuccess) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * 1024); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
  return n > 0 ? n : 0;
}

// Facts about a device, looked up once per device under a lock (the queries cost milliseconds).
struct TcDevFacts { int known, major, sms, pair_clusters; };
inline int tc_device_facts(int dev, TcDevFacts* out) {
  static std::mutex mu;
  static TcDevFacts facts[64] = {};
  if (dev < 0 || dev >= 64) return CONQUR_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  TcDevFacts& f = facts[dev];
  if (!f.known) {
    if (cudaDeviceGetAttribute(&f.major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&f.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return CONQUR_ERR_CUDA;
    f.pair_clusters = f.major == 10 ? tc_query_pair_clusters() : 0;
    f.known = 1;
  }
  *out = f;
  return CONQUR_OK;
}

inline int tc_init(TcHost* h, char* ws, const TcLayout& L, int d, int P, int64_t n_max, int quant_bits, float* R,
                   float* M, float* Xa, float* Xb, float* E, float* B, float* rnorm, DevState* st, double* part_d,
                   float* part_f, float* Y, unsigned* rowmax, QuantSpec qs, int diagnostics, double* part_diag, Prof* prof,
                   int single_cta, float gram_single_pass_tau, float lo_budget) {
  h->d = d; h->P = P; h->n_max = n_max; h->quant_bits = quant_bits; h->ws = ws; h->L = L;
  h->R = R; h->M = M; h->Xa = Xa; h->Xb = Xb; h->E = E; h->B = B; h->rnorm = rnorm; h->st = st;
  h->part_d = part_d; h->part_f = part_f; h->Y = Y; h->rowmax = rowmax; h->qs = qs; h->diagnostics = diagnostics; h->part_diag = part_diag; h->prof = prof; h->ns_k = -1;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return CONQUR_ERR_CUDA;
  TcDevFacts f;
  if (tc_device_facts(dev, &f) != CONQUR_OK) return CONQUR_ERR_CUDA;
  if (f.major != 10) {
    std::fprintf(stderr, "conqur: the tensor-core mode needs an sm_100 device (found compute capability %d.x)\n", f.major);
    return CONQUR_ERR_UNSUPPORTED;
  }
  h->num_sms = f.sms;
  h->device = dev;
  h->pair_clusters = single_cta ? 0 : f.pair_clusters;
  h->e1_tau = gram_single_pass_tau > 0.f ? gram_single_pass_tau : 2e-3f;
  h->lo_budget = lo_budget;
  const uint64_t D = (uint64_t)d;
  int rc = 0;
  if (P > 1) {
    // all rotations stacked: problem p's R is rows [128 p, 128 p + 128); one box = 64 columns x all 128 rows
    rc |= tc_make_tmap(&h->tmRb_mn, ws + L.Rb, (uint64_t)P * D, D, D, 128);
    // destinations of the per-head write-out: all cross-covariances stacked, and the partials of split problems
    // (the idle Newton-Schulz buffers: 4 P matrices of 128 x 128 starting at Xa)
    rc |= tc_make_tmap_f32_blocks(&h->tmM_blk, M, (uint64_t)P * D);
    rc |= tc_make_tmap_f32_blocks(&h->tmMpart_blk, Xa, 4ull * (uint64_t)P * D);
    return rc ? CONQUR_ERR_CUDA : CONQUR_OK;
  }
  rc |= tc_make_tmap(&h->tmRb_mn, ws + L.Rb, D, D, D, 64);
  for (int i = 0; i < 2; ++i) {
    rc |= tc_make_tmap(&h->tmXh_mn[i], ws + L.Xh[i], 2 * D, D, D, 64);
    rc |= tc_make_tmap(&h->tmXh_k[i], ws + L.Xh[i], 2 * D, D, D, 128);
  }
  rc |= tc_make_tmap(&h->tmEh_k, ws + L.Eh, D, D, D, 128);
  rc |= tc_make_tmap(&h->tmEh_mn, ws + L.Eh, D, D, D, 64);
  rc |= tc_make_tmap(&h->tmBh_mn, ws + L.Bh, D, D, D, 64);
  return rc ? CONQUR_ERR_CUDA : CONQUR_OK;
}

inline int tc_ew_blocks(int64_t count4) {
  const int64_t b = (count4 + 255) / 256;
  return (int)(b < 148 * 8 ? b : 148 * 8);
}

inline int tc_refresh_R(TcHost& h, cudaStream_t s, int) {
  const int64_t dd = (int64_t)h.d * h.d * h.P;
  split_bf16_kernel<<<tc_ew_blocks(dd / 4), 256, 0, s>>>(h.R, reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Rb), dd, 0);
  if (h.prof) h.prof->count(K_OTHER);
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}

inline TcGemmArgs tc_args(const TcHost& h, int M, int N, int K) {
  TcGemmArgs g{};
  g.M = M; g.N = N; g.K = K; g.nseg = 1; g.st = h.st; g.part_d = h.part_d; g.part_f = h.part_f;
  return g;
}

// a1 of one streamed batch: row norms and the sanitised bf16 copy, written at rows [row0, row0 + n) of the per-step
// buffers (row0 > 0 only in a context that queues several batches before running the products).
inline int tc_stage(TcHost& h, cudaStream_t s, const void* X, int in_dtype, int64_t n, int64_t ld, int64_t row0) {
  const int d = h.d;
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Xs) + row0 * d;
  const int rb = (int)((n + 7) / 8);
  if (in_dtype == CONQUR_F32)
    rownorm_stage_kernel<float><<<rb, 256, 0, s>>>(static_cast<const float*>(X), n, d, ld, h.rnorm + row0, Xs, h.st);
  else
    rownorm_stage_kernel<__nv_bfloat16><<<rb, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(X), n, d, ld, h.rnorm + row0, Xs, h.st);
  if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
  if (h.prof) h.prof->count(K_ROWNORM);
  return CONQUR_OK;
}

// a2-a5 over the first n staged rows: rotate + target (+ the second pass of the fake-quant / diagnostics route),
// objective, accumulate.
inline int tc_process(TcHost& h, cudaStream_t s, int64_t n) {
  const int d = h.d;
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Xs);
  __nv_bfloat16* Cp = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Cp);
  const int rb = (int)((n + 7) / 8);
  // per-call maps over the first n rows: rows past n read as zeros
  CUtensorMap tmXs_k, tmXs_mn, tmCp_mn;
  int rc = tc_make_tmap(&tmXs_k, Xs, (uint64_t)n, (uint64_t)d, (uint64_t)d, 128);
  rc |= tc_make_tmap(&tmXs_mn, Xs, (uint64_t)n, (uint64_t)d, (uint64_t)d, 64);
  rc |= tc_make_tmap(&tmCp_mn, Cp, (uint64_t)n, (uint64_t)d, (uint64_t)d, 64);
  if (rc) return CONQUR_ERR_CUDA;
  const double isd = 1.0 / std::sqrt((double)d);
  TcGemmArgs g = tc_args(h, (int)n, d, d);
  g.rnorm = h.rnorm;
  int per_problem;
  if (h.quant_bits == 0 && !h.diagnostics) {
    g.outH = Cp; g.ldh = d;
    rc = tc_launch_n<false, true, TC_EPI_ROTATE>(h, s, tmXs_k, h.tmRb_mn, g);
    if (rc) return rc;
    per_problem = tc_part_slots(h, tc_variant(h, d), (int)n, d, 0);
  } else {
    unsigned* rowmin = h.rowmax + h.n_max;
    if (cudaMemsetAsync(h.rowmax, 0, sizeof(unsigned) * n, s) != cudaSuccess) return CONQUR_ERR_CUDA;
    if (cudaMemsetAsync(rowmin, 0xff, sizeof(unsigned) * n, s) != cudaSuccess) return CONQUR_ERR_CUDA;
    g.outF = h.Y; g.ldo = d; g.rowmax = h.rowmax; g.rowmin = rowmin;
    rc = tc_launch_n<false, true, TC_EPI_ROTATE_Q>(h, s, tmXs_k, h.tmRb_mn, g);
    if (rc) return rc;
    quant_target_bf16_kernel<<<rb, 256, 0, s>>>(h.Y, n, d, h.rnorm, h.rowmax, rowmin, h.qs, h.part_d, Cp,
                                                h.diagnostics ? h.part_diag : nullptr);
    if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
    if (h.prof) h.prof->count(K_OTHER);
    per_problem = rb;
  }
  finalize_step_kernel<<<1, 256, 0, s>>>(h.st, h.part_d, per_problem, n, isd, h.diagnostics ? h.part_diag : nullptr, rb);
  if (cudaGetLastError() != cudaSuccess) return CONQUR_ERR_CUDA;
  if (h.prof) h.prof->count(K_OTHER);
  TcGemmArgs a = tc_args(h, d, d, (int)n);
  a.outF = h.M; a.ldo = d;
  return tc_launch_n<true, true, TC_EPI_ACCUM>(h, s, tmXs_mn, tmCp_mn, a);
}

// X0 = (M_raw + lam R) * x0_scale, written straight as the stacked bf16 split [hi; lo] (no fp32 copy of X0)
static __global__ void tc_x0_split_kernel(const float* __restrict__ M, const float* __restrict__ R,
                                          __nv_bfloat16* __restrict__ dst, int64_t dd, const DevState* st) {
  const float lam = st->lam, sc = st->x0_scale;
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < dd; i += (int64_t)gridDim.x * blockDim.x * 4) {
    const float4 m = *reinterpret_cast<const float4*>(M + i), r = *reinterpret_cast<const float4*>(R + i);
    uint2 o, l;
    bf16x2_split(fmaf(lam, r.x, m.x) * sc, fmaf(lam, r.y, m.y) * sc, o.x, l.x);
    bf16x2_split(fmaf(lam, r.z, m.z) * sc, fmaf(lam, r.w, m.w) * sc, o.y, l.y);
    *reinterpret_cast<uint2*>(dst + i) = o;
    *reinterpret_cast<uint2*>(dst + dd + i) = l;
  }
}
inline int tc_ns_begin(TcHost& h, cudaStream_t s) {
  const int64_t dd = (int64_t)h.d * h.d;
  tc_x0_split_kernel<<<tc_ew_blocks(dd / 4), 256, 0, s>>>(h.M, h.R, reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Xh[0]), dd, h.st);
  if (h.prof) h.prof->count(K_OTHER);
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}


// Partials of the Newton-Schulz epilogues: [0, parts) sums of squares, [parts, 2 parts) traces / iterate norms.
inline int tc_ns_parts(const TcHost& h) { return tc_part_slots(h, tc_variant(h, h.d), h.d, h.d, 1); }
inline int tc_ns_next_parts(const TcHost& h) { return tc_part_slots(h, tc_variant(h, h.d), h.d, h.d, 0); }

// G = X^T X from the split iterate in Xh[buf] (three passes: hi hi, hi lo, lo hi; symmetric tiles only);
// stores E = G - tau I as fp32 and bf16, and the statistics of G - I.
inline int tc_ns_residual(TcHost& h, cudaStream_t s, int buf) {
  const int d = h.d;
  TcGemmArgs g = tc_args(h, d, d, d);
  g.nseg = 3; g.nseg_from_state = 2; g.a_off[2] = d; g.b_off[1] = d; g.check_done = 1; g.sym = 1;
  g.outH = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Eh); g.ldh = d;
  g.part_t = h.part_d + tc_ns_parts(h);
  return tc_launch_n<true, true, TC_EPI_RESID>(h, s, h.tmXh_mn[buf], h.tmXh_mn[buf], g);
}

// B = beta2 E E + beta1 E - kappa I (one bf16 pass, symmetric tiles only) ;  X_next = X B + (gamma + kappa) X
// (the iterate enters as hi, or hi + lo while small singular values are still being lifted).
inline int tc_ns_poly_next(TcHost& h, cudaStream_t s, int cur) {
  const int d = h.d;
  const long long dd = (long long)d * d;
  TcGemmArgs g = tc_args(h, d, d, d);
  g.nseg = 1; g.check_done = 1; g.sym = 1;
  g.inH = reinterpret_cast<const __nv_bfloat16*>(h.ws + h.L.Eh);
  g.outH = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Bh); g.ldh = d;
  int rc = tc_launch_n<false, true, TC_EPI_POLY>(h, s, h.tmEh_k, h.tmEh_mn, g);
  if (rc) return rc;
  TcGemmArgs x = tc_args(h, d, d, d);
  x.nseg = 2; x.nseg_from_state = 1; x.a_off[1] = d; x.check_done = 1;
  x.inH = reinterpret_cast<const __nv_bfloat16*>(h.ws + h.L.Xh[cur]);
  x.outH = reinterpret_cast<__nv_bfloat16*>(h.ws + h.L.Xh[1 - cur]); x.ldh = d; x.lo_elems = dd;
  x.part_t = h.part_d + tc_ns_parts(h);
  rc = tc_launch_n<false, true, TC_EPI_NEXT>(h, s, h.tmXh_k[cur], h.tmBh_mn, x);
  if (rc) return rc;
  ns_tau_kernel<<<1, 256, 0, s>>>(h.st, h.part_d + tc_ns_parts(h), tc_ns_next_parts(h), d, h.e1_tau, h.lo_budget);
  if (h.prof) h.prof->count(K_OTHER);
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}

// Accept the update in tensor-core mode: R <- hi + lo of the final iterate, M <- 0.
static __global__ void tc_commit_kernel(DevState* st, const __nv_bfloat16* __restrict__ X0, const __nv_bfloat16* __restrict__ X1,
                                        float* __restrict__ R, float* __restrict__ M, int64_t dd) {
  if (st->ns_done != NS_DONE_CONVERGED) return;
  const __nv_bfloat16* X = st->ns_final_buf ? X1 : X0;
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 2; i < dd; i += (int64_t)gridDim.x * blockDim.x * 2) {
    const uint32_t hb = *reinterpret_cast<const uint32_t*>(X + i), lb = *reinterpret_cast<const uint32_t*>(X + dd + i);
    float2 o;
    o.x = __uint_as_float(hb << 16) + __uint_as_float(lb << 16);
    o.y = __uint_as_float(hb & 0xffff0000u) + __uint_as_float(lb & 0xffff0000u);
    *reinterpret_cast<float2*>(R + i) = o;
    *reinterpret_cast<float2*>(M + i) = make_float2(0.f, 0.f);
  }
}
inline int tc_ns_commit(TcHost& h, cudaStream_t s) {
  const int64_t dd = (int64_t)h.d * h.d;
  tc_commit_kernel<<<tc_ew_blocks(dd / 2), 256, 0, s>>>(h.st, reinterpret_cast<const __nv_bfloat16*>(h.ws + h.L.Xh[0]),
                                                       reinterpret_cast<const __nv_bfloat16*>(h.ws + h.L.Xh[1]), h.R, h.M, dd);
  if (h.prof) h.prof->count(K_OTHER);
  return cudaGetLastError() == cudaSuccess ? CONQUR_OK : CONQUR_ERR_CUDA;
}

inline const __nv_bfloat16* tc_cp_ptr(const TcHost& h) { return reinterpret_cast<const __nv_bfloat16*>(h.ws + h.L.Cp); }

// Stand-alone product (tests, weight folding): D (fp32, M x N, row stride ldo; 0 = N) = A * B^T-style contraction with
// the given orientations.  a_mn / b_mn: 0 = K-major ([M|N rows][K cols]), 1 = MN-major ([K rows][M|N cols]).  split:
// operands are stacked [hi; lo] pairs (3 products).  All device pointers; bf16 operands; shapes as checked below.
inline int tc_plain_gemm(const __nv_bfloat16* A, const __nv_bfloat16* B, float* D, int M, int N, int K, int a_mn,
                         int b_mn, int split, DevState* st, cudaStream_t s, long long ldo = 0) {
  if (M < 1 || N < 32 || (N % 32) || K < 1 || (K % 8) || (M % 8)) return CONQUR_ERR_INVALID_ARG;
  if (ldo == 0) ldo = N;
  if (ldo < N || (ldo % 4)) return CONQUR_ERR_INVALID_ARG;
  TcHost h{};
  h.prof = nullptr; h.ns_k = -1;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return CONQUR_ERR_CUDA;
  TcDevFacts f;
  if (tc_device_facts(dev, &f) != CONQUR_OK) return CONQUR_ERR_CUDA;
  if (f.major != 10) return CONQUR_ERR_UNSUPPORTED;
  h.num_sms = f.sms;
  h.device = dev;
  h.pair_clusters = f.pair_clusters;
  const uint64_t mul = split ? 2 : 1;
  CUtensorMap ta, tb;
  int rc;
  if (a_mn) rc = tc_make_tmap(&ta, A, mul * K, M, M, 64); else rc = tc_make_tmap(&ta, A, mul * M, K, K, 128);
  if (rc) return rc;
  const TcVariant v = tc_variant(h, N);
  const uint32_t bn = v.pair ? 128 : (uint32_t)v.tile_n;      // rows of B one CTA loads per stage
  if (b_mn) rc = tc_make_tmap(&tb, B, mul * K, N, N, 64); else rc = tc_make_tmap(&tb, B, mul * N, K, K, bn);
  if (rc) return rc;
  TcGemmArgs g{};
  g.M = M; g.N = N; g.K = K; g.nseg = split ? 3 : 1; g.st = st;
  g.a_off[2] = a_mn ? K : M; g.b_off[1] = b_mn ? K : N;
  g.outF = D; g.ldo = ldo;
  if (!a_mn && !b_mn) return tc_launch_n<false, false, TC_EPI_PLAIN>(h, s, ta, tb, g);
  if (!a_mn && b_mn) return tc_launch_n<false, true, TC_EPI_PLAIN>(h, s, ta, tb, g);
  if (a_mn && !b_mn) return tc_launch_n<true, false, TC_EPI_PLAIN>(h, s, ta, tb, g);
  return tc_launch_n<true, true, TC_EPI_PLAIN>(h, s, ta, tb, g);
}

}  // namespace conqur
