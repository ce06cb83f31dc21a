// Tensor-core (tcgen05 / TMEM / TMA) mode.  Placeholder interface until the kernels land.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/conqur.h"
#include "conqur_internal.h"

namespace conqur {

struct TcLayout { size_t dummy; };
struct TcHost { int dummy; };

inline bool tc_supported_shape(int, int) { return false; }
template <typename Take>
inline void tc_make_layout(int, int, int64_t, int, TcLayout*, Take&&) {}
inline int tc_init(TcHost*, char*, const TcLayout&, int, int, int64_t, int, float*, float*, float*, float*, float*,
                   float*, float*, DevState*, double*, float*) { return CONQUR_ERR_UNSUPPORTED; }
inline int tc_refresh_R(TcHost&, cudaStream_t, int) { return CONQUR_ERR_UNSUPPORTED; }
inline int tc_step(TcHost&, cudaStream_t, const void*, int, int64_t, int64_t, int64_t) { return CONQUR_ERR_UNSUPPORTED; }
inline int tc_ns_begin(TcHost&, cudaStream_t) { return CONQUR_ERR_UNSUPPORTED; }
inline int tc_ns_residual(TcHost&, cudaStream_t, int) { return CONQUR_ERR_UNSUPPORTED; }
inline int tc_ns_parts(const TcHost&) { return 0; }
inline int tc_ns_poly_next(TcHost&, cudaStream_t, int) { return CONQUR_ERR_UNSUPPORTED; }
inline const __nv_bfloat16* tc_ct_ptr(const TcHost&) { return nullptr; }
inline int64_t tc_ct_ld(const TcHost&) { return 0; }

}  // namespace conqur
