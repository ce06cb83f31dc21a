"""Thin ctypes binding of libconqur.so (argument marshalling only).

Function names mirror the C ABI in ``include/conqur.h``.  PyTorch supplies device
memory and the stream; every step of the path runs in the library's kernels.
The library is required: there is no fallback if it is missing or no GPU exists.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libconqur.so")
_lib = None

CONQUR_F32, CONQUR_BF16 = 0, 1
CONQUR_EXACT_F32, CONQUR_TC_BF16 = 0, 1
CONQUR_QUANT_SYMMETRIC, CONQUR_QUANT_ZEROPOINT = 0, 1
CONQUR_FOLD_INPUT, CONQUR_FOLD_OUTPUT = 0, 1
CONQUR_DEBUG_CANARIES, CONQUR_DEBUG_SINGLE_CTA, CONQUR_DEBUG_NO_GRAPH = 1, 2, 4
CONQUR_HADAMARD_CUDA_CORES_ONLY = 1

# Test support: when set, every Context is created with guard bands around its workspace regions, registers itself
# here, and has them checked when it is closed; damaged bands are collected in CANARY_FAILURES.
DEBUG_CANARIES = False
CANARY_FAILURES: list = []
_live_contexts = None

EXPORTS = [
    "conqur_workspace_bytes", "conqur_init", "conqur_destroy", "conqur_set_R", "conqur_step",
    "conqur_step_batched", "conqur_step_batched_range", "conqur_update", "conqur_get_R", "conqur_get_objective", "conqur_get_objective_async", "conqur_get_M",
    "conqur_set_M", "conqur_debug_get_signs", "conqur_debug_capture_signs", "conqur_get_stats", "conqur_debug_check_canaries", "conqur_debug_trace_heads", "conqur_plan_schedule", "conqur_debug_gemm",
    "conqur_set_profiling", "conqur_get_profile", "conqur_objective_noalloc", "conqur_debug_wait_timeout",
    "conqur_get_diagnostics", "conqur_fold_scratch_bytes", "conqur_fold_weight", "conqur_hadamard_rows", "conqur_hadamard_status",
    "conqur_strerror",
]


class conqur_config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("in_dtype", C.c_int32), ("mode", C.c_int32), ("quant_bits", C.c_int32),
        ("ns_steps", C.c_int32), ("ns_max_steps", C.c_int32), ("orth_tol", C.c_float), ("prior_rel", C.c_float),
        ("ns_sigma_min_rel", C.c_float), ("n_max", C.c_int64), ("batch", C.c_int32),
        ("quant_mode", C.c_int32), ("clip_ratio", C.c_float), ("diagnostics", C.c_int32),
        ("defer_batches", C.c_int32), ("ns_gram_single_pass_tau", C.c_float), ("ns_lo_gap_budget", C.c_float),
        ("debug_flags", C.c_int32),
    ]


class conqur_stats(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("status", C.c_int32), ("ns_steps_used", C.c_int32), ("updates", C.c_int32),
        ("orth_err", C.c_float), ("orth_fro", C.c_float), ("scale", C.c_float), ("n_skipped", C.c_int64),
        ("last_J", C.c_double), ("last_N", C.c_int64), ("ns_lift_plan", C.c_int32), ("reserved", C.c_int32),
    ]


class conqur_diagnostics(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("reserved", C.c_int32), ("sum_pr_over_d", C.c_double), ("sum_rho", C.c_double),
        ("qerr_num", C.c_double), ("qerr_den", C.c_double), ("n_tokens", C.c_int64),
    ]


class conqur_profile(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("reserved", C.c_int32), ("launches", C.c_int64 * 8),
        ("timed_launches", C.c_int64 * 8), ("flops", C.c_double * 8), ("ms", C.c_double * 8),
        ("total_launches", C.c_int64),
    ]


KERNEL_CLASSES = ["rownorm", "rotate_target", "accumulate", "ns_residual", "ns_poly", "ns_next", "other", "unused"]


class ConqurError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})")


def load() -> C.CDLL:
    """Load libconqur.so (built in-tree by paper_2605_10793_b200.build); fail loudly if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2605_10793_b200.build` "
                           "(the CUDA library is the only implementation; there is no fallback)")
    lib = C.CDLL(_LIB_PATH)
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int32
    lib.conqur_workspace_bytes.restype = C.c_size_t
    lib.conqur_workspace_bytes.argtypes = [i32, C.POINTER(conqur_config)]
    lib.conqur_init.restype = C.c_int
    lib.conqur_init.argtypes = [C.POINTER(vp), i32, C.POINTER(conqur_config), vp, C.c_size_t, vp]
    lib.conqur_destroy.restype = C.c_int
    lib.conqur_destroy.argtypes = [vp]
    lib.conqur_set_R.restype = C.c_int
    lib.conqur_set_R.argtypes = [vp, vp]
    lib.conqur_step.restype = C.c_int
    lib.conqur_step.argtypes = [vp, vp, i64, i64]
    lib.conqur_step_batched.restype = C.c_int
    lib.conqur_step_batched.argtypes = [vp, vp, i64, i64, i64]
    lib.conqur_step_batched_range.restype = C.c_int
    lib.conqur_step_batched_range.argtypes = [vp, vp, i64, i64, i64, i32, i32]
    lib.conqur_update.restype = C.c_int
    lib.conqur_update.argtypes = [vp]
    lib.conqur_get_R.restype = C.c_int
    lib.conqur_get_R.argtypes = [vp, vp]
    lib.conqur_get_objective.restype = C.c_int
    lib.conqur_get_objective.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.conqur_get_objective_async.restype = C.c_int
    lib.conqur_get_objective_async.argtypes = [vp, vp, vp]
    lib.conqur_get_M.restype = C.c_int
    lib.conqur_get_M.argtypes = [vp, vp]
    lib.conqur_set_M.restype = C.c_int
    lib.conqur_set_M.argtypes = [vp, vp, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.conqur_debug_get_signs.restype = C.c_int
    lib.conqur_debug_get_signs.argtypes = [vp, vp, i64]
    lib.conqur_debug_capture_signs.restype = C.c_int
    lib.conqur_debug_capture_signs.argtypes = [vp, vp, i64]
    lib.conqur_debug_trace_heads.restype = C.c_int
    lib.conqur_debug_trace_heads.argtypes = [vp, vp, i64]
    lib.conqur_debug_check_canaries.restype = C.c_int
    lib.conqur_debug_check_canaries.argtypes = [vp]
    lib.conqur_get_stats.restype = C.c_int
    lib.conqur_get_stats.argtypes = [vp, C.POINTER(conqur_stats)]
    lib.conqur_plan_schedule.restype = C.c_int
    lib.conqur_plan_schedule.argtypes = [C.c_double, i32, C.POINTER(C.c_double), i32]
    lib.conqur_set_profiling.restype = C.c_int
    lib.conqur_set_profiling.argtypes = [vp, i32]
    lib.conqur_get_profile.restype = C.c_int
    lib.conqur_get_profile.argtypes = [vp, C.POINTER(conqur_profile)]
    lib.conqur_objective_noalloc.restype = C.c_int
    lib.conqur_objective_noalloc.argtypes = [vp, i32, i64, i32, i64, vp, vp, vp, vp]
    lib.conqur_debug_gemm.restype = C.c_int
    lib.conqur_debug_gemm.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp]
    lib.conqur_get_diagnostics.restype = C.c_int
    lib.conqur_get_diagnostics.argtypes = [vp, C.POINTER(conqur_diagnostics)]
    lib.conqur_debug_wait_timeout.restype = C.c_int
    lib.conqur_debug_wait_timeout.argtypes = [vp, i64, vp]
    lib.conqur_fold_scratch_bytes.restype = i64
    lib.conqur_fold_scratch_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.conqur_fold_weight.restype = C.c_int
    lib.conqur_fold_weight.argtypes = [vp, i64, i32, i32, vp, i32, i32, i32, vp, i64, vp, i64, vp]
    lib.conqur_hadamard_rows.restype = C.c_int
    lib.conqur_hadamard_rows.argtypes = [vp, i32, i64, i32, i64, vp, i32, i64, i32, vp]
    lib.conqur_hadamard_status.restype = C.c_int
    lib.conqur_hadamard_status.argtypes = [vp]
    lib.conqur_strerror.restype = C.c_char_p
    lib.conqur_strerror.argtypes = [C.c_int]
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().conqur_strerror(int(status)).decode()


def make_config(*, in_dtype=CONQUR_BF16, mode=CONQUR_TC_BF16, quant_bits=0, ns_steps=0, ns_max_steps=0,
                orth_tol=0.0, prior_rel=0.0, ns_sigma_min_rel=0.0, n_max=1, batch=1, quant_mode=CONQUR_QUANT_SYMMETRIC,
                clip_ratio=0.0, diagnostics=0, defer_batches=0, ns_gram_single_pass_tau=0.0, ns_lo_gap_budget=0.0,
                debug_flags=0) -> conqur_config:
    return conqur_config(C.sizeof(conqur_config), in_dtype, mode, quant_bits, ns_steps, ns_max_steps, orth_tol,
                         prior_rel, ns_sigma_min_rel, n_max, batch, quant_mode, clip_ratio, diagnostics,
                         defer_batches, ns_gram_single_pass_tau, ns_lo_gap_budget, debug_flags)


# ---- the C calls, one to one -------------------------------------------------------------------

def conqur_workspace_bytes(d: int, cfg: conqur_config) -> int:
    return int(load().conqur_workspace_bytes(d, C.byref(cfg)))


def conqur_init(d: int, cfg: conqur_config, workspace_ptr: int, workspace_bytes: int, stream_ptr: int) -> int:
    h = C.c_void_p()
    rc = load().conqur_init(C.byref(h), d, C.byref(cfg), workspace_ptr, workspace_bytes, stream_ptr)
    if rc != 0:
        raise ConqurError(rc, "conqur_init")
    return h.value


def conqur_destroy(h: int) -> int:
    return load().conqur_destroy(h)


def conqur_set_R(h: int, r_ptr: int) -> int:
    return load().conqur_set_R(h, r_ptr)


def conqur_step(h: int, x_ptr: int, n: int, ld: int) -> int:
    return load().conqur_step(h, x_ptr, n, ld)


def conqur_step_batched(h: int, x_ptr: int, n: int, ld: int, problem_stride: int) -> int:
    return load().conqur_step_batched(h, x_ptr, n, ld, problem_stride)


def conqur_step_batched_range(h: int, x_ptr: int, n: int, ld: int, problem_stride: int, first: int, count: int) -> int:
    return load().conqur_step_batched_range(h, x_ptr, n, ld, problem_stride, first, count)


def conqur_update(h: int) -> int:
    return load().conqur_update(h)


def conqur_get_R(h: int, out_ptr: int) -> int:
    return load().conqur_get_R(h, out_ptr)


def conqur_get_objective(h: int, batch: int) -> Tuple[int, np.ndarray, np.ndarray]:
    j = (C.c_double * batch)()
    n = (C.c_int64 * batch)()
    rc = load().conqur_get_objective(h, j, n)
    return rc, np.array(j[:], dtype=np.float64), np.array(n[:], dtype=np.int64)


def conqur_get_M(h: int, out_ptr: int) -> int:
    return load().conqur_get_M(h, out_ptr)


def conqur_set_M(h: int, m_ptr: int, j_sum, n_tokens) -> int:
    j_sum = np.atleast_1d(np.asarray(j_sum, dtype=np.float64))
    n_tokens = np.atleast_1d(np.asarray(n_tokens, dtype=np.int64))
    j = (C.c_double * j_sum.size)(*j_sum.tolist())
    n = (C.c_int64 * n_tokens.size)(*n_tokens.tolist())
    return load().conqur_set_M(h, m_ptr, j, n)


def conqur_debug_get_signs(h: int, out_ptr: int, capacity_rows: int) -> int:
    return load().conqur_debug_get_signs(h, out_ptr, capacity_rows)


def conqur_debug_capture_signs(h: int, buf_ptr: int, capacity_rows: int) -> int:
    return load().conqur_debug_capture_signs(h, buf_ptr, capacity_rows)


def conqur_get_stats(h: int) -> Tuple[int, conqur_stats]:
    st = conqur_stats()
    st.struct_size = C.sizeof(conqur_stats)
    rc = load().conqur_get_stats(h, C.byref(st))
    return rc, st


def conqur_set_profiling(h: int, enabled: bool) -> int:
    return load().conqur_set_profiling(h, int(enabled))


def conqur_get_profile(h: int) -> Tuple[int, conqur_profile]:
    pr = conqur_profile()
    pr.struct_size = C.sizeof(conqur_profile)
    rc = load().conqur_get_profile(h, C.byref(pr))
    return rc, pr


def conqur_plan_schedule(sigma_min_rel: float = 0.0, ns_steps: int = 0, max_steps: int = 100) -> np.ndarray:
    buf = (C.c_double * (3 * max_steps))()
    n = load().conqur_plan_schedule(sigma_min_rel, ns_steps, buf, max_steps)
    if n < 0:
        raise ConqurError(n, "conqur_plan_schedule")
    return np.array(buf[: 3 * n], dtype=np.float64).reshape(n, 3)


def conqur_objective_noalloc(x_ptr: int, in_dtype: int, n: int, d: int, ld: int, r_ptr: int, j_out_ptr: int,
                             n_out_ptr: int, stream_ptr: int) -> int:
    """Objective of one batch using only the library's built-in scratch (see include/conqur.h)."""
    return load().conqur_objective_noalloc(x_ptr, in_dtype, n, d, ld, r_ptr, j_out_ptr, n_out_ptr, stream_ptr)


def conqur_debug_wait_timeout(limit_cycles: int) -> int:
    """Run the bounded-wait probe (see include/conqur.h); returns the status code (-8 = the wait gave up as designed)."""
    import torch
    scratch = torch.zeros(512, dtype=torch.uint8, device="cuda")
    return load().conqur_debug_wait_timeout(scratch.data_ptr(), int(limit_cycles), torch.cuda.current_stream().cuda_stream)


def conqur_debug_gemm(a, b, m: int, n: int, k: int, a_mn: bool, b_mn: bool, split: bool = False):
    """D = A x B (see include/conqur.h) for torch bf16 CUDA tensors; returns an fp32 (m, n) tensor."""
    import torch
    out = torch.empty((m, n), dtype=torch.float32, device="cuda")
    scratch = torch.zeros(512, dtype=torch.uint8, device="cuda")
    rc = load().conqur_debug_gemm(a.data_ptr(), b.data_ptr(), out.data_ptr(), m, n, k, int(a_mn), int(b_mn),
                                  int(split), scratch.data_ptr(), torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise ConqurError(rc, "conqur_debug_gemm")
    return out


def conqur_fold_scratch_bytes(rows: int, cols: int, block: int, side: int, mode: int) -> int:
    return int(load().conqur_fold_scratch_bytes(rows, cols, block, side, mode))


def conqur_fold_weight(w, r, side: str, mode: str = "tc"):
    """Appendix A: W' = W R (side "input") or R^T W (side "output"); see include/conqur.h.

    w: fp32 CUDA tensor (rows, cols), unit column stride.  r: fp32 CUDA tensor, one (b, b) rotation or a stack
    (k, b, b) of diagonal blocks.  Returns a new fp32 tensor (rows, cols)."""
    import torch
    assert w.is_cuda and w.dtype == torch.float32 and w.dim() == 2 and w.stride(1) == 1
    assert r.is_cuda and r.dtype == torch.float32 and r.is_contiguous() and r.shape[-1] == r.shape[-2]
    side_c = {"input": CONQUR_FOLD_INPUT, "output": CONQUR_FOLD_OUTPUT}[side]
    mode_c = {"exact": CONQUR_EXACT_F32, "tc": CONQUR_TC_BF16}[mode]
    rows, cols, block = int(w.shape[0]), int(w.shape[1]), int(r.shape[-1])
    nbytes = conqur_fold_scratch_bytes(rows, cols, block, side_c, mode_c)
    if nbytes < 0:
        raise ConqurError(-1, "conqur_fold_scratch_bytes")
    scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    sp = (scratch.data_ptr() + 255) // 256 * 256
    out = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
    rc = load().conqur_fold_weight(w.data_ptr(), w.stride(0), rows, cols, r.data_ptr(), block, side_c, mode_c,
                                   out.data_ptr(), out.stride(0), sp, nbytes, torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise ConqurError(rc, "conqur_fold_weight")
    return out


def conqur_hadamard_rows(x, out_dtype=None, out=None, cuda_cores_only=False):
    """y = x H_d / sqrt(d) for every row of a 2-D fp32 / bf16 CUDA tensor (see include/conqur.h)."""
    import torch
    code = {torch.float32: CONQUR_F32, torch.bfloat16: CONQUR_BF16}
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1 and x.dtype in code
    if out is None:
        out = torch.empty(x.shape, dtype=out_dtype or x.dtype, device="cuda")
    assert out.is_cuda and out.shape == x.shape and out.stride(1) == 1 and out.dtype in code
    rc = load().conqur_hadamard_rows(x.data_ptr(), code[x.dtype], x.shape[0], x.shape[1], x.stride(0), out.data_ptr(),
                                     code[out.dtype], out.stride(0),
                                     CONQUR_HADAMARD_CUDA_CORES_ONLY if cuda_cores_only else 0,
                                     torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise ConqurError(rc, "conqur_hadamard_rows")
    return out


def conqur_hadamard_status() -> int:
    """Synchronise the current stream; status of the transform kernels run since the last call (0 = ok)."""
    import torch
    return int(load().conqur_hadamard_status(torch.cuda.current_stream().cuda_stream))


# ---- convenience wrapper: owns the workspace tensor, checks status codes ------------------------

class Context:
    """One calibration context on the current CUDA device / current torch stream."""

    def __init__(self, d: int, n_max: int, *, in_dtype="bf16", mode="tc", quant_bits=0, batch=1, prior_rel=0.0,
                 ns_steps=0, ns_max_steps=0, orth_tol=0.0, ns_sigma_min_rel=0.0, stream=None, quant_mode="sym", clip_ratio=0.0,
                 diagnostics=False, defer_batches=0, ns_gram_single_pass_tau=0.0, ns_lo_gap_budget=0.0, debug_flags=0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("conqur needs a CUDA device (B200); there is no CPU path")
        self.torch = torch
        self.d, self.n_max, self.batch = int(d), int(n_max), int(batch)
        self.in_dtype = {"f32": CONQUR_F32, "bf16": CONQUR_BF16}[in_dtype]
        self.mode = {"exact": CONQUR_EXACT_F32, "tc": CONQUR_TC_BF16}[mode]
        self.cfg = make_config(in_dtype=self.in_dtype, mode=self.mode, quant_bits=quant_bits, ns_steps=ns_steps,
                               ns_max_steps=ns_max_steps, orth_tol=orth_tol, prior_rel=prior_rel,
                               ns_sigma_min_rel=ns_sigma_min_rel, n_max=n_max, batch=batch,
                               quant_mode={"sym": CONQUR_QUANT_SYMMETRIC, "zp": CONQUR_QUANT_ZEROPOINT}[quant_mode],
                               clip_ratio=clip_ratio, diagnostics=int(bool(diagnostics)), defer_batches=defer_batches,
                               ns_gram_single_pass_tau=ns_gram_single_pass_tau, ns_lo_gap_budget=ns_lo_gap_budget,
                               debug_flags=debug_flags | (CONQUR_DEBUG_CANARIES if DEBUG_CANARIES else 0))
        nbytes = conqur_workspace_bytes(self.d, self.cfg)
        if nbytes == 0:
            raise ConqurError(-1, "conqur_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self.h = conqur_init(self.d, self.cfg, self._ws_ptr, nbytes, self.stream.cuda_stream)
        if DEBUG_CANARIES:
            global _live_contexts
            if _live_contexts is None:
                import weakref
                _live_contexts = weakref.WeakSet()
            _live_contexts.add(self)

    def _chk(self, rc: int, where: str):
        if rc != 0:
            raise ConqurError(rc, where)

    def _x_dtype(self):
        return self.torch.float32 if self.in_dtype == CONQUR_F32 else self.torch.bfloat16

    def set_R(self, r):
        assert r.is_cuda and r.dtype == self.torch.float32 and r.is_contiguous()
        assert r.numel() == self.batch * self.d * self.d
        self._chk(conqur_set_R(self.h, r.data_ptr()), "conqur_set_R")

    def step(self, x):
        assert x.is_cuda and x.dtype == self._x_dtype() and x.dim() == 2 and x.stride(1) == 1
        self._chk(conqur_step(self.h, x.data_ptr(), x.shape[0], x.stride(0)), "conqur_step")

    def step_batched(self, x, n: int, ld: int, problem_stride: int):
        assert x.is_cuda and x.dtype == self._x_dtype()
        self._chk(conqur_step_batched(self.h, x.data_ptr(), n, ld, problem_stride), "conqur_step_batched")

    def step_batched_range(self, x, n: int, ld: int, problem_stride: int, first: int, count: int):
        assert x.is_cuda and x.dtype == self._x_dtype()
        self._chk(conqur_step_batched_range(self.h, x.data_ptr(), n, ld, problem_stride, first, count),
                  "conqur_step_batched_range")

    def update(self):
        self._chk(conqur_update(self.h), "conqur_update")

    def get_R(self, check=True):
        shape = (self.d, self.d) if self.batch == 1 else (self.batch, self.d, self.d)
        out = self.torch.empty(shape, dtype=self.torch.float32, device="cuda")
        rc = conqur_get_R(self.h, out.data_ptr())
        if check:
            self._chk(rc, "conqur_get_R")
        return out

    def get_M(self, check=True):
        shape = (self.d, self.d) if self.batch == 1 else (self.batch, self.d, self.d)
        out = self.torch.empty(shape, dtype=self.torch.float32, device="cuda")
        rc = conqur_get_M(self.h, out.data_ptr())
        if check:
            self._chk(rc, "conqur_get_M")
        return out

    def set_M(self, m, j_sum, n_tokens):
        assert m.is_cuda and m.dtype == self.torch.float32 and m.is_contiguous()
        self._chk(conqur_set_M(self.h, m.data_ptr(), j_sum, n_tokens), "conqur_set_M")

    def get_objective(self, check=True):
        rc, j, n = conqur_get_objective(self.h, self.batch)
        if check:
            self._chk(rc, "conqur_get_objective")
        return (float(j[0]), int(n[0])) if self.batch == 1 else (j, n)

    def get_objective_async(self, j_host, n_host):
        """Enqueue the read of (J, N) into page-locked host tensors (float64 / int64, one entry per problem) on the
        context's stream and return at once; the values are there once the stream has passed this point."""
        t = self.torch
        assert j_host.device.type == "cpu" and j_host.dtype == t.float64 and j_host.numel() == self.batch and j_host.is_contiguous()
        assert n_host.device.type == "cpu" and n_host.dtype == t.int64 and n_host.numel() == self.batch and n_host.is_contiguous()
        self._chk(load().conqur_get_objective_async(self.h, j_host.data_ptr(), n_host.data_ptr()), "conqur_get_objective_async")

    def get_diagnostics(self):
        """Section-4 diagnostics since the last update: list of dicts (one per problem)."""
        arr = (conqur_diagnostics * self.batch)()
        for a in arr:
            a.struct_size = C.sizeof(conqur_diagnostics)
        self._chk(load().conqur_get_diagnostics(self.h, arr), "conqur_get_diagnostics")
        return [dict(sum_pr_over_d=a.sum_pr_over_d, sum_rho=a.sum_rho, qerr_num=a.qerr_num, qerr_den=a.qerr_den,
                     n_tokens=a.n_tokens) for a in arr]

    def debug_get_signs(self, n: int, problems: int = 1):
        """Sign decisions of the last step call: (n, d) int8, or (problems, n, d) for a batched call."""
        shape = (n, self.d) if problems == 1 else (problems, n, self.d)
        out = self.torch.empty(shape, dtype=self.torch.int8, device="cuda")
        self._chk(conqur_debug_get_signs(self.h, out.data_ptr(), n * problems), "conqur_debug_get_signs")
        return out

    def debug_capture_signs(self, buf):
        """Tensor-core contexts with batch > 1: let the following batched steps write their sign decisions to `buf`
        (int8 CUDA tensor, rows x d; None stops it).  The tensor must stay alive while the capture is on."""
        if buf is None:
            self._sign_buf = None
            self._chk(conqur_debug_capture_signs(self.h, 0, 0), "conqur_debug_capture_signs")
            return
        assert buf.is_cuda and buf.dtype == self.torch.int8 and buf.is_contiguous()
        self._sign_buf = buf
        self._chk(conqur_debug_capture_signs(self.h, buf.data_ptr(), buf.numel() // self.d), "conqur_debug_capture_signs")

    def get_stats(self) -> conqur_stats:
        rc, st = conqur_get_stats(self.h)
        self._chk(rc, "conqur_get_stats")
        return st

    def set_profiling(self, enabled: bool):
        self._chk(conqur_set_profiling(self.h, enabled), "conqur_set_profiling")

    def get_profile(self) -> dict:
        rc, pr = conqur_get_profile(self.h)
        self._chk(rc, "conqur_get_profile")
        out = {"total_launches": int(pr.total_launches)}
        for i, name in enumerate(KERNEL_CLASSES[:7]):
            out[name] = {"launches": int(pr.launches[i]), "timed": int(pr.timed_launches[i]),
                         "flops": float(pr.flops[i]), "ms": float(pr.ms[i])}
        return out

    def debug_trace_heads(self, buf):
        """Per-head tensor-core contexts: record the step kernel's timeline into `buf` (int64 CUDA tensor of at least
        96 * 16 entries; None stops it).  See include/conqur.h for the slots."""
        self._trace_buf = buf
        ptr, cap = (0, 0) if buf is None else (buf.data_ptr(), buf.numel())
        self._chk(load().conqur_debug_trace_heads(self.h, ptr, cap), "conqur_debug_trace_heads")

    def check_canaries(self) -> int:
        """Guard bands of the workspace that were overwritten (0 = intact); needs CONQUR_DEBUG_CANARIES."""
        rc = load().conqur_debug_check_canaries(self.h)
        if rc < 0:
            raise ConqurError(rc, "conqur_debug_check_canaries")
        return rc

    def close(self):
        if getattr(self, "h", None):
            if self.cfg.debug_flags & CONQUR_DEBUG_CANARIES:
                bad = load().conqur_debug_check_canaries(self.h)
                if bad != 0:
                    CANARY_FAILURES.append((self.d, self.batch, self.mode, bad))
            conqur_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
