"""CPU-side checks of the boundary: the library loads, exports what the header declares,
and its host-only logic (argument checks, workspace sizing, Newton-Schulz planning) behaves."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2605_10793_b200 import build, binding
    build.build()
    binding.load()
    return binding


def test_every_declared_symbol_is_exported(B):
    hdr = open(os.path.join(ROOT, "include", "conqur.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(conqur_[a-zA-Z_]+)\s*\(", hdr))
    assert declared, "no declarations parsed"
    lib = B.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)


def test_workspace_bytes_and_argument_checks(B):
    ok = B.make_config(in_dtype=B.CONQUR_F32, mode=B.CONQUR_EXACT_F32, n_max=2048)
    small = B.conqur_workspace_bytes(128, ok)
    big = B.conqur_workspace_bytes(256, ok)
    assert 0 < small < big
    assert small % 256 == 0
    for bad in (dict(n_max=0), dict(batch=0), dict(quant_bits=1), dict(quant_bits=9), dict(prior_rel=-1.0),
                dict(in_dtype=7), dict(mode=5)):
        kw = dict(in_dtype=B.CONQUR_F32, mode=B.CONQUR_EXACT_F32, n_max=16)
        kw.update(bad)
        assert B.conqur_workspace_bytes(64, B.make_config(**kw)) == 0, bad
    assert B.conqur_workspace_bytes(1, ok) == 0
    wrong = B.make_config(in_dtype=B.CONQUR_F32, mode=B.CONQUR_EXACT_F32, n_max=16)
    wrong.struct_size = 8
    assert B.conqur_workspace_bytes(64, wrong) == 0
    # tensor-core mode wants d to be a multiple of 128
    tc = B.make_config(in_dtype=B.CONQUR_BF16, mode=B.CONQUR_TC_BF16, n_max=256)
    assert B.conqur_workspace_bytes(100, tc) == 0
    # deferring batches: tensor-core single-problem contexts only; every per-row buffer grows with the queue
    plain = B.conqur_workspace_bytes(256, tc)
    queued = B.conqur_workspace_bytes(256, B.make_config(in_dtype=B.CONQUR_BF16, mode=B.CONQUR_TC_BF16, n_max=256, defer_batches=8))
    assert queued >= plain + 7 * 4 * 256 * 256
    assert B.conqur_workspace_bytes(128, B.make_config(in_dtype=B.CONQUR_BF16, mode=B.CONQUR_TC_BF16, n_max=256, batch=4,
                                                       defer_batches=8)) == 0
    assert B.conqur_workspace_bytes(64, B.make_config(in_dtype=B.CONQUR_F32, mode=B.CONQUR_EXACT_F32, n_max=16, defer_batches=2)) == 0
    assert B.conqur_workspace_bytes(64, B.make_config(in_dtype=B.CONQUR_F32, mode=B.CONQUR_EXACT_F32, n_max=16, debug_flags=64)) == 0
    # guard bands (test hook) cost 256 bytes per workspace region
    guarded = B.conqur_workspace_bytes(128, B.make_config(in_dtype=B.CONQUR_F32, mode=B.CONQUR_EXACT_F32, n_max=2048,
                                                          debug_flags=B.CONQUR_DEBUG_CANARIES))
    assert small < guarded <= small + 48 * 256


def test_init_rejects_bad_arguments_without_a_device(B):
    cfg = B.make_config(in_dtype=B.CONQUR_F32, mode=B.CONQUR_EXACT_F32, n_max=16)
    lib = B.load()
    h = C.c_void_p()
    assert lib.conqur_init(C.byref(h), 64, C.byref(cfg), None, 0, None) == -1          # null workspace
    assert lib.conqur_init(C.byref(h), 64, C.byref(cfg), C.c_void_p(256 + 8), 1 << 30, None) == -1  # misaligned
    assert lib.conqur_init(C.byref(h), 64, C.byref(cfg), C.c_void_p(4096), 16, None) == -2   # too small
    assert h.value is None
    assert lib.conqur_update(None) == -1 and lib.conqur_step(None, None, 1, 1) == -1
    assert B.strerror(0) == "ok" and "Newton" in B.strerror(-6)


@pytest.mark.parametrize("l0", [1e-2, 1e-4, 1e-7, 1e-9])
def test_planned_polynomials_drive_the_assumed_interval_to_one(B, l0):
    abc = B.conqur_plan_schedule(l0)
    x = np.concatenate([np.logspace(np.log10(l0), 0, 4000), np.linspace(l0, 1, 4000)])
    lo_track = l0
    for a, b, c in abc:
        x = a * x + b * x ** 3 + c * x ** 5
        assert x.max() <= 1.0 + 1e-9                   # never leaves [0, 1]: no divergence
        assert x.min() > lo_track                      # the bottom of the spectrum only moves up
        lo_track = x.min()
    assert 1.0 - x.min() < 5e-6 and len(abc) <= 20
    # below the assumed bound singular values still grow monotonically (slower convergence, no failure)
    y = np.array([l0 * 1e-3])
    for a, b, c in abc:
        y2 = a * y + b * y ** 3 + c * y ** 5
        assert y2 > y
        y = y2


def test_lifting_steps_never_push_a_large_singular_value_down(B):
    """The repeated lifting quintic keeps everything that has reached [0.05, 1] above its floor (about 0.2), so
    directions that already carry weight are never brought back to the rounding-noise level."""
    abc = B.conqur_plan_schedule(1e-9)
    a, b, c = abc[0]
    assert np.allclose(abc[1], abc[0]) and np.allclose(abc[5], abc[0])      # the same quintic, repeated
    x = np.linspace(0.05, 1.0, 100001)
    p = a * x + b * x ** 3 + c * x ** 5
    assert p.min() > 0.19 and p.max() <= 1.0 / 1.02 + 1e-9
    x = np.logspace(-9, 0, 20001)
    for k in range(40):                                                       # far more often than planned
        x = a * x + b * x ** 3 + c * x ** 5
    assert x.min() > 0.19 and x.max() <= 1.0


def test_plan_for_a_step_budget(B):
    for steps in (4, 8, 12):
        abc = B.conqur_plan_schedule(0.0, steps)
        assert len(abc) <= steps
    assert len(B.conqur_plan_schedule(0.0, 8)) == 8


def test_lifting_polynomial_is_the_minimax_quintic(B):
    # equioscillation: |1 - p| attains the same maximum at both ends and two interior points of [0.05, 1]
    lf = 0.05
    a, b, c = B.conqur_plan_schedule(1e-6)[0]
    x = np.linspace(lf, 1.0, 200001)
    p = a * x + b * x ** 3 + c * x ** 5
    top = p.max()
    err = 1 - p / top                                  # undo the output rescaling: p/top ranges over [1-2E/(1+E), 1]
    assert abs(err[0] - err.max()) < 1e-6
    assert abs(p[-1] - top) < 1e-6 * top
    interior_min = p[(x > 0.4) & (x < 0.95)].min()
    assert abs((1 - interior_min / top) - err[0]) < 1e-6
