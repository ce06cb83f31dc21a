"""GPU parity, tensor-core mode (bf16 operands, fp32 accumulation on tcgen05) through the C ABI."""
import numpy as np
import pytest

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I
from tests.parity_util import TOL, assert_step, effective_m, log_parity, step_parity, update_parity

pytestmark = pytest.mark.gpu
T = TOL["tc"]


def _torch():
    import torch
    return torch


def _ctx(**kw):
    from paper_2605_10793_b200 import binding as B
    return B.Context(mode="tc", **kw)


def _dev(x, dtype):
    torch = _torch()
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _check_step(ctx, x_np, dtype, quant_bits=0, before=None):
    r = ctx.get_R().cpu().numpy().astype(np.float64)
    ctx.step(_dev(x_np, dtype))
    j, n = ctx.get_objective()
    m = ctx.get_M().cpu().numpy().astype(np.float64)
    s = ctx.debug_get_signs(x_np.shape[0]).cpu().numpy()
    mb, jb, nb = before if before is not None else (None, 0.0, 0)
    x64 = (I.round_to_bf16(x_np) if dtype == "f32" else x_np).astype(np.float64)   # fp32 input is rounded on the way in
    rep = step_parity(x64, r, s, m, j, n, "tc", quant_bits, mb, jb, nb)
    assert rep["N_equal"]
    assert rep["J_rel"] <= T["J"], rep
    assert rep["M_rel_tie_aware"] <= T["M"], rep
    assert rep["flips_outside_band"] == 0, rep
    assert rep["flip_frac"] < 2e-2, rep
    return rep, m, j, n, r


def _check_update(ctx, m64, r_prev64, prior_rel=0.0):
    ctx.update()
    st = ctx.get_stats()
    assert st.status == 0, st.status
    r_new = ctx.get_R().cpu().numpy().astype(np.float64)
    rep = update_parity(effective_m(m64, r_prev64, prior_rel), r_new)
    assert rep["orth"] <= T["orth"], rep
    assert rep["gap"] <= T["gap"], rep
    j, n = ctx.get_objective()
    assert j == 0.0 and n == 0 and not ctx.get_M().any().item()
    return rep, st


def test_c0_in_tensor_core_mode():
    """d=128 alternation with the fp32 batch rounded to bf16 inside the library."""
    w = I.WORKLOADS["c0"]
    x = I.batch(w, 0)
    ctx = _ctx(d=w.d, n_max=w.n, in_dtype="f32")
    js = []
    for it in range(4):
        rep, m, j, n, r = _check_step(ctx, x, "f32")
        js.append(j / n)
        _check_update(ctx, m, r)
    assert all(b >= a * (1 - 1e-3) for a, b in zip(js, js[1:])), js


@pytest.mark.parametrize("d,n", [(256, 1000), (384, 2048), (512, 300)])
def test_stream_steps_then_update(d, n):
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=max(2, d // 256), r0="hadamard" if d & (d - 1) == 0 else "qr")
    ctx = _ctx(d=d, n_max=n, in_dtype="bf16", prior_rel=0.0 if 3 * n >= 4 * d else 1e-2)
    ctx.set_R(_dev(I.initial_rotation(w), "f32"))
    before = None
    r = None
    for b in range(3):
        rep, m, j, nn, r = _check_step(ctx, I.batch(w, b), "bf16", before=before)
        before = (m, j, nn)
    _check_update(ctx, before[0], r, prior_rel=ctx.cfg.prior_rel)


def test_quant_mode_int4_tc():
    d, n = 256, 1024
    w = I.scaled(I.WORKLOADS["c4a"], d=d, n=n, n_outlier=2)
    ctx = _ctx(d=d, n_max=n, in_dtype="bf16", quant_bits=4)
    ctx.set_R(_dev(I.initial_rotation(w), "f32"))
    rep, m, j, nn, r = _check_step(ctx, I.batch(w, 0), "bf16", quant_bits=4)
    _check_update(ctx, m, r)


def test_skipped_rows_tc():
    d, n = 128, 200
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2)
    x = I.batch(w, 0).copy()
    x[7] = 0.0
    x[100, 3] = np.nan
    x[150, 100] = -np.inf
    ctx = _ctx(d=d, n_max=n, in_dtype="bf16")
    ctx.step(_dev(x, "bf16"))
    j, nn = ctx.get_objective(check=False)
    ref = O.OpuOracle(d).step(x.astype(np.float64))
    assert nn == n - 3 == ref.N and abs(j - ref.J) / ref.J < 1e-3
    m = ctx.get_M(check=False).cpu().numpy()
    assert np.isfinite(m).all()
    st = ctx.get_stats()
    assert st.status == -7 and st.n_skipped == 3


def test_tc_matches_exact_mode_of_the_library():
    """Both arithmetic modes of the library on the same stream end at rotations with the same objective."""
    from paper_2605_10793_b200 import binding as B
    d, n = 256, 2048
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2)
    r0 = _dev(I.initial_rotation(w), "f32")
    out = {}
    for mode in ("exact", "tc"):
        ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode=mode)
        ctx.set_R(r0)
        for b in range(2):
            ctx.step(_dev(I.batch(w, b), "bf16"))
        ctx.update()
        ctx.step(_dev(I.batch(w, 2), "bf16"))
        out[mode] = ctx.get_objective()
    assert out["exact"][1] == out["tc"][1]
    assert abs(out["exact"][0] - out["tc"][0]) / out["exact"][0] < 1e-3


@pytest.mark.parametrize("layout,n,P,quant_bits,dtype", [("interleaved", 700, 5, 0, "bf16"), ("stacked", 256, 3, 0, "bf16"),
                                                         ("stacked", 1000, 151, 0, "bf16"), ("interleaved", 300, 4, 4, "bf16"),
                                                         ("stacked", 200, 3, 0, "f32")])
def test_batched_heads_fused_kernel(layout, n, P, quant_bits, dtype):
    """Per-head problems (d = 128) through the fused tensor-core kernel: each problem against an independent oracle run
    (objective, tie-aware cross-covariance with the sign decisions the kernel took, every differing sign inside the
    rounding band)."""
    d = 128
    w = I.scaled(I.WORKLOADS["c4b"], n=n, problems=P, dtype=dtype)
    xs = [I.batch(w, 0, problem=p) for p in range(P)]
    xs[0] = xs[0].copy()
    xs[0][3] = 0.0                                    # a skipped row in problem 0
    r0 = np.stack([I.initial_rotation(w, p) for p in range(P)])
    ctx = _ctx(d=d, n_max=n, in_dtype=dtype, batch=P, quant_bits=quant_bits)
    ctx.set_R(_dev(r0, "f32"))
    signs = _torch().zeros((P, n, d), dtype=_torch().int8, device="cuda")
    ctx.debug_capture_signs(signs)
    if layout == "interleaved":
        ctx.step_batched(_dev(np.concatenate(xs, axis=1), dtype), n, P * d, d)
    else:
        ctx.step_batched(_dev(np.concatenate(xs, axis=0), dtype), n, d, n * d)
    js, ns = ctx.get_objective()
    ms = ctx.get_M().cpu().numpy().astype(np.float64)
    ctx.update()
    st = ctx.get_stats()
    assert st.status == 0 and st.n_skipped == 1
    rs = ctx.get_R().cpu().numpy().astype(np.float64)
    check = range(P) if P <= 8 else [0, 1, P // 2, P - 2, P - 1]
    for p in check:
        x64 = (I.round_to_bf16(xs[p]) if dtype == "f32" else xs[p]).astype(np.float64)
        srep = step_parity(x64, r0[p].astype(np.float64), signs[p].cpu().numpy(), ms[p], js[p], ns[p], "tc", quant_bits)
        assert_step(srep, "tc", 2e-2)
        rep = update_parity(ms[p], rs[p])
        assert rep["orth"] <= T["orth"] and rep["gap"] <= T["gap"], (p, rep)
    j2, n2 = ctx.get_objective()
    assert not n2.any() and not ctx.get_M().any().item()


def test_tensor_core_rerun_is_bit_identical():
    """Same stream twice (steps + update, graph-replayed second update included): identical M, R and objective.
    The accumulate epilogue adds with L2 reductions, but every element of M receives exactly one addition per launch."""
    torch = _torch()
    d, n = 512, 1024
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2)
    xs = [_dev(I.batch(w, b), "bf16") for b in range(4)]
    outs = []
    for rep in range(2):
        ctx = _ctx(d=d, n_max=n, in_dtype="bf16")
        ctx.set_R(_dev(I.initial_rotation(w), "f32"))
        trace = []
        for cyc in range(3):
            for x in xs[:2] if cyc % 2 == 0 else xs[2:]:
                ctx.step(x)
            trace.append(ctx.get_M().clone())
            ctx.update()
            trace.append(ctx.get_R().clone())
        st = ctx.get_stats()
        assert st.status == 0 and st.updates == 3
        outs.append((trace, st.last_J))
    assert all(torch.equal(a, b) for a, b in zip(outs[0][0], outs[1][0])) and outs[0][1] == outs[1][1]


def test_zero_point_quant_mode_tc_and_batched():
    """Zero-point INT4 with clipping ratio 0.9 in tensor-core mode: one large problem and the fused per-head kernel."""
    d, n = 256, 1024
    w = I.scaled(I.WORKLOADS["c4a_zp"], d=d, n=n, n_outlier=2)
    x = I.batch(w, 0)
    ctx = _ctx(d=d, n_max=n, in_dtype="bf16", quant_bits=4, quant_mode="zp", clip_ratio=0.9)
    ctx.set_R(_dev(I.initial_rotation(w), "f32"))
    r = ctx.get_R().cpu().numpy().astype(np.float64)
    ctx.step(_dev(x, "bf16"))
    j, nn = ctx.get_objective()
    m = ctx.get_M().cpu().numpy().astype(np.float64)
    s = ctx.debug_get_signs(n).cpu().numpy()
    rep = step_parity(x.astype(np.float64), r, s, m, j, nn, "tc", 4, quant_mode="zp", clip_ratio=0.9)
    assert rep["N_equal"] and rep["J_rel"] <= T["J"], rep
    assert rep["M_rel_tie_aware"] <= T["M"] and rep["flips_outside_band"] == 0 and rep["flip_frac"] < 2e-2, rep
    _check_update(ctx, m, r)
    # per-head problems
    P, n2 = 4, 300
    wb = I.scaled(I.WORKLOADS["c4b"], n=n2, problems=P)
    xs = [I.batch(wb, 0, problem=p) for p in range(P)]
    r0 = np.stack([I.initial_rotation(wb, p) for p in range(P)])
    cb = _ctx(d=128, n_max=n2, in_dtype="bf16", batch=P, quant_bits=4, quant_mode="zp", clip_ratio=0.9)
    cb.set_R(_dev(r0, "f32"))
    signs = _torch().zeros((P, n2, 128), dtype=_torch().int8, device="cuda")
    cb.debug_capture_signs(signs)
    cb.step_batched(_dev(np.concatenate(xs, axis=0), "bf16"), n2, 128, n2 * 128)
    js, ns = cb.get_objective()
    ms = cb.get_M().cpu().numpy().astype(np.float64)
    for p in range(P):
        srep = step_parity(xs[p].astype(np.float64), r0[p].astype(np.float64), signs[p].cpu().numpy(), ms[p], js[p], ns[p],
                           "tc", 4, quant_mode="zp", clip_ratio=0.9)
        assert_step(srep, "tc", 2e-2)


@pytest.mark.parametrize("mode", ["tc", "exact"])
@pytest.mark.parametrize("spectrum", ["gauss", "log1e4", "near_orth", "spiky1e8", "below_bound"])
def test_update_on_synthetic_spectra(mode, spectrum):
    """The polar update on cross-covariances with prescribed singular values (loaded through conqur_set_M):
    well conditioned, log-spaced, already orthogonal, a few dominant directions over a 1e-8 tail, and a spectrum whose
    smallest singular value lies below the bound the schedule was planned for (the iteration must re-enter and
    still deliver)."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    d = 512
    rng = np.random.default_rng(5)
    u, _ = np.linalg.qr(rng.standard_normal((d, d)))
    v, _ = np.linalg.qr(rng.standard_normal((d, d)))
    kw = {}
    if spectrum == "gauss":
        m = rng.standard_normal((d, d))
    elif spectrum == "log1e4":
        m = (u * np.logspace(0, -4, d)) @ v.T
    elif spectrum == "near_orth":
        m = u @ v.T + 1e-3 * rng.standard_normal((d, d)) / np.sqrt(d)
    elif spectrum == "spiky1e8":
        m = (u * np.concatenate([np.ones(8), np.logspace(-3, -8, d - 8)])) @ v.T
    else:
        m = (u * np.concatenate([np.ones(8), np.logspace(-2, -6, d - 8)])) @ v.T
        kw = dict(ns_sigma_min_rel=1e-3, ns_max_steps=40)        # planned for a far better conditioned matrix
    m32 = m.astype(np.float32)
    ctx = B.Context(d=d, n_max=128, in_dtype="bf16", mode=mode, **kw)
    ctx.set_M(torch.from_numpy(m32).cuda(), 1.0, d)
    ctx.update()
    st = ctx.get_stats()
    assert st.status == 0, (st.status, st.ns_steps_used)
    r = ctx.get_R().cpu().numpy().astype(np.float64)
    rep = update_parity(m32.astype(np.float64), r)
    tol = TOL[mode]
    assert rep["orth"] <= tol["orth"], rep
    assert rep["gap"] <= tol["gap"], (rep["gap"], st.ns_steps_used)


@pytest.mark.parametrize("mode", ["tc", "exact"])
def test_update_recovers_when_the_learnt_lifting_count_is_far_too_short(mode):
    """The number of lifting steps an update starts with is learnt from the updates before it.  A context that has only
    seen well-conditioned cross-covariances (and has learnt a short plan) is then given one with singular values down
    to 1e-8 of the largest: the update must still deliver the polar factor (more steps, never a failure), and the
    plan must climb."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    d = 512
    rng = np.random.default_rng(9)
    u, _ = np.linalg.qr(rng.standard_normal((d, d)))
    v, _ = np.linalg.qr(rng.standard_normal((d, d)))
    easy = (u * np.linspace(1.0, 0.3, d)) @ v.T
    hard = (u * np.concatenate([np.ones(8), np.logspace(-3, -8, d - 8)])) @ v.T
    ctx = B.Context(d=d, n_max=128, in_dtype="bf16", mode=mode)
    plans, steps = [], []
    for k in range(6):
        ctx.set_M(torch.from_numpy(easy.astype(np.float32)).cuda(), 1.0, d)
        ctx.update()
        st = ctx.get_stats()
        assert st.status == 0
        plans.append(st.ns_lift_plan); steps.append(st.ns_steps_used)
    assert plans[-1] <= 3 and steps[-1] < steps[0], (plans, steps)          # learnt: a handful of steps suffice
    m32 = hard.astype(np.float32)
    ctx.set_M(torch.from_numpy(m32).cuda(), 1.0, d)
    ctx.update()
    st = ctx.get_stats()
    assert st.status == 0, (st.status, st.ns_steps_used)
    assert st.ns_steps_used > steps[-1] and st.ns_lift_plan > plans[-1], (st.ns_steps_used, st.ns_lift_plan)
    rep = update_parity(m32.astype(np.float64), ctx.get_R().cpu().numpy().astype(np.float64))
    assert rep["orth"] <= TOL[mode]["orth"] and rep["gap"] <= TOL[mode]["gap"], (rep["orth"], rep["gap"], st.ns_steps_used)


def test_lifting_count_comes_down_again_after_a_hard_update():
    """One badly conditioned cross-covariance must not fix the lifting count for good: the count goes up for it, and
    when the updates that follow need no extra steps it comes down again, one step at a time (every rotation on the
    way passes the orthogonality gate)."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    d = 256
    rng = np.random.default_rng(11)
    u, _ = np.linalg.qr(rng.standard_normal((d, d)))
    v, _ = np.linalg.qr(rng.standard_normal((d, d)))
    easy = torch.from_numpy(((u * np.linspace(1.0, 0.3, d)) @ v.T).astype(np.float32)).cuda()
    hard = torch.from_numpy(((u * np.concatenate([np.ones(8), np.logspace(-3, -7, d - 8)])) @ v.T).astype(np.float32)).cuda()
    ctx = B.Context(d=d, n_max=128, in_dtype="bf16", mode="tc")

    def run(m):
        ctx.set_M(m, 1.0, d)
        ctx.update()
        st = ctx.get_stats()
        assert st.status == 0 and st.orth_err <= TOL["tc"]["orth"], (st.status, st.orth_err)
        return st.ns_lift_plan, st.ns_steps_used

    low = [run(easy) for _ in range(6)][-1][0]
    peak = max(run(hard)[0] for _ in range(3))
    assert peak >= low + 3, (low, peak)
    plans = [run(easy)[0] for _ in range(24)]
    assert plans[-1] <= peak - 3 and all(b <= a for a, b in zip(plans, plans[1:])), (low, peak, plans)
