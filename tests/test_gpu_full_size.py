"""GPU parity at the full workload sizes, in the launch configuration bench.py times (tensor-core mode,
same Context arguments).  Where the oracle is too slow for a whole stream, a stated subset is checked:
whole steps where a float64 step takes about a second, sampled columns / properties where it does not."""
import numpy as np
import pytest

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I
from tests.parity_util import TOL, assert_step, effective_m, log_parity, step_parity, unit_roundoff, update_parity

pytestmark = pytest.mark.gpu
T = TOL["tc"]


def _torch():
    import torch
    return torch


def _bench_ctx(w, **kw):
    from paper_2605_10793_b200 import binding as B
    args = dict(d=w.d, n_max=w.n, in_dtype="bf16", mode="tc", quant_bits=w.quant_bits, prior_rel=w.prior_rel,
                quant_mode=w.quant_mode, clip_ratio=w.clip_ratio, ns_steps=w.ns_steps)
    if w.problems == 1:
        args["defer_batches"] = w.update_every          # as bench.py runs it: the products run once per update cycle
    args.update(kw)
    return B.Context(**args)


def _dev_bf16(x):
    torch = _torch()
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda().to(torch.bfloat16)


def _f64(t):
    return t.cpu().numpy().astype(np.float64)


def _full_step_check(ctx, w, x, before):
    r = _f64(ctx.get_R())
    ctx.step(_dev_bf16(x))
    j, n = ctx.get_objective()
    m = _f64(ctx.get_M())
    s = ctx.debug_get_signs(x.shape[0]).cpu().numpy()
    mb, jb, nb = before if before is not None else (None, 0.0, 0)
    rep = step_parity(x.astype(np.float64), r, s, m, j, n, "tc", w.quant_bits, mb, jb, nb, w.quant_mode, w.clip_ratio)
    log_parity(w.name, "tc", f"cycle 1 step ({n // w.n} of {w.update_every})", rep)
    assert_step(rep, "tc", 2e-2)
    return rep, (m, j, n), r


def test_c2_one_update_cycle_headline_workload():
    """d = 4096 as bench.py times it: 8 batches of 2048 tokens queued and run through the two products in one go,
    then the polar update.  All 16384 rows against the oracle (objective, tie-aware cross-covariance, every differing
    sign inside the rounding band); the update against the SVD polar factor of the library's own M."""
    w = I.WORKLOADS["c2"]
    ctx = _bench_ctx(w)
    torch = _torch()
    r0 = I.initial_rotation(w)
    ctx.set_R(torch.from_numpy(r0).cuda())
    r = _f64(ctx.get_R())
    xs = [I.batch(w, b) for b in range(w.update_every)]
    for x in xs:
        ctx.step(_dev_bf16(x))
    j, n = ctx.get_objective()
    m = _f64(ctx.get_M())
    rows = w.update_every * w.n
    s = ctx.debug_get_signs(rows).cpu().numpy()
    rep = step_parity(np.concatenate(xs, axis=0).astype(np.float64), r, s, m, j, n, "tc")
    log_parity(w.name, "tc", f"cycle 1, all {w.update_every} batches in one run of the products", rep)
    assert n == rows
    assert_step(rep, "tc", 2e-2)
    del s, rep
    ctx.update()
    st = ctx.get_stats()
    assert st.status == 0 and st.ns_steps_used <= 24, (st.status, st.ns_steps_used)
    r_new = _f64(ctx.get_R())
    rep = update_parity(m, r_new)
    log_parity(w.name, "tc", "cycle 1 update", rep, ns_steps_used=int(st.ns_steps_used))
    assert rep["orth"] <= T["orth"], rep
    assert rep["gap"] <= T["gap"], rep
    # ascent on the statistics the update was computed from: <R_new, M> >= <R_old, M> = J
    assert np.sum(r_new * m) >= j * (1.0 - 1e-3)


def test_c4a_int4_fake_quant_step_at_d4096():
    w = I.WORKLOADS["c4a"]
    ctx = _bench_ctx(w)
    ctx.set_R(_torch().from_numpy(I.initial_rotation(w)).cuda())
    _full_step_check(ctx, w, I.batch(w, 0), None)


def test_c4a_zero_point_int4_clip09_step_at_d4096():
    """The quantiser the paper's evaluation uses (zero-point, clipping ratio 0.9) at the headline size."""
    w = I.WORKLOADS["c4a_zp"]
    ctx = _bench_ctx(w)
    ctx.set_R(_torch().from_numpy(I.initial_rotation(w)).cuda())
    _full_step_check(ctx, w, I.batch(w, 0), None)


def test_c1_fewer_tokens_than_dimensions_proximal_update_at_d3072():
    w = I.WORKLOADS["c1"]
    ctx = _bench_ctx(w)
    ctx.set_R(_torch().from_numpy(I.initial_rotation(w)).cuda())
    rep, (m, j, n), r = _full_step_check(ctx, w, I.batch(w, 0), None)
    ctx.update()
    st = ctx.get_stats()
    assert st.status == 0
    rep = update_parity(effective_m(m, r, w.prior_rel), _f64(ctx.get_R()))
    log_parity(w.name, "tc", "cycle 1 update (proximal)", rep, ns_steps_used=int(st.ns_steps_used))
    assert rep["orth"] <= T["orth"] and rep["gap"] <= T["gap"], rep


def test_c4b_1024_heads_sampled_problems():
    """1024 independent d = 128 problems of 4096 tokens in one batched call (64 distinct seeded problems repeated
    16 times, generation being the slow part); sampled problems against independent oracle runs, the cross-covariance
    tie-aware with the sign decisions the fused kernel took."""
    w = I.WORKLOADS["c4b"]
    torch = _torch()
    P, distinct = w.problems, 64
    xs = [I.batch(w, 0, problem=p) for p in range(distinct)]
    r0s = [I.initial_rotation(w, p) for p in range(distinct)]
    x_all = _dev_bf16(np.concatenate(xs, axis=0)).repeat(P // distinct, 1)
    r_all = torch.from_numpy(np.stack(r0s)).cuda().repeat(P // distinct, 1, 1).contiguous()
    ctx = _bench_ctx(w, batch=P)
    ctx.set_R(r_all)
    signs = torch.zeros((P, w.n, w.d), dtype=torch.int8, device="cuda")
    ctx.debug_capture_signs(signs)
    ctx.step_batched(x_all, w.n, w.d, w.n * w.d)
    ctx.debug_capture_signs(None)
    js, ns = ctx.get_objective()
    ms = _f64(ctx.get_M())
    ctx.update()
    st = ctx.get_stats()
    assert st.status == 0
    rs = _f64(ctx.get_R())
    for p in (0, 17, 63, 64 + 5, 511, 1023):
        q = p % distinct
        srep = step_parity(xs[q].astype(np.float64), r0s[q].astype(np.float64), signs[p].cpu().numpy(), ms[p], js[p], ns[p],
                           "tc")
        log_parity(w.name, "tc", f"problem {p} step", srep)
        assert_step(srep, "tc", 2e-2)
        rep = update_parity(ms[p], rs[p])
        log_parity(w.name, "tc", f"problem {p} update", rep)
        assert rep["orth"] <= T["orth"] and rep["gap"] <= T["gap"], (p, rep)
    # identical problems give bit-identical results wherever they ran
    assert np.array_equal(ms[5], ms[64 + 5]) and np.array_equal(rs[5], rs[64 * 7 + 5])


def test_fold_hadamard_and_algorithm1_legs_at_bench_sizes():
    """The three extra bench legs at the sizes bench.py times them, on outputs the oracle can afford:
    weight folding R^T W with W 4096 x 14336 (tensor-core mode) on sampled output columns; the Walsh-Hadamard
    transform of 32768 x 4096 bf16 rows on sampled rows; block 0 of the 8B-class Algorithm-1 mini-batch (4096 tokens:
    two residual-stream steps at d = 4096 and the 32 head problems) on objective, token counts and sampled heads."""
    torch = _torch()
    from paper_2605_10793_b200 import algorithm1 as A1
    from paper_2605_10793_b200 import binding as B
    rng = np.random.default_rng(11)
    # --- fold
    d, cols = 4096, 14336
    w = I.random_weight(1, d, cols)
    q, _ = np.linalg.qr(np.random.default_rng(2).standard_normal((d, d)))
    r = q.astype(np.float32)
    out = B.conqur_fold_weight(torch.from_numpy(w).cuda(), torch.from_numpy(r).cuda(), "output", "tc").cpu().numpy()
    sel = rng.choice(cols, size=48, replace=False)
    ref = r.astype(np.float64).T @ w[:, sel].astype(np.float64)
    assert np.linalg.norm(out[:, sel] - ref) / np.linalg.norm(ref) <= 2e-5
    mag = np.abs(r.astype(np.float64)).T @ np.abs(w[:, sel].astype(np.float64))
    assert np.max(np.abs(out[:, sel] - ref) / mag) <= 8e-5
    del out
    # --- Hadamard
    n = 32768
    x = torch.randn(n, d, device="cuda").to(torch.bfloat16)
    y = B.conqur_hadamard_rows(x)
    assert B.conqur_hadamard_status() == 0
    rows = rng.choice(n, size=32, replace=False)
    xs = x[rows].float().cpu().numpy().astype(np.float64)
    ref = O.hadamard_rows(xs)
    got = y[rows].float().cpu().numpy().astype(np.float64)
    bound = np.log2(d) * 2.0 ** -24 * np.linalg.norm(xs, axis=1, keepdims=True) + 2.0 ** -8 * np.abs(ref)
    assert (np.abs(got - ref) <= bound).all()
    del x, y
    # --- Algorithm 1, block 0 of a mini-batch
    a = I.SITE_MODELS["a1_8b"]
    cal = A1.Calibrator(a.d, a.n_heads, a.d_head, a.n_layers, a.n, in_dtype="bf16", mode="tc")
    r1, r2 = I.site_initial_rotations(a)
    cal.set_rotations(torch.from_numpy(r1).cuda(), torch.from_numpy(r2).cuda())
    s = I.site_activations(a, 0, 0)
    dev = {k: torch.from_numpy(v).cuda().to(torch.bfloat16) for k, v in s.items()}
    signs = torch.zeros((a.n_heads, a.n, a.d_head), dtype=torch.int8, device="cuda")
    cal.ctx2.debug_capture_signs(signs)
    cal.collect(0, dev["attn"], dev["mlp"], dev["o"])
    cal.ctx2.debug_capture_signs(None)
    j1, n1 = cal.ctx1.get_objective()
    j_ref = 0.0
    for k in ("attn", "mlp"):
        xt, used = O.normalise_rows(s[k].astype(np.float64))
        j_ref += np.abs(xt @ r1.astype(np.float64)).sum() / np.sqrt(a.d)
        assert used.all()
    assert n1 == 2 * a.n and abs(j1 - j_ref) / j_ref <= T["J"]
    j2, n2 = cal.ctx2.get_objective()
    m2 = cal.ctx2.get_M().cpu().numpy().astype(np.float64)
    assert (n2[:a.n_heads] == a.n).all() and not n2[a.n_heads:].any()          # only block 0's problems were fed
    for h in (0, 13, 31):
        srep = step_parity(s["o"][:, h * a.d_head:(h + 1) * a.d_head].astype(np.float64), r2[0, h].astype(np.float64),
                           signs[h].cpu().numpy(), m2[h], j2[h], n2[h], "tc")
        assert_step(srep, "tc", 2e-2)
    assert B.conqur_update(cal.ctx2.h) == -4                                    # the other blocks' problems have no rows yet
    cal.close()
