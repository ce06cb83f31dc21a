"""Pins for the float64 oracle: what the paper and the mathematics fix.

Each test checks the oracle against something other than itself: an identity
of Sections 3.1-3.3 / Appendix B, a closed form, brute force on tiny inputs,
or an independent route to the same object.  CPU only.
"""
import os

import numpy as np
import pytest
import scipy.linalg

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")) as fh:
    for line in fh:
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            GOLD[k] = float(v)


def _x(seed, n, d, outliers=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, d))
    if outliers:
        x[:, : max(1, d // 32)] *= 50.0
    return x


def _rand_orth(seed, d):
    q, r = np.linalg.qr(np.random.default_rng(seed).standard_normal((d, d)))
    return q * np.sign(np.diag(r))[None, :]


# ---------------------------------------------------------------- normalisation


def test_rows_have_unit_norm_and_scale_invariance():
    x = _x(1, 200, 32)
    xt, used = O.normalise_rows(x)
    assert used.all()
    assert np.allclose(np.linalg.norm(xt, axis=1), 1.0, atol=1e-15)
    # a positive per-row scale changes nothing downstream (Eq. 1 normalises it away)
    scale = np.exp(0.5 * np.random.default_rng(2).standard_normal((200, 1)))
    r = _rand_orth(3, 32)
    a = O.OpuOracle(32, r).step(x)
    b = O.OpuOracle(32, r).step(x * scale)
    assert np.allclose(a.M, b.M, atol=1e-13) and abs(a.J - b.J) < 1e-11


def test_zero_and_nonfinite_rows_are_skipped():
    x = _x(4, 10, 8)
    x[3] = 0.0
    x[7, 2] = np.inf
    x[8, 1] = np.nan
    orc = O.OpuOracle(8).step(x)
    keep = [0, 1, 2, 4, 5, 6, 9]
    ref = O.OpuOracle(8).step(x[keep])
    assert orc.N == 7 and orc.n_skipped == 3
    assert np.allclose(orc.M, ref.M, atol=1e-15) and np.isclose(orc.J, ref.J)


# ---------------------------------------------------------------- target (Eq. 2)


def test_target_is_a_unit_norm_hypercube_vertex():
    y = _x(5, 50, 64)
    z = O.corner_target(y)
    assert np.allclose(np.abs(z), 1.0 / 8.0)
    assert np.allclose(np.linalg.norm(z, axis=1), 1.0, atol=1e-15)
    assert np.all(np.sign(z) == np.sign(y))


def test_sign_of_zero_is_zero_one_hot_rows():
    d = 16
    k = np.array([0, 3, 3, 7, 15, 15, 15])
    x = np.zeros((k.size, d))
    x[np.arange(k.size), k] = np.array([2.0, -1.0, 4.0, 0.5, 1.0, 3.0, -2.0])
    orc = O.OpuOracle(d).step(x)          # R = I: y = +-e_k, target +-e_k/sqrt(d)
    counts = np.bincount(k, minlength=d).astype(float)
    assert np.allclose(orc.M, np.diag(counts) / np.sqrt(d), atol=1e-15)
    assert np.isclose(orc.J, k.size / np.sqrt(d))            # ||e_k||_1 = 1: the lower bound of Section 3.2
    # with the other reading (sign(0)=+1) M would have off-diagonal mass: rule it out
    assert np.count_nonzero(orc.M - np.diag(np.diag(orc.M))) == 0


def test_one_hot_rows_under_hadamard_are_corners():
    d = 32
    h = I.hadamard_pm1(d).astype(np.float64) / np.sqrt(d)
    x = np.eye(d)[[1, 5, 9, 30]] * np.array([[3.0], [-2.0], [0.1], [7.0]])
    orc = O.OpuOracle(d, h).step(x)
    assert np.isclose(orc.objective_per_token(), 1.0, atol=1e-14)   # upper bound attained (Section 3.2)
    assert abs(orc.corner_distance()) < 1e-12


# ---------------------------------------------------------------- objective (Section 3.2)


@pytest.mark.parametrize("d,n", [(8, 40), (64, 300), (128, 257)])
def test_corner_distance_identity_and_bounds(d, n):
    x = _x(6 + d, n, d)
    r = _rand_orth(7, d)
    orc = O.OpuOracle(d, r).step(x)
    lhs = O.corner_distance_direct(x, r)            # sum ||R x~ - z||^2, literally
    assert np.isclose(lhs, 2 * orc.N - 2 * orc.J, rtol=1e-12)
    assert 1.0 / np.sqrt(d) - 1e-12 <= orc.objective_per_token() <= 1.0 + 1e-12


def test_objective_equals_inner_product_with_cross_covariance():
    # J = sum_i <y_i, c_i> = tr(R^T X~^T C) = <R, M>: ties both products and the reduction
    d = 48
    x = _x(8, 500, d)
    r = _rand_orth(9, d)
    orc = O.OpuOracle(d, r).step(x)
    assert np.isclose(orc.J, O.procrustes_value(r, orc.M), rtol=1e-12)
    # a transposed cross-covariance would break this
    assert not np.isclose(orc.J, O.procrustes_value(r, orc.M.T), rtol=1e-6)


def test_cross_covariance_elementwise_brute_force():
    d, n = 5, 7
    x = _x(10, n, d, outliers=False)
    r = _rand_orth(11, d)
    m = np.zeros((d, d))
    j = 0.0
    for i in range(n):
        nrm = np.sqrt(sum(x[i, k] ** 2 for k in range(d)))
        xt = [x[i, k] / nrm for k in range(d)]
        y = [sum(xt[k] * r[k, c] for k in range(d)) for c in range(d)]
        for c in range(d):
            s = int(y[c] > 0) - int(y[c] < 0)
            j += abs(y[c]) / np.sqrt(d)
            for a in range(d):
                m[a, c] += xt[a] * s / np.sqrt(d)
    orc = O.OpuOracle(d, r).step(x)
    assert np.allclose(orc.M, m, atol=1e-14) and np.isclose(orc.J, j, rtol=1e-13)


def test_accumulation_over_batches_equals_one_big_batch():
    d = 24
    x = _x(12, 300, d)
    r = _rand_orth(13, d)
    whole = O.OpuOracle(d, r).step(x)
    parts = O.OpuOracle(d, r)
    for blk in np.array_split(x, 7):
        parts.step(blk)
    assert np.allclose(whole.M, parts.M, atol=1e-13) and np.isclose(whole.J, parts.J) and whole.N == parts.N


# ---------------------------------------------------------------- polar (Section 3.3)


@pytest.mark.parametrize("d", [2, 3, 16, 128])
def test_polar_is_orthogonal_and_optimal(d):
    m = np.random.default_rng(20 + d).standard_normal((d, d)) @ np.diag(np.logspace(0, -4, d))
    r, s = O.polar_svd(m)
    assert np.max(np.abs(r.T @ r - np.eye(d))) < 1e-12
    assert np.isclose(np.trace(r.T @ m), s.sum(), rtol=1e-12)      # value = nuclear norm
    h = r.T @ m
    assert np.allclose(h, h.T, atol=1e-12 * s[0])                    # R^T M symmetric ...
    assert np.linalg.eigvalsh((h + h.T) / 2).min() > -1e-12 * s[0]   # ... and PSD
    for k in range(20):                                             # no orthogonal matrix does better
        q = _rand_orth(100 + k, d)
        assert np.trace(q.T @ m) <= s.sum() + 1e-12


def test_procrustes_optimum_closed_forms_and_bound():
    """tr(R^T M) at the optimum: d = 2 closed form (the better of the best rotation and the best reflection),
    a diagonal matrix (sum of |entries|), an orthogonal matrix (d), the trace of (M^T M)^(1/2) by an
    eigendecomposition, and the fact that no orthogonal matrix exceeds it while polar_svd's factor attains it."""
    rng = np.random.default_rng(41)
    m = rng.standard_normal((2, 2)) * np.array([[3.0, 0.5]])
    rot = np.hypot(m[0, 0] + m[1, 1], m[0, 1] - m[1, 0])
    ref = np.hypot(m[0, 0] - m[1, 1], m[0, 1] + m[1, 0])
    assert np.isclose(O.procrustes_optimum(m), max(rot, ref), rtol=1e-12)
    dg = np.array([3.0, -2.0, 0.5, -0.25])
    assert np.isclose(O.procrustes_optimum(np.diag(dg)), 5.75, rtol=1e-13)
    q = _rand_orth(7, 24)
    assert np.isclose(O.procrustes_optimum(q), 24.0, rtol=1e-12)
    a = rng.standard_normal((40, 40)) @ np.diag(np.logspace(0, -5, 40))
    w = np.linalg.eigvalsh(a.T @ a)
    assert np.isclose(O.procrustes_optimum(a), np.sqrt(np.clip(w, 0.0, None)).sum(), rtol=1e-7)
    r, _ = O.polar_svd(a)
    assert np.isclose(np.trace(r.T @ a), O.procrustes_optimum(a), rtol=1e-12)
    for k in range(10):
        assert np.trace(_rand_orth(200 + k, 40).T @ a) <= O.procrustes_optimum(a) + 1e-12


@pytest.mark.parametrize("d", [4, 32, 96])
def test_polar_against_independent_routes(d):
    m = np.random.default_rng(30 + d).standard_normal((d, d))
    r, _ = O.polar_svd(m)
    # route 2: M (M^T M)^(-1/2) by a symmetric eigendecomposition
    w, v = np.linalg.eigh(m.T @ m)
    r2 = m @ (v @ np.diag(w ** -0.5) @ v.T)
    assert np.allclose(r, r2, atol=1e-9)
    # route 3: Newton iteration X <- (X + X^-T)/2 (converges to the polar factor)
    xk = m.copy()
    for _ in range(60):
        xk = 0.5 * (xk + np.linalg.inv(xk).T)
    assert np.allclose(r, xk, atol=1e-10)
    # route 4: a library polar decomposition
    u, _p = scipy.linalg.polar(m)
    assert np.allclose(r, u, atol=1e-10)


def test_polar_d2_closed_form_and_angle_grid():
    rng = np.random.default_rng(40)
    for trial in range(6):
        m = rng.standard_normal((2, 2)) * np.array([[5.0, 1.0]])
        r, s = O.polar_svd(m)
        rot = np.hypot(m[0, 0] + m[1, 1], m[0, 1] - m[1, 0])     # best proper rotation
        ref = np.hypot(m[0, 0] - m[1, 1], m[0, 1] + m[1, 0])     # best reflection
        assert np.isclose(max(rot, ref), s.sum(), rtol=1e-12)
        th = np.linspace(0.0, 2 * np.pi, 100_000, endpoint=False)
        c, sn = np.cos(th), np.sin(th)
        # rotations [[c,-s],[s,c]] and reflections [[c,s],[s,-c]]: tr(R^T M) on the grid
        val_rot = c * (m[0, 0] + m[1, 1]) + sn * (m[1, 0] - m[0, 1])
        val_ref = c * (m[0, 0] - m[1, 1]) + sn * (m[0, 1] + m[1, 0])
        if val_rot.max() >= val_ref.max():
            k = val_rot.argmax()
            best = np.array([[c[k], -sn[k]], [sn[k], c[k]]])
            best_val = val_rot[k]
        else:
            k = val_ref.argmax()
            best = np.array([[c[k], sn[k]], [sn[k], -c[k]]])
            best_val = val_ref[k]
        assert abs(best_val - np.trace(r.T @ m)) <= 1e-8 * s.sum()
        assert np.max(np.abs(best - r)) < 2 * (2 * np.pi / th.size)


def test_d2_workload_full_opu_matches_grid_search():
    # the Procrustes subproblem min_R ||X~ R - C||_F^2 (Section 3.3), literally, over a fine grid of O(2)
    w = I.WORKLOADS["c0_d2"]
    x = I.batch(w, 0).astype(np.float64)
    th = np.linspace(0.0, 2 * np.pi, 100_000, endpoint=False)
    c, sn = np.cos(th), np.sin(th)
    rots = np.stack([np.stack([c, -sn], -1), np.stack([sn, c], -1)], -2)
    refl = np.stack([np.stack([c, sn], -1), np.stack([sn, -c], -1)], -2)
    grid = np.concatenate([rots, refl], axis=0)               # (200000, 2, 2)
    for r0 in (np.eye(2), _rand_orth(41, 2)):
        orc = O.OpuOracle(2, r0).step(x)
        xt, _ = O.normalise_rows(x)
        cmat = O.corner_target(xt @ r0)
        orc.update()
        dist = np.sum((np.einsum("na,kab->knb", xt, grid) - cmat[None]) ** 2, axis=(1, 2))
        k = dist.argmin()
        dist_oracle = np.sum((xt @ orc.R - cmat) ** 2)
        assert dist_oracle <= dist[k] + 1e-12
        assert dist[k] - dist_oracle < 1e-6
        assert np.max(np.abs(grid[k] - orc.R)) < 2 * (2 * np.pi / th.size)


# ---------------------------------------------------------------- alternation (Sections 3.3, App. B)


def test_alternation_is_monotone_on_a_fixed_batch_c0():
    w = I.WORKLOADS["c0"]
    x = I.batch(w, 0).astype(np.float64)
    orc = O.OpuOracle(w.d, I.initial_rotation(w).astype(np.float64))
    prev = -np.inf
    js = []
    for it in range(10):
        orc.step(x)
        j_t, m_t, r_t = orc.J, orc.M.copy(), orc.R.copy()
        assert np.isclose(j_t, O.procrustes_value(r_t, m_t), rtol=1e-12)
        orc.update()
        nuc = orc.last_sigma.sum()
        assert np.isclose(O.procrustes_value(orc.R, m_t), nuc, rtol=1e-12)
        assert j_t <= nuc * (1 + 1e-12)            # J(R_t) = <R_t,M_t> <= ||M_t||_*
        assert j_t >= prev * (1 - 1e-12)           # objective never decreases
        prev = j_t
        js.append(j_t / x.shape[0])
        assert np.max(np.abs(orc.R.T @ orc.R - np.eye(w.d))) < 1e-12
    # next step's J at the new R is at least the Procrustes value of the old signs
    orc.step(x)
    assert orc.J >= nuc * (1 - 1e-12)
    assert js[-1] > js[0] + 0.05                   # and it actually moves towards the corners


def test_a_transposed_update_would_break_monotonicity():
    # planted mistake: using polar(M^T) (column/row convention mix-up) is caught by the chain above
    w = I.WORKLOADS["c0"]
    x = I.batch(w, 0).astype(np.float64)[:512]
    r0 = _rand_orth(50, w.d)
    good = O.OpuOracle(w.d, r0).step(x)
    j0, m0 = good.J, good.M.copy()
    bad_r, _ = O.polar_svd(m0.T)
    j_bad = O.OpuOracle(w.d, bad_r).step(x).J
    good.update()
    j_good = O.OpuOracle(w.d, good.R).step(x).J
    assert j_good >= j0 and j_bad < j_good - 1e-3 * j0


def test_proximal_update_for_rank_deficient_statistics():
    d, n = 32, 12                                # fewer tokens than dimensions
    x = _x(51, n, d)
    r0 = _rand_orth(52, d)
    with pytest.raises(np.linalg.LinAlgError):
        O.OpuOracle(d, r0).step(x).update()
    orc = O.OpuOracle(d, r0, prior_rel=1e-2).step(x)
    m, j = orc.M.copy(), orc.J
    orc.update()
    assert np.max(np.abs(orc.R.T @ orc.R - np.eye(d))) < 1e-12
    assert O.procrustes_value(orc.R, m) >= j * (1 - 1e-12)     # still an ascent step on the batch


# ---------------------------------------------------------------- fake-quant (Appendix B)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_fake_quant_error_bounds(bits):
    y = _x(60, 100, 64)
    qy, q, delta = O.fake_quant_sym(y, bits)
    lv = 2 ** (bits - 1) - 1
    assert np.all(np.abs(qy - y) <= delta[:, None] / 2 * (1 + 1e-12))
    assert np.all(np.sum((qy - y) ** 2, axis=1) <= 64 * delta ** 2 / 4 * (1 + 1e-12))
    assert np.all(np.abs(q) <= lv) and np.all(q == np.rint(q))
    assert np.allclose(delta, np.abs(y).max(axis=1) / lv)


def test_fake_quant_corners_fixed_points_and_printed_bounds():
    d = 4096
    s = np.where(np.random.default_rng(61).random(d) < 0.5, -1.0, 1.0)
    corner = s / np.sqrt(d)
    qy, q, delta = O.fake_quant_sym(corner[None, :], 4)
    assert np.all(np.abs(q) == 7) and np.allclose(qy, corner, rtol=1e-15)
    # printed constants of Appendix B
    assert np.isclose(corner.max() - corner.min(), GOLD["corner_signed_range_d4096"])
    assert 1.0 - np.sqrt(2.0 / d) > GOLD["corner_range_recovered_min_d4096"]
    bound_corner = d * delta[0] ** 2 / 4
    assert np.isclose(bound_corner, GOLD["corner_quant_bound_b4"], rtol=1e-12)
    pole = np.zeros(d)
    pole[3] = 1.0
    _, _, dp = O.fake_quant_sym(pole[None, :], 4)
    assert np.isclose((d * dp[0] ** 2 / 4) / bound_corner, GOLD["pole_over_corner_bound_ratio_d4096"])


def test_fake_quant_dead_zone_identity_and_brute_force():
    y = _x(62, 30, 16)
    y[0, 5] = 0.0
    qy, q, delta = O.fake_quant_sym(y, 4)
    # half-even rounding: |y| > Delta/2 keeps its sign, |y| <= Delta/2 goes to zero
    assert np.array_equal(O.sgn(q), np.sign(y) * (np.abs(y) > delta[:, None] / 2))
    # exact tie at Delta/2 -> 0 (half to even)
    row = np.array([[7.0, 0.5, -0.5, 1.5, -2.5, 0.0, 3.2, -7.0]])
    _, qt, dt = O.fake_quant_sym(row, 4)
    assert dt[0] == 1.0 and list(qt[0]) == [7, 0, -0, 2, -2, 0, 3, -7]
    for i in range(y.shape[0]):
        dl = max(abs(v) for v in y[i]) / 7
        for c in range(y.shape[1]):
            v = y[i, c] / dl
            f = np.floor(v)
            r = f if v - f < 0.5 else f + 1 if v - f > 0.5 else (f if f % 2 == 0 else f + 1)
            assert q[i, c] == min(7, max(-7, r))


def test_many_bits_reproduce_plain_signs_and_objective():
    d = 32
    x = _x(63, 200, d)
    r = _rand_orth(64, d)
    plain = O.OpuOracle(d, r).step(x)
    fine = O.OpuOracle(d, r, quant_bits=24).step(x)
    assert np.mean(plain.last_S != fine.last_S) < 1e-4
    assert np.isclose(plain.J, fine.J, rtol=1e-6)


def test_quant_mode_statistics_brute_force():
    d, n = 6, 9
    x = _x(65, n, d, outliers=False)
    r = _rand_orth(66, d)
    orc = O.OpuOracle(d, r, quant_bits=4).step(x)
    m = np.zeros((d, d))
    j = 0.0
    for i in range(n):
        xt = x[i] / np.linalg.norm(x[i])
        y = xt @ r
        dl = np.abs(y).max() / 7
        for c in range(d):
            q = min(7.0, max(-7.0, float(np.rint(y[c] / dl))))
            j += dl * abs(q) / np.sqrt(d)
            m[:, c] += xt * np.sign(q) / np.sqrt(d)
    assert np.allclose(orc.M, m, atol=1e-14) and np.isclose(orc.J, j, rtol=1e-13)


# ---------------------------------------------------------------- batched / streams / Appendix A


def test_batched_equals_independent_runs():
    d = 16
    xs = [_x(70 + p, 50, d, outliers=False) for p in range(4)]
    rs = [_rand_orth(80 + p, d) for p in range(4)]
    out = O.run_batched(d, xs, rs)
    for p in range(4):
        solo = O.OpuOracle(d, rs[p]).step(xs[p])
        m = solo.M.copy()
        solo.update()
        assert np.array_equal(out[p]["R"], solo.R) and np.array_equal(out[p]["M"], m)


def test_stream_update_cadence_and_reset():
    d = 16
    batches = [_x(90 + b, 64, d) for b in range(6)]
    orc, log = O.run_stream(d, batches, np.eye(d), update_every=3)
    assert len(log) == 2 and log[0]["N"] == 192 and orc.N == 0 and not orc.M.any()
    # the second update only saw batches 3..5 at the rotation produced by the first
    first = O.OpuOracle(d, np.eye(d))
    for b in range(3):
        first.step(batches[b])
    first.update()
    for b in range(3, 6):
        first.step(batches[b])
    assert np.isclose(first.J, log[1]["J"], rtol=1e-14)


def test_rotation_invariance_of_a_linear_layer():
    # Appendix A: X W^T = (X R)(R^T W^T)
    d = 24
    x = _x(95, 40, d)
    wgt = np.random.default_rng(96).standard_normal((10, d))
    r, _ = O.polar_svd(np.random.default_rng(97).standard_normal((d, d)))
    assert np.allclose(x @ wgt.T, (x @ r) @ (r.T @ wgt.T), atol=1e-10)


def test_reflections_are_allowed():
    # R in O(d), not SO(d): the update may have determinant -1 and is not corrected
    m = np.diag([3.0, 2.0, -1.0])
    r, _ = O.polar_svd(m)
    assert np.isclose(np.linalg.det(r), -1.0) and np.allclose(r, np.diag([1.0, 1.0, -1.0]))


# ---- zero-point quantiser (Appendix B, Q_zp; clipping ratio of Appendix C)

@pytest.mark.parametrize("bits", [2, 4, 8])
def test_zero_point_quantiser_error_bounds_and_grid(bits):
    rng = np.random.default_rng(40 + bits)
    y = rng.standard_normal((50, 64)) * np.exp(rng.standard_normal((50, 1))) + 0.3 * rng.standard_normal((50, 1))
    qy, k, delta = O.fake_quant_zp(y, bits)
    levels = 2 ** bits - 1
    assert np.allclose(delta, (y.max(axis=1) - y.min(axis=1)) / levels)
    assert np.all(np.abs(qy - y) <= delta[:, None] / 2 + 1e-12)                    # rounding error <= Delta/2 per coordinate
    assert np.all(np.sum((qy - y) ** 2, axis=1) <= y.shape[1] * delta ** 2 / 4 + 1e-12)   # the printed MSE bound
    assert np.all(y.max(axis=1) - y.min(axis=1) <= 2 * np.abs(y).max(axis=1) + 1e-15)     # range <= 2 ||x||_inf
    assert np.all(k.max(axis=1) - k.min(axis=1) == levels)                         # min and max sit on the two grid ends
    assert np.all(k == np.rint(k))                                                 # integer codes


def test_zero_point_quantiser_brute_force_and_clipping():
    rng = np.random.default_rng(7)
    y = rng.standard_normal((6, 17))
    for clip in (1.0, 0.9):
        qy, k, delta = O.fake_quant_zp(y, 4, clip)
        for i in range(y.shape[0]):
            lo, hi = clip * min(y[i]), clip * max(y[i])
            dl = (hi - lo) / 15.0
            z = -int(np.rint(lo / dl))
            for j in range(y.shape[1]):
                q = min(max(int(np.rint(y[i, j] / dl)) + z, 0), 15)
                assert q - z == k[i, j] and abs(dl * (q - z) - qy[i, j]) < 1e-15
    # with a clipping ratio the extremes saturate at the ends of the grid and lose more than Delta/2
    qy, k, delta = O.fake_quant_zp(y, 4, 0.9)
    imax = np.argmax(y, axis=1)
    assert np.allclose(qy[np.arange(6), imax], 0.9 * y.max(axis=1), atol=delta.max())      # clamped to the top of the clipped range
    assert np.all(y[np.arange(6), imax] - qy[np.arange(6), imax] > 0) and np.all(k.max(axis=1) - k.min(axis=1) == 15)
    # a constant row quantises to zero; many bits reproduce the plain signs
    assert not O.fake_quant_zp(np.full((1, 8), 0.3), 4)[0].any()
    qy16, k16, _ = O.fake_quant_zp(y, 16)
    assert np.array_equal(O.sgn(k16), O.sgn(y)) and np.allclose(qy16, y, atol=1e-4)


def test_zero_point_mode_statistics_and_shift_sensitivity():
    """OPU statistics in zero-point mode: brute force on a small case; and, unlike the symmetric quantiser, the
    dead zone follows the signed range (max - min)/(2^b - 1), not ||y||_inf."""
    d, n = 8, 30
    rng = np.random.default_rng(11)
    x = rng.standard_normal((n, d))
    r = np.linalg.qr(rng.standard_normal((d, d)))[0]
    orc = O.OpuOracle(d, r, quant_bits=4, quant_mode="zp", clip_ratio=0.9).step(x)
    m = np.zeros((d, d)); j = 0.0
    for i in range(n):
        xt = x[i] / np.linalg.norm(x[i])
        y = xt @ r
        lo, hi = 0.9 * y.min(), 0.9 * y.max()
        dl = (hi - lo) / 15.0
        z = -np.rint(lo / dl)
        k = np.clip(np.rint(y / dl) + z, 0, 15) - z
        j += dl * np.abs(k).sum() / np.sqrt(d)
        m += np.outer(xt, np.sign(k) / np.sqrt(d))
    assert abs(orc.J - j) < 1e-12 and np.allclose(orc.M, m, atol=1e-14) and orc.N == n
    # scale invariance of the codes: a positive row scale changes nothing
    orc2 = O.OpuOracle(d, r, quant_bits=4, quant_mode="zp", clip_ratio=0.9).step(x * np.exp(rng.standard_normal((n, 1))))
    assert abs(orc2.J - orc.J) < 1e-12 and np.allclose(orc2.M, orc.M, atol=1e-13)


# ---- diagnostics of Section 4 (participation ratio, dynamic-range ratio, relative quantisation error)

def test_participation_ratio_and_dynamic_range_bounds_and_extremes():
    d = 64
    rng = np.random.default_rng(21)
    x = rng.standard_normal((200, d)) * np.exp(rng.standard_normal((200, 1)))
    spr, srho, num, den, n = O.token_diagnostics(x, np.eye(d))
    assert n == 200 and num == 0.0 and abs(den - np.sum(x * x)) < 1e-9 * den
    # per-row bounds 1/d <= PR/d <= 1, 1/d <= rho <= 1, and PR >= 1/rho (||y||_4^4 <= ||y||_inf^2 ||y||_2^2)
    for row in x[:20]:
        pr, rho, _, _, _ = O.token_diagnostics(row[None], np.eye(d))
        assert 1 / d - 1e-12 <= pr <= 1 + 1e-12 and 1 / d - 1e-12 <= rho <= 1 + 1e-12 and pr * rho >= 1 / d - 1e-12
    # extremes printed in the paper: one-sparse -> 1/d, equal magnitudes -> 1
    one_hot = np.zeros((1, d)); one_hot[0, 5] = -3.0
    corner = np.where(rng.random((1, d)) < 0.5, -1.0, 1.0) * 0.7
    assert abs(O.token_diagnostics(one_hot, np.eye(d))[0] - 1 / d) < 1e-15 and abs(O.token_diagnostics(one_hot, np.eye(d))[1] - 1) < 1e-15
    assert abs(O.token_diagnostics(corner, np.eye(d))[0] - 1) < 1e-12 and abs(O.token_diagnostics(corner, np.eye(d))[1] - 1 / d) < 1e-12
    # a Hadamard rotation turns one-hot rows into corners (PR/d: 1/d -> 1)
    h = I.hadamard_pm1(d) / np.sqrt(d)
    assert abs(O.token_diagnostics(one_hot, h)[0] - 1) < 1e-12
    # invariance to the row scale and to skipped rows
    x2 = x * 7.0; x2[3] = 0.0
    a = O.token_diagnostics(np.delete(x, 3, axis=0), np.eye(d)); b = O.token_diagnostics(x2, np.eye(d))
    assert abs(a[0] - b[0]) < 1e-10 and abs(a[1] - b[1]) < 1e-10 and b[4] == 199


@pytest.mark.parametrize("mode,clip", [("sym", 1.0), ("zp", 1.0), ("zp", 0.9)])
def test_relative_quantisation_error_definition_and_bound(mode, clip):
    d, n, bits = 32, 40, 4
    rng = np.random.default_rng(22)
    x = rng.standard_normal((n, d)) * np.exp(rng.standard_normal((n, 1)))
    r = np.linalg.qr(rng.standard_normal((d, d)))[0]
    spr, srho, num, den, used = O.token_diagnostics(x, r, bits, mode, clip)
    y = x @ r
    q = O.fake_quant_sym(y, bits)[0] if mode == "sym" else O.fake_quant_zp(y, bits, clip)[0]
    assert abs(num - np.linalg.norm(y - q) ** 2) < 1e-12 * num and abs(den - np.linalg.norm(x) ** 2) < 1e-12 * den
    if clip == 1.0:      # Appendix B: ||Q(y) - y||^2 <= d Delta^2 / 4 per row
        delta = (np.abs(y).max(axis=1) / 7) if mode == "sym" else ((y.max(axis=1) - y.min(axis=1)) / 15)
        assert num <= np.sum(d * delta ** 2 / 4) + 1e-12
    # the error is relative: scaling the activations changes nothing
    num2, den2 = O.token_diagnostics(3.0 * x, r, bits, mode, clip)[2:4]
    assert abs(num2 / den2 - num / den) < 1e-12
    # ... and against a per-element search that uses none of the oracle's quantiser code: every code on the row's
    # grid is tried and the nearest level taken (Appendix B: Q maps to the nearest grid point; ties do not change
    # the distance), with the grid written out from the definition of the step and the code range
    total = 0.0
    for row in y:
        if mode == "sym":
            step = np.abs(row).max() / (2 ** (bits - 1) - 1)
            levels = [step * k for k in range(-(2 ** (bits - 1) - 1), 2 ** (bits - 1))]
        else:
            lo, hi = clip * row.min(), clip * row.max()
            step = (hi - lo) / (2 ** bits - 1)
            zeta = -round(lo / step)                                   # integer zero-point
            levels = [step * (k - zeta) for k in range(0, 2 ** bits)]
        for v in row:
            total += min((v - lv) ** 2 for lv in levels)
    assert abs(num - total) <= 1e-10 * total
