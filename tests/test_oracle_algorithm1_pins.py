"""Pins for the oracle's Algorithm-1 composition, the weight folding of Appendix A and the Walsh-Hadamard
transform: each against something other than the oracle itself (hand-typed small cases, an independent library
routine, brute force, identities the paper states).  CPU only."""
import numpy as np
import pytest
import scipy.linalg

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I


def _orth(seed, d):
    q, r = np.linalg.qr(np.random.default_rng(seed).standard_normal((d, d)))
    return q * np.sign(np.diag(r))[None, :]


# ------------------------------------------------------------------------------------------ Walsh-Hadamard
def test_hadamard_small_cases_typed_by_hand():
    assert np.array_equal(O.hadamard_matrix(1), [[1]])
    assert np.array_equal(O.hadamard_matrix(2), [[1, 1], [1, -1]])
    assert np.array_equal(O.hadamard_matrix(4), [[1, 1, 1, 1], [1, -1, 1, -1], [1, 1, -1, -1], [1, -1, -1, 1]])
    with pytest.raises(ValueError):
        O.hadamard_matrix(12)


@pytest.mark.parametrize("d", [8, 64, 512])
def test_hadamard_entry_formula_library_routine_and_orthogonality(d):
    h = O.hadamard_matrix(d)
    i, j = np.meshgrid(np.arange(d), np.arange(d), indexing="ij")
    parity = np.zeros((d, d), dtype=np.int64)
    for b in range(d.bit_length()):
        parity ^= ((i & j) >> b) & 1
    assert np.array_equal(h, 1 - 2 * parity)                      # H[i][j] = (-1)^popcount(i & j)
    assert np.array_equal(h, scipy.linalg.hadamard(d))
    assert np.array_equal(h @ h.T, d * np.eye(d))
    assert np.array_equal(h, I.hadamard_pm1(d))


def test_hadamard_rows_against_butterflies_unit_vectors_and_involution():
    rng = np.random.default_rng(5)
    d = 32
    x = rng.standard_normal((7, d))
    y = O.hadamard_rows(x)
    # the textbook in-place butterfly network, written out with loops
    ref = x.copy()
    h = 1
    while h < d:
        for r in range(ref.shape[0]):
            for s in range(0, d, 2 * h):
                for k in range(s, s + h):
                    a, b = ref[r, k], ref[r, k + h]
                    ref[r, k], ref[r, k + h] = a + b, a - b
        h *= 2
    ref /= np.sqrt(d)
    assert np.allclose(y, ref, rtol=0, atol=1e-13)
    e = np.eye(d)
    assert np.allclose(O.hadamard_rows(e), O.hadamard_matrix(d) / np.sqrt(d), atol=1e-15)
    assert np.allclose(O.hadamard_rows(y), x, atol=1e-13)          # symmetric and orthogonal: its own inverse
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1))
    # a constant row concentrates in coordinate 0; an outlier spreads evenly (what R_3 / R_4 are used for)
    assert np.allclose(O.hadamard_rows(np.ones((1, d))), np.sqrt(d) * e[:1])
    assert np.allclose(np.abs(O.hadamard_rows(5.0 * e[3:4])), 5.0 / np.sqrt(d))


# ------------------------------------------------------------------------------------------ weight folding
def test_fold_weight_preserves_the_layer_as_appendix_a_states():
    rng = np.random.default_rng(11)
    t, d, do = 9, 16, 12
    x = rng.standard_normal((t, d))
    w = rng.standard_normal((do, d))
    r = _orth(1, d)
    assert np.linalg.norm(r - r.T) > 0.5                          # not symmetric: a transposed R would fail below
    # input side: X W^T = (X R)(W R)^T
    assert np.allclose(x @ w.T, (x @ r) @ O.fold_weight(w, r, "input").T, atol=1e-12)
    # output side: (X W2^T) R = X (R^T W2)^T for a layer writing d-dimensional outputs
    w2 = rng.standard_normal((d, do))
    z = rng.standard_normal((t, do))
    assert np.allclose((z @ w2.T) @ r, z @ O.fold_weight(w2, r, "output").T, atol=1e-12)
    # and the wrong side breaks the identity
    assert not np.allclose(x @ w.T, (x @ r) @ O.fold_weight(w, r.T, "input").T, atol=1e-3)


def test_fold_weight_element_by_element_and_block_diagonal():
    rng = np.random.default_rng(12)
    nh, dh, do = 3, 4, 5
    blocks = np.stack([_orth(20 + h, dh) for h in range(nh)])
    w = rng.standard_normal((do, nh * dh))
    got = O.fold_weight(w, blocks, "input")
    for i in range(do):
        for h in range(nh):
            for j in range(dh):
                acc = 0.0
                for k in range(dh):
                    acc += w[i, h * dh + k] * blocks[h, k, j]
                assert abs(got[i, h * dh + j] - acc) < 1e-13
    assert np.allclose(got, w @ scipy.linalg.block_diag(*blocks))
    wv = rng.standard_normal((nh * dh, do))
    got = O.fold_weight(wv, blocks, "output")
    for h in range(nh):
        for i in range(dh):
            for j in range(do):
                acc = 0.0
                for k in range(dh):
                    acc += blocks[h, k, i] * wv[h * dh + k, j]
                assert abs(got[h * dh + i, j] - acc) < 1e-13


def test_folding_a_whole_block_leaves_its_function_unchanged():
    """R_1 on the residual stream and per-head R_2 between the value and output projections (Appendix A): the
    value -> output chain and an MLP-like chain computed from rotated residuals with folded weights reproduce the
    rotated outputs of the original chain."""
    rng = np.random.default_rng(13)
    t, d, nh, dh, dff = 6, 8, 2, 4, 10
    x = rng.standard_normal((t, d))
    wv, wo = rng.standard_normal((nh * dh, d)), rng.standard_normal((d, nh * dh))
    wup, wdown = rng.standard_normal((dff, d)), rng.standard_normal((d, dff))
    r1 = _orth(2, d)
    r2 = np.stack([_orth(30 + h, dh) for h in range(nh)])
    wv_f = O.fold_weight(O.fold_weight(wv, r1, "input"), r2, "output")
    wo_f = O.fold_weight(O.fold_weight(wo, r2, "input"), r1, "output")
    xr = x @ r1
    v_rot = xr @ wv_f.T
    assert np.allclose(v_rot, (x @ wv.T) @ scipy.linalg.block_diag(*r2), atol=1e-12)   # the o_proj input is rotated by R_2
    assert np.allclose(v_rot @ wo_f.T, (x @ wv.T @ wo.T) @ r1, atol=1e-12)
    wup_f, wdown_f = O.fold_weight(wup, r1, "input"), O.fold_weight(wdown, r1, "output")
    act = lambda u: np.maximum(u, 0.0)
    assert np.allclose(act(xr @ wup_f.T) @ wdown_f.T, (act(x @ wup.T) @ wdown.T) @ r1, atol=1e-12)


# ------------------------------------------------------------------------------------------ Algorithm 1
def _tiny_sites(seed, L, n, d, nh, dh):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(L):
        s = {"attn": rng.standard_normal((n, d)), "mlp": rng.standard_normal((n, d)),
             "o": rng.standard_normal((n, nh * dh))}
        s["attn"][:, 0] *= 20.0
        s["o"][:, ::dh] *= 10.0
        out.append(s)
    return out


def _polar_of_pooled(x, r):
    """R <- polar of sum_i x_tilde_i^T sign(x_tilde_i R)/sqrt(d), by an independent route (scipy's polar)."""
    xt = x / np.linalg.norm(x, axis=1, keepdims=True)
    m = xt.T @ (np.sign(xt @ r) / np.sqrt(x.shape[1]))
    return scipy.linalg.polar(m)[0], m


def test_algorithm1_one_minibatch_is_the_pooled_problem_per_rotation():
    L, n, d, nh, dh = 3, 40, 8, 2, 4
    sites = _tiny_sites(1, L, n, d, nh, dh)
    r1_0 = _orth(3, d)
    r2_0 = np.stack([np.stack([_orth(100 + l * nh + h, dh) for h in range(nh)]) for l in range(L)])
    r1, r2, log = O.run_algorithm1(d, nh, dh, L, [sites], r1_0, r2_0)
    pooled = np.concatenate([s[k] for s in sites for k in ("attn", "mlp")], axis=0)
    ref1, m1 = _polar_of_pooled(pooled, r1_0)
    assert np.allclose(r1, ref1, atol=1e-10)
    assert log[0]["N1"] == 2 * L * n
    xt = pooled / np.linalg.norm(pooled, axis=1, keepdims=True)
    assert np.isclose(log[0]["J1"], np.abs(xt @ r1_0).sum() / np.sqrt(d))
    for l in range(L):
        for h in range(nh):
            ref2, _ = _polar_of_pooled(sites[l]["o"][:, h * dh:(h + 1) * dh], r2_0[l, h])
            assert np.allclose(r2[l, h], ref2, atol=1e-10), (l, h)
            assert log[0]["N2"][l, h] == n
    # heads and blocks are independent problems; the R_1 problem does not see the o_proj inputs
    sites2 = [dict(s) for s in sites]
    sites2[1] = dict(sites2[1])
    o = sites2[1]["o"].copy()
    o[:, dh:] = np.random.default_rng(9).standard_normal((n, dh))
    sites2[1]["o"] = o
    r1b, r2b, _ = O.run_algorithm1(d, nh, dh, L, [sites2], r1_0, r2_0)
    assert np.array_equal(r1b, r1)
    changed = np.array([[not np.array_equal(r2b[l, h], r2[l, h]) for h in range(nh)] for l in range(L)])
    expect = np.zeros((L, nh), dtype=bool)
    expect[1, 1] = True
    assert np.array_equal(changed, expect)
    # the order in which the blocks contribute to X_1 does not matter
    r1c, _, _ = O.run_algorithm1(d, nh, dh, L, [sites[::-1]], r1_0, r2_0[::-1])
    assert np.allclose(r1c, r1, atol=1e-12)


def test_algorithm1_second_minibatch_starts_from_the_updated_rotations_and_ascends():
    L, n, d, nh, dh = 2, 64, 8, 2, 4
    mb = [_tiny_sites(2, L, n, d, nh, dh), _tiny_sites(3, L, n, d, nh, dh)]
    r1_0 = np.eye(d)
    r2_0 = np.tile(np.eye(dh), (L, nh, 1, 1))
    r1a, r2a, _ = O.run_algorithm1(d, nh, dh, L, mb[:1], r1_0, r2_0)
    r1b, r2b, log = O.run_algorithm1(d, nh, dh, L, mb, r1_0, r2_0)
    pooled = np.concatenate([s[k] for s in mb[1] for k in ("attn", "mlp")], axis=0)
    ref, _ = _polar_of_pooled(pooled, r1a)                      # targets of mini-batch 2 come from R_1 after mini-batch 1
    assert np.allclose(r1b, ref, atol=1e-10)
    ref2, _ = _polar_of_pooled(mb[1][0]["o"][:, :dh], r2a[0, 0])
    assert np.allclose(r2b[0, 0], ref2, atol=1e-10)
    for r in (r1b, r2b[1, 1]):
        assert np.allclose(r.T @ r, np.eye(r.shape[0]), atol=1e-12)
    # the update is an ascent step of the l1 objective on the mini-batch it was computed from (Section 3.3)
    xt = pooled / np.linalg.norm(pooled, axis=1, keepdims=True)
    j_old = np.abs(xt @ r1a).sum() / np.sqrt(d)
    j_new = np.abs(xt @ r1b).sum() / np.sqrt(d)
    assert np.isclose(log[1]["J1"], j_old)
    assert j_new >= j_old


def test_site_model_generator_shapes_and_determinism():
    a = I.SITE_MODELS["a1_small"]
    s = I.site_activations(a, 1, 0)
    assert s["attn"].shape == (a.n, a.d) and s["mlp"].shape == (a.n, a.d) and s["o"].shape == (a.n, a.n_heads * a.d_head)
    assert np.array_equal(s["o"], I.site_activations(a, 1, 0)["o"])
    assert not np.array_equal(s["attn"], s["mlp"])
    assert not np.array_equal(s["o"][:, :a.d_head], s["o"][:, a.d_head:])
    r1, r2 = I.site_initial_rotations(a)
    assert np.allclose(r1.T.astype(np.float64) @ r1, np.eye(a.d), atol=1e-5)
    assert r2.shape == (a.n_layers, a.n_heads, a.d_head, a.d_head)
