"""Float64 CPU oracle for ConQuR's orthogonal-Procrustes-update (OPU) hot path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
library is checked against.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it; the product path never does.  It shares no code
with the CUDA path and imports nothing from the package.

Conventions (row-vector form, as in the paper's Appendix A, "X_hat = X R"):
activations are the rows of X (n x d); the rotation acts on the right,
Y = X_tilde R.  The paper's Section 3.3 writes the same thing in column form
(R x_tilde, C = Z^T X_tilde, R <- U V^T); with R_here = R_paper^T and
M_here = C_paper^T the update R <- polar(M) below is that update transposed.

What each function follows:
  normalise_rows      Section 3.3, x_tilde = x / ||x||_2 (also Eq. 1)
  corner_target       Eq. 2, z = sign(R x) / sqrt(d)
  fake_quant_sym      Appendix B, Q_sym(x) = Delta * round(x / Delta),
                      Delta = ||x||_inf / (2^(b-1) - 1)
  fake_quant_zp       Appendix B, Q_zp(x) = Delta * (round(x / Delta + zeta) - zeta),
                      Delta = (max x - min x) / (2^b - 1), zeta the integer zero-point
                      that puts min x on the lower end of the grid; with the clipping
                      ratio of Appendix C (0.9 for activations) applied to the range
  OpuOracle.step      Section 3.3 (cross-covariance Z^T X_tilde) accumulated
                      across tensors as Section 3.4 allows; objective in the
                      l1 form of Section 3.2
  token_diagnostics   Section 4 diagnostics of the rotated rows: normalised participation ratio
                      PR(y)/d = ||y||_2^4 / (d ||y||_4^4), dynamic-range ratio
                      rho(y) = ||y||_inf^2 / ||y||_2^2 (Appendix B), and the relative squared
                      quantisation error ||X R - Q(X R)||_F^2 / ||X||_F^2 (on un-normalised rows)
  polar_svd           Section 3.3, C = U Sigma V^T, R <- U V^T
  procrustes_optimum  Section 3.3, the value tr(R^T C) = sum of singular values the update attains
  OpuOracle.update    Section 3.3 / Algorithm 1: R replaced, statistics reset
  run_algorithm1      Algorithm 1: per mini-batch, the attention-input and MLP-input activations of
                      every block accumulate into the shared R_1 problem, every head of every
                      block's o_proj input is its own d_h x d_h problem updated at once, and R_1 is
                      updated at the end of the mini-batch
  fold_weight         Appendix A: X W^T = (X R)(W R)^T, so a layer reading rotated activations
                      takes W R, and a layer writing into the rotated space takes R^T W
                      (block-diagonal R for the per-head rotations)
  hadamard_matrix / hadamard_rows
                      the fixed online transforms R_3, R_4 of Appendix A: the Sylvester
                      (Walsh-Hadamard) matrix H_d, applied as x H_d / sqrt(d)

Readings where the paper is silent (kept identical in the CUDA library):
  * sign(0) = 0: a zero coordinate adds nothing to the target or objective.
  * rows with zero or non-finite norm are skipped and counted.
  * fake-quant: b bits, levels -(2^(b-1)-1)..(2^(b-1)-1), clip ratio 1,
    round-half-to-even; the quantised row feeds the target and the objective,
    the unquantised normalised row feeds the cross-covariance.
  * zero-point fake-quant (quant_mode = "zp"): the range is [c min x, c max x] with
    clipping ratio c (Appendix C; the paper does not say how the ratio enters: it
    scales both ends, as in the evaluation code bases it follows), zeta =
    -round(c min x / Delta), codes are clamped to 0..2^b-1 (only matters for c < 1),
    round-half-to-even; a constant row (max = min) quantises to zero.
  * prior_rel = lam_rel > 0 makes the update polar(M + lam * R_prev) with
    lam = lam_rel * ||M||_F / sqrt(d) (a proximal Procrustes step, needed only
    when fewer tokens than dimensions were accumulated; not in the paper).

Pins: tests/test_oracle_pins.py (identities of Sections 3.1-3.3 and Appendix B,
d = 2 brute force, an independent Newton iteration for the polar factor,
per-element brute force).  The paper prints no worked numeric example of an
OPU, so there is no printed value to pin against: parity unpinned by worked
example; pinned by the identities and brute force above.
"""
from __future__ import annotations

import numpy as np


def normalise_rows(x):
    """x_tilde_i = x_i / ||x_i||_2 (Section 3.3).  Returns (x_tilde, used_mask).

    Rows whose norm is zero or not finite are dropped from the statistics
    (the paper does not define them); their x_tilde row is zero.
    """
    x = np.asarray(x, dtype=np.float64)
    with np.errstate(over="ignore", invalid="ignore"):
        s = np.sqrt(np.sum(x * x, axis=1))
    used = np.isfinite(s) & (s > 0.0)
    xt = np.zeros_like(x)
    xt[used] = x[used] / s[used, None]
    return xt, used


def sgn(y):
    """Mathematical sign with sgn(0) = 0 (also for -0.0)."""
    return np.sign(y) + 0.0


def corner_target(y):
    """Eq. 2: nearest vertex of the hypercube inscribed in the unit sphere."""
    d = y.shape[-1]
    return sgn(y) / np.sqrt(d)


def fake_quant_sym(y, bits):
    """Appendix B: per-row symmetric uniform quantiser.

    Returns (Q(y), integer codes q, step Delta per row).  Rows that are all
    zero get Delta = 0 and codes 0.
    """
    y = np.asarray(y, dtype=np.float64)
    levels = 2 ** (bits - 1) - 1
    delta = np.max(np.abs(y), axis=-1) / levels
    safe = np.where(delta > 0.0, delta, 1.0)
    q = np.rint(y / safe[..., None])          # numpy rint = round half to even
    q = np.clip(q, -levels, levels)
    q = np.where(delta[..., None] > 0.0, q, 0.0)
    return q * delta[..., None], q, delta


def fake_quant_zp(y, bits, clip_ratio=1.0):
    """Appendix B: per-row asymmetric (zero-point) uniform quantiser, range scaled by clip_ratio (Appendix C).

    Returns (Q(y), codes minus zero-point k = q - zeta, step Delta per row).
    """
    y = np.asarray(y, dtype=np.float64)
    levels = 2 ** bits - 1
    lo = clip_ratio * np.min(y, axis=-1)
    hi = clip_ratio * np.max(y, axis=-1)
    delta = (hi - lo) / levels
    ok = delta > 0.0
    safe = np.where(ok, delta, 1.0)
    zeta = -np.rint(lo / safe)                             # integer zero-point: round(lo/Delta + zeta) = 0
    q = np.rint(y / safe[..., None]) + zeta[..., None]     # round(y/Delta + zeta), zeta integer
    q = np.clip(q, 0.0, float(levels))
    k = np.where(ok[..., None], q - zeta[..., None], 0.0)
    return k * delta[..., None], k, delta


def token_diagnostics(x, r, quant_bits=0, quant_mode="sym", clip_ratio=1.0):
    """Sums over the used rows of x of PR(y)/d and rho(y) for y = x R, and numerator / denominator of the relative
    squared quantisation error (Section 4).  Returns (sum_pr_over_d, sum_rho, qerr_num, qerr_den, rows_used)."""
    x = np.asarray(x, dtype=np.float64)
    _, used = normalise_rows(x)
    y = x[used] @ np.asarray(r, dtype=np.float64)          # un-normalised: PR and rho do not depend on the row scale
    d = y.shape[1]
    n2 = np.sum(y * y, axis=1)
    pr = n2 * n2 / (d * np.sum(y ** 4, axis=1))
    rho = np.max(np.abs(y), axis=1) ** 2 / n2
    num = 0.0
    if quant_bits:
        qy = fake_quant_sym(y, quant_bits)[0] if quant_mode == "sym" else fake_quant_zp(y, quant_bits, clip_ratio)[0]
        num = float(np.sum((y - qy) ** 2))
    return float(pr.sum()), float(rho.sum()), num, float(np.sum(x[used] ** 2)), int(used.sum())


def polar_svd(m):
    """Orthogonal polar factor of m via the SVD: m = U S V^T -> U V^T (Section 3.3)."""
    u, s, vt = np.linalg.svd(np.asarray(m, dtype=np.float64))
    return u @ vt, s


def procrustes_optimum(m):
    """The value tr(R^T m) reaches at R = U V^T: the sum of the singular values of m (Section 3.3; for a full-rank m the
    maximiser is unique and no orthogonal R gives more).  Singular values only -- at d = 8192 the full factorisation
    of polar_svd takes minutes, this a fraction of that -- so an updated rotation can be judged by how much of the
    optimum it reaches."""
    return float(np.sum(np.linalg.svd(np.asarray(m, dtype=np.float64), compute_uv=False)))


class OpuOracle:
    """State machine R = OPU(R, X) with accumulate-then-update (Sections 3.3-3.4)."""

    def __init__(self, d, r0=None, quant_bits=0, prior_rel=0.0, quant_mode="sym", clip_ratio=1.0):
        self.d = int(d)
        self.quant_bits = int(quant_bits)
        self.quant_mode = quant_mode
        self.clip_ratio = float(clip_ratio)
        self.prior_rel = float(prior_rel)
        self.R = np.eye(self.d) if r0 is None else np.array(r0, dtype=np.float64)
        assert self.R.shape == (self.d, self.d)
        self.reset_stats()
        self.last_S = None      # sign matrix of the last step (n x d)
        self.last_Y = None
        self.last_sigma = None  # singular values seen by the last update

    def reset_stats(self):
        self.M = np.zeros((self.d, self.d))
        self.J = 0.0
        self.N = 0
        self.n_skipped = 0

    def step(self, x, signs_override=None):
        """Accumulate one batch with R fixed.

        signs_override (n x d of -1/0/+1), if given, replaces the oracle's own
        sign decisions in the cross-covariance (used for tie-aware parity:
        the objective still uses the oracle's own arithmetic).
        """
        d = self.d
        xt, used = normalise_rows(x)                     # Section 3.3
        y = xt @ self.R                                  # Eq. 1 in row form
        if self.quant_bits == 0:
            s = sgn(y)                                   # Eq. 2
            a = np.abs(y)                                # |y| summed -> l1 objective
        elif self.quant_mode == "sym":
            qy, q, delta = fake_quant_sym(y, self.quant_bits)   # Appendix B
            s = sgn(q)
            a = np.abs(qy)
        else:
            qy, q, delta = fake_quant_zp(y, self.quant_bits, self.clip_ratio)   # Appendix B / C
            s = sgn(q)
            a = np.abs(qy)
        s[~used] = 0.0
        a[~used] = 0.0
        s_used = s if signs_override is None else np.asarray(signs_override, dtype=np.float64)
        c = s_used / np.sqrt(d)                          # Eq. 2 scale
        self.M += xt.T @ c                               # Section 3.3 cross-covariance
        self.J += float(np.sum(a)) / np.sqrt(d)          # Section 3.2 l1 form
        self.N += int(np.count_nonzero(used))
        self.n_skipped += int(np.count_nonzero(~used))
        self.last_S = s
        self.last_Y = y
        return self

    def effective_m(self):
        """M, plus the proximal term lam * R_prev when prior_rel > 0."""
        if self.prior_rel > 0.0:
            lam = self.prior_rel * np.linalg.norm(self.M) / np.sqrt(self.d)
            return self.M + lam * self.R
        return self.M

    def update(self):
        """R <- polar(M_eff); statistics reset (Algorithm 1)."""
        if self.N == 0:
            raise ValueError("update with no accumulated tokens")
        m_eff = self.effective_m()
        r_new, sigma = polar_svd(m_eff)
        tol = sigma[0] * self.d * np.finfo(np.float64).eps
        if not (sigma[-1] > tol):
            raise np.linalg.LinAlgError("cross-covariance is rank deficient: polar factor not unique")
        self.last_sigma = sigma
        self.R = r_new
        self.reset_stats()
        return self

    # derived quantities of Section 3.2
    def objective_per_token(self):
        return self.J / self.N

    def corner_distance(self):
        """sum_i ||x_tilde_i R - c_i||^2 = 2N - 2J."""
        return 2.0 * self.N - 2.0 * self.J


def corner_distance_direct(x, r):
    """Left side of the identity of Section 3.2, evaluated literally."""
    xt, used = normalise_rows(x)
    y = xt[used] @ np.asarray(r, dtype=np.float64)
    z = corner_target(y)
    return float(np.sum((y - z) ** 2))


def procrustes_value(r, m):
    """<R, M>_F = tr(R^T M): the linear objective of the Procrustes subproblem."""
    return float(np.sum(np.asarray(r, dtype=np.float64) * np.asarray(m, dtype=np.float64)))


def run_stream(d, batches, r0, update_every, quant_bits=0, prior_rel=0.0):
    """Drive an oracle over an iterable of batches; returns (oracle, per-update log)."""
    orc = OpuOracle(d, r0, quant_bits, prior_rel)
    log = []
    for b, x in enumerate(batches):
        orc.step(x)
        if (b + 1) % update_every == 0:
            log.append({"J": orc.J, "N": orc.N, "J_per_token": orc.objective_per_token()})
            orc.update()
    return orc, log


def run_batched(d, xs, r0s, quant_bits=0, prior_rel=0.0):
    """Independent problems (one Procrustes problem per head): one step + one update each."""
    out = []
    for x, r0 in zip(xs, r0s):
        orc = OpuOracle(d, r0, quant_bits, prior_rel)
        orc.step(x)
        j, n = orc.J, orc.N
        m = orc.M.copy()
        orc.update()
        out.append({"R": orc.R, "J": j, "N": n, "M": m})
    return out


# ----------------------------------------------------------------------------- Algorithm 1, Appendix A
def run_algorithm1(d, n_heads, d_head, n_layers, minibatches, r1_0, r2_0, quant_bits=0, prior_rel=0.0,
                   quant_mode="sym", clip_ratio=1.0):
    """Algorithm 1 on given activations.

    minibatches: iterable; each item is a list over the L blocks of dicts with the activations collected at
    the three calibration sites of the block: "attn" and "mlp" (n x d, inputs of the attention and MLP
    sublayers) and "o" (n x n_heads*d_head, input of the attention output projection, head h in columns
    h*d_head .. (h+1)*d_head).  r1_0: d x d; r2_0: L x n_heads x d_head x d_head.
    Returns (R_1, R_2 as L x n_heads x d_head x d_head, log) where log holds, per mini-batch, the objective
    and token count of the R_1 problem and of every head problem before its update.
    """
    o1 = OpuOracle(d, r1_0, quant_bits, prior_rel, quant_mode, clip_ratio)
    r2 = np.array(r2_0, dtype=np.float64)
    assert r2.shape == (n_layers, n_heads, d_head, d_head)
    log = []
    for sites in minibatches:
        assert len(sites) == n_layers
        rec = {"J2": np.zeros((n_layers, n_heads)), "N2": np.zeros((n_layers, n_heads), dtype=np.int64)}
        for ell in range(n_layers):
            o1.step(sites[ell]["attn"])                           # accumulate into X_1
            o1.step(sites[ell]["mlp"])
            xo = np.asarray(sites[ell]["o"], dtype=np.float64)
            for h in range(n_heads):                              # R_{2,ell} is block diagonal: one problem per head
                oh = OpuOracle(d_head, r2[ell, h], quant_bits, prior_rel, quant_mode, clip_ratio)
                oh.step(xo[:, h * d_head:(h + 1) * d_head])
                rec["J2"][ell, h], rec["N2"][ell, h] = oh.J, oh.N
                oh.update()                                       # R_{2,ell} <- OPU(R_{2,ell}, X_o)
                r2[ell, h] = oh.R
        rec["J1"], rec["N1"] = o1.J, o1.N
        o1.update()                                               # R_1 <- OPU(R_1, X_1)
        log.append(rec)
    return o1.R, r2, log


def block_diag_rotation(blocks):
    """Dense (k*b) x (k*b) matrix with the given b x b blocks on its diagonal."""
    blocks = np.asarray(blocks, dtype=np.float64)
    if blocks.ndim == 2:
        return blocks
    k, b, _ = blocks.shape
    out = np.zeros((k * b, k * b))
    for i in range(k):
        out[i * b:(i + 1) * b, i * b:(i + 1) * b] = blocks[i]
    return out


def fold_weight(w, r_blocks, side):
    """Appendix A.  w: d_out x d_in weight of a layer y = x W^T.

    side "input":  the layer's input is rotated (x_hat = x R):              W' = W R
    side "output": the layer's output lives in the rotated space (y R):     W' = R^T W
    r_blocks: one square matrix, or a stack of blocks forming a block-diagonal R.
    """
    w = np.asarray(w, dtype=np.float64)
    r = block_diag_rotation(r_blocks)
    if side == "input":
        return w @ r
    if side == "output":
        return r.T @ w
    raise ValueError(side)


def hadamard_matrix(d):
    """Sylvester construction: H_1 = [1], H_2m = [[H_m, H_m], [H_m, -H_m]] (entries +-1, H H^T = d I)."""
    d = int(d)
    if d < 1 or d & (d - 1):
        raise ValueError("d must be a power of two")
    h = np.ones((1, 1))
    while h.shape[0] < d:
        h = np.block([[h, h], [h, -h]])
    return h


def hadamard_rows(x):
    """Each row times the orthonormal Walsh-Hadamard matrix: x H_d / sqrt(d) (the online R_3 / R_4 transform)."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    return x @ hadamard_matrix(d) / np.sqrt(d)
