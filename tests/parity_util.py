"""Shared parity protocol: CUDA library vs the float64 oracle on the same seeded bits.

Teacher-forced: at every checked step the oracle is given the library's current R
(fp32 -> fp64, exact) and the same X values, so differences are the step's own
arithmetic.  Signs inside the rounding band of y = 0 (or of the fake-quant
dead-zone edge) are legitimately ambiguous: M is compared "tie-aware" (the
oracle re-forms M with the library's signs) and every differing sign must lie
inside the band; the raw M difference and the flip fraction are reported too.
"""
from __future__ import annotations

import numpy as np

from oracle import conqur_oracle as O

# tolerances: exact fp32 mode / bf16 tensor-core mode (M and J: stated requirements of the path; orth, gap: derived from the arithmetic)
TOL = {
    "exact": {"M": 1e-5, "J": 1e-6, "orth": 1e-4, "gap": 2e-5},
    "tc": {"M": 1e-2, "J": 1e-3, "orth": 1e-4, "gap": 1e-3},
}


# figures measured by the GPU tests of this session (written out by --parity-report)
REPORT: list = []


def log_parity(config: str, mode: str, what: str, rep: dict, **extra) -> None:
    """Record the numbers of one comparison (config = workload name, what = which step / update of it)."""
    keep = ("J_rel", "M_rel_tie_aware", "M_rel_raw", "flip_frac", "flips_outside_band", "orth", "gap", "R_dist", "cond")
    row = {"config": config, "mode": mode, "what": what}
    row.update({k: (float(rep[k]) if not isinstance(rep[k], int) else rep[k]) for k in keep if k in rep})
    row.update(extra)
    REPORT.append(row)


def assert_step(rep: dict, mode: str, flip_max: float) -> None:
    """The step assertions shared by every parity test: token count, objective, tie-aware cross-covariance, every
    differing sign inside the rounding band; and the raw cross-covariance too whenever no sign differs."""
    t = TOL[mode]
    assert rep["N_equal"], rep
    assert rep["J_rel"] <= t["J"], rep
    assert rep["M_rel_tie_aware"] <= t["M"], rep
    assert rep["flips_outside_band"] == 0, rep
    assert rep["flip_frac"] < flip_max, rep
    if rep["flip_frac"] == 0.0:
        assert rep["M_rel_raw"] <= t["M"], rep


def unit_roundoff(mode: str, d: int) -> float:
    """Relative size of the rounding band around a sign decision."""
    if mode == "exact":
        return np.sqrt(d) * 2.0 ** -24
    return 2.0 ** -8 + np.sqrt(d) * 2.0 ** -24


def step_parity(x64: np.ndarray, r64: np.ndarray, s_gpu: np.ndarray, m_gpu: np.ndarray, j_gpu: float, n_gpu: int,
                mode: str, quant_bits: int = 0, m_before: np.ndarray | None = None, j_before: float = 0.0,
                n_before: int = 0, quant_mode: str = "sym", clip_ratio: float = 1.0) -> dict:
    """Compare one library step against the oracle.  Returns a report dict (asserts nothing)."""
    d = x64.shape[1]
    qkw = dict(quant_bits=quant_bits, quant_mode=quant_mode, clip_ratio=clip_ratio)
    orc = O.OpuOracle(d, r64, **qkw).step(x64)
    s_ref = orc.last_S
    y = orc.last_Y
    m_ref = orc.M + (0.0 if m_before is None else m_before)
    j_ref = orc.J + j_before
    # tie-aware M: the oracle's arithmetic with the library's sign decisions
    ta = O.OpuOracle(d, r64, **qkw).step(x64, signs_override=s_gpu.astype(np.float64))
    m_ta = ta.M + (0.0 if m_before is None else m_before)
    diff = s_gpu.astype(np.float64) != s_ref
    flip_frac = float(diff.mean())
    # rounding band of each y_ij: u * sqrt(sum_k (x~_ik R_kj)^2)
    xt, used = O.normalise_rows(x64)
    scale = np.sqrt((xt * xt) @ (r64 * r64))
    u = unit_roundoff(mode, d)
    if quant_bits == 0:
        dist = np.abs(y)
    elif quant_mode == "sym":
        levels = 2 ** (quant_bits - 1) - 1
        delta = np.max(np.abs(y), axis=1, keepdims=True) / levels
        # distance to the dead-zone edge |y| = Delta/2; Delta itself carries the band of the row maximum
        dist = np.abs(np.abs(y) - delta / 2)
        row_arg = np.argmax(np.abs(y), axis=1)
        scale = scale + 0.5 * scale[np.arange(y.shape[0]), row_arg][:, None] / levels
    else:
        levels = 2 ** quant_bits - 1
        delta = clip_ratio * (np.max(y, axis=1, keepdims=True) - np.min(y, axis=1, keepdims=True)) / levels
        # sgn(q - zeta) = sgn(rint(y / Delta)): the same dead zone |y| < Delta/2, Delta from the row's max and min
        dist = np.abs(np.abs(y) - delta / 2)
        rows = np.arange(y.shape[0])
        ends = scale[rows, np.argmax(y, axis=1)] + scale[rows, np.argmin(y, axis=1)]
        scale = scale + 0.5 * clip_ratio * ends[:, None] / levels
    band = 6.0 * u * scale
    outside = diff & (dist > band) & used[:, None]
    rep = {
        "J_rel": abs(j_gpu - j_ref) / abs(j_ref),
        "N_equal": int(n_gpu) == int(orc.N + n_before),
        "M_rel_tie_aware": float(np.linalg.norm(m_gpu - m_ta) / np.linalg.norm(m_ta)),
        "M_rel_raw": float(np.linalg.norm(m_gpu - m_ref) / np.linalg.norm(m_ref)),
        "flip_frac": flip_frac,
        "flips_outside_band": int(outside.sum()),
        "J_per_token": j_ref / max(1, orc.N + n_before),
        "oracle": orc,
    }
    return rep


def update_parity(m_eff64: np.ndarray, r_new64: np.ndarray) -> dict:
    """Compare an updated rotation against the SVD polar factor of the same M_eff."""
    d = m_eff64.shape[0]
    r_ref, sigma = O.polar_svd(m_eff64)
    nuc = sigma.sum()
    return {
        "orth": float(np.max(np.abs(r_new64.T @ r_new64 - np.eye(d)))),
        "gap": float(1.0 - np.sum(r_new64 * m_eff64) / nuc),
        "R_dist": float(np.linalg.norm(r_new64 - r_ref) / np.sqrt(d)),
        "cond": float(sigma[0] / sigma[-1]),
        "R_ref": r_ref,
    }


def effective_m(m64: np.ndarray, r_prev64: np.ndarray, prior_rel: float) -> np.ndarray:
    """M_eff of the oracle for a given accumulated M (proximal term included)."""
    orc = O.OpuOracle(m64.shape[0], r_prev64, prior_rel=prior_rel)
    orc.M = np.array(m64, dtype=np.float64)
    return orc.effective_m()
