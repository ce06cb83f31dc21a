"""Seeded synthetic calibration inputs (shared data for the oracle and the CUDA path).

Stand-ins for the activations the paper taps from Llama models during
calibration (Section 4: 128 sequences of 2048 tokens): heavy-tailed rows with
a few outlier channels, a per-token scale and a few massive-activation tokens.
This module only *draws numbers*: it holds none of the method's arithmetic
(no normalisation, rotation, sign, cross-covariance or polar step), so both
the float64 oracle and the GPU library can consume its output bits.

Every value is generated in float64 from ``numpy.random.Generator(PCG64(seed))``
and rounded ONCE to the workload's storage type (bf16 round-to-nearest-even or
fp32).  Arrays are returned as float32 whose values are exactly representable
in that storage type; ``to_bf16_bits`` gives the uint16 payload for the GPU.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np

# ----------------------------------------------------------------------------
# storage-type rounding (data conversion only)
# ----------------------------------------------------------------------------


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round to bfloat16 (nearest, ties to even); result held in float32."""
    a32 = np.ascontiguousarray(a, dtype=np.float32)
    u = a32.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = ((u + bias) & np.uint32(0xFFFF0000)).astype(np.uint32)
    nan = np.isnan(a32)
    if nan.any():
        r = np.where(nan, np.uint32(0x7FC00000), r)
    return r.view(np.float32).reshape(a32.shape)


def to_bf16_bits(a_bf16_in_f32: np.ndarray) -> np.ndarray:
    """uint16 payload of a float32 array whose values are bf16-representable."""
    u = np.ascontiguousarray(a_bf16_in_f32, dtype=np.float32).view(np.uint32)
    return (u >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(bits: np.ndarray) -> np.ndarray:
    """float32 array from a uint16 bf16 payload."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# workloads
# ----------------------------------------------------------------------------


@dataclass(frozen=True)
class Workload:
    """One calibration stream: shapes, value distribution and update cadence."""

    name: str
    index: int                 # used for seeding: seed = 1000*index + batch
    d: int                     # feature dimension of one Procrustes problem
    n: int                     # tokens (rows) per streamed batch
    n_batches: int             # batches in the stream
    update_every: int          # `update` after this many `step` calls
    dtype: str                 # "f32" or "bf16": storage type of X
    dist: str                  # "normal" or "student_t3"
    n_outlier: int             # outlier channels
    outlier_scale: float
    token_scale_sigma: float   # row scale exp(sigma*N(0,1)); 0 = none
    n_massive_rows: int        # massive-activation tokens per batch
    massive_scale: float
    r0: str                    # "identity" | "qr" | "hadamard"
    quant_bits: int = 0        # 0 = plain corner target, 4 = INT4 fake-quant first
    prior_rel: float = 0.0     # proximal weight for rank-deficient updates
    problems: int = 1          # independent problems (batched variant)
    same_batch: bool = False   # every step sees batch 0 (alternation on a fixed batch)
    quant_mode: str = "sym"    # "sym": symmetric per-token quantiser; "zp": zero-point quantiser
    clip_ratio: float = 1.0    # range clipping ratio of the zero-point quantiser
    ns_steps: int = 0          # Newton-Schulz steps the polar update plans for (0 = the library's default plan)


WORKLOADS: Dict[str, Workload] = {
    # d=128 alternation on one fixed fp32 batch, 10 (step, update) rounds
    "c0": Workload("c0", 0, 128, 2048, 10, 1, "f32", "normal", 4, 50.0, 0.0, 0, 1.0,
                   "identity", same_batch=True),
    # d=2 brute-force companion of c0
    "c0_d2": Workload("c0_d2", 9, 2, 64, 1, 1, "f32", "normal", 1, 5.0, 0.0, 0, 1.0,
                      "identity", same_batch=True),
    # 3B-class residual width, one update per batch (fewer tokens than dims)
    "c1": Workload("c1", 1, 3072, 2048, 32, 1, "bf16", "student_t3", 8, 100.0, 0.5, 0, 1.0,
                   "qr", prior_rel=1e-2),
    # 7B/8B-class residual width: the headline timing workload
    "c2": Workload("c2", 2, 4096, 2048, 128, 8, "bf16", "student_t3", 16, 100.0, 0.5, 4, 1000.0,
                   "hadamard"),
    # 70B-class residual width
    "c3": Workload("c3", 3, 8192, 4096, 64, 16, "bf16", "student_t3", 32, 100.0, 0.5, 4, 1000.0,
                   "hadamard", ns_steps=8),
    # c2 with per-token symmetric INT4 fake-quantisation of the rotated rows
    "c4a": Workload("c4a", 4, 4096, 2048, 128, 8, "bf16", "student_t3", 16, 100.0, 0.5, 4, 1000.0,
                    "hadamard", quant_bits=4),
    # c2 with the quantiser the paper's evaluation uses: per-token zero-point INT4, clipping ratio 0.9
    "c4a_zp": Workload("c4a_zp", 6, 4096, 2048, 128, 8, "bf16", "student_t3", 16, 100.0, 0.5, 4, 1000.0,
                       "hadamard", quant_bits=4, quant_mode="zp", clip_ratio=0.9),
    # per-head problems: 1024 independent d=128 problems, one step + one update each
    "c4b": Workload("c4b", 5, 128, 4096, 1, 1, "bf16", "student_t3", 2, 100.0, 0.5, 1, 1000.0,
                    "hadamard", problems=1024),
}


def scaled(w: Workload, **kw) -> Workload:
    """A reduced copy of a workload (same recipe, smaller sizes) for parity tests."""
    return replace(w, **kw)


def _config_rng(w: Workload, salt: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(7_000_000 + 100 * w.index + salt))


def outlier_channels(w: Workload) -> np.ndarray:
    """Outlier channel indices, drawn once per workload."""
    if w.n_outlier == 0:
        return np.zeros(0, dtype=np.int64)
    return np.sort(_config_rng(w, 1).choice(w.d, size=min(w.n_outlier, w.d), replace=False))


def massive_dims(w: Workload) -> np.ndarray:
    """The (up to) 4 fixed dimensions that massive-activation tokens blow up."""
    return np.sort(_config_rng(w, 2).choice(w.d, size=min(4, w.d), replace=False))


def batch_seed(w: Workload, b: int, problem: int = 0) -> int:
    b_eff = 0 if w.same_batch else b
    return 1000 * w.index + b_eff + 1_000_003 * problem


def batch(w: Workload, b: int, problem: int = 0) -> np.ndarray:
    """Batch ``b`` of the stream: (n, d) float32, values exact in ``w.dtype``."""
    rng = np.random.Generator(np.random.PCG64(batch_seed(w, b, problem)))
    if w.dist == "normal":
        x = rng.standard_normal((w.n, w.d))
    elif w.dist == "student_t3":
        x = rng.standard_t(3.0, size=(w.n, w.d))
    else:
        raise ValueError(w.dist)
    ch = outlier_channels(w)
    if ch.size:
        x[:, ch] *= w.outlier_scale
    if w.token_scale_sigma > 0.0:
        x *= np.exp(w.token_scale_sigma * rng.standard_normal((w.n, 1)))
    if w.n_massive_rows > 0:
        rows = np.zeros(1, dtype=np.int64)  # the first token of a sequence ...
        if w.n_massive_rows > 1:            # ... plus seeded positions
            extra = rng.choice(np.arange(1, w.n), size=w.n_massive_rows - 1, replace=False)
            rows = np.concatenate([rows, np.sort(extra)])
        md = massive_dims(w)
        x[np.ix_(rows, md)] *= w.massive_scale
    if w.dtype == "bf16":
        return round_to_bf16(x)
    if w.dtype == "f32":
        return x.astype(np.float32)
    raise ValueError(w.dtype)


def hadamard_pm1(d: int) -> np.ndarray:
    """Sylvester Hadamard matrix with entries +-1 (int8); d a power of two."""
    if d < 1 or (d & (d - 1)) != 0:
        raise ValueError("Hadamard size must be a power of two")
    h = np.ones((1, 1), dtype=np.int8)
    while h.shape[0] < d:
        h = np.block([[h, h], [h, -h]])
    return h


def initial_rotation(w: Workload, problem: int = 0) -> np.ndarray:
    """R0 as float32 (d, d): identity, sign-fixed QR of a Gaussian, or H*diag(+-1)/sqrt(d)."""
    rng = _config_rng(w, 3 + 17 * problem)
    if w.r0 == "identity":
        return np.eye(w.d, dtype=np.float32)
    if w.r0 == "qr":
        g = rng.standard_normal((w.d, w.d))
        q, r = np.linalg.qr(g)
        q = q * np.where(np.diag(r) < 0, -1.0, 1.0)[None, :]
        return q.astype(np.float32)
    if w.r0 == "hadamard":
        s = rng.choice(np.array([-1.0, 1.0]), size=w.d)
        h = hadamard_pm1(w.d).astype(np.float32)
        return (h * s[None, :].astype(np.float32)) * np.float32(1.0 / np.sqrt(w.d))
    raise ValueError(w.r0)


def stream(w: Workload):
    """Yield (batch_index, X, do_update_after) over the whole stream."""
    for b in range(w.n_batches):
        yield b, batch(w, b), ((b + 1) % w.update_every == 0)


def storage_bytes_per_element(w: Workload) -> int:
    return 2 if w.dtype == "bf16" else 4


# ----------------------------------------------------------------------------
# Algorithm 1: calibration sites of a synthetic transformer
# ----------------------------------------------------------------------------


@dataclass(frozen=True)
class SiteModel:
    """Shapes of a pre-norm transformer as Algorithm 1 sees it, and the recipes of its site activations.

    Per mini-batch every block yields three activation matrices: the attention input and the MLP input
    (n x d, residual-stream statistics: recipe ``resid``) and the input of the attention output projection
    (n x n_heads*d_head, head h in columns h*d_head..(h+1)*d_head: recipe ``head`` per head).
    """

    name: str
    index: int
    d: int
    n_heads: int
    d_head: int
    n_layers: int
    n: int                 # tokens per mini-batch (sequences x sequence length)
    n_minibatches: int
    resid: Workload
    head: Workload
    d_ff: int = 0          # MLP width, for the weight-folding shapes


def _site_model(name, index, d, n_heads, d_head, n_layers, n, n_minibatches, dtype, d_ff) -> SiteModel:
    resid = Workload(name + "_resid", 20 + index, d, n, n_minibatches, 1, dtype, "student_t3", max(1, d // 256), 100.0,
                     0.5, 1, 1000.0, "hadamard")
    head = Workload(name + "_head", 40 + index, d_head, n, n_minibatches, 1, dtype, "student_t3", 2, 30.0, 0.5, 0, 1.0,
                    "hadamard")
    return SiteModel(name, index, d, n_heads, d_head, n_layers, n, n_minibatches, resid, head, d_ff)


SITE_MODELS: Dict[str, SiteModel] = {
    # a model the float64 oracle runs in seconds: 2 blocks, 2 heads of 128, residual width 256
    "a1_small": _site_model("a1_small", 0, 256, 2, 128, 2, 640, 2, "bf16", 512),
    # 8B-class shapes: 32 blocks, residual width 4096, 32 heads of 128, two 2048-token sequences per mini-batch
    "a1_8b": _site_model("a1_8b", 1, 4096, 32, 128, 32, 4096, 1, "bf16", 14336),
}


def site_activations(a: SiteModel, minibatch: int, layer: int) -> Dict[str, np.ndarray]:
    """The three activation matrices of block ``layer`` for one mini-batch (float32, exact in the storage type)."""
    b_attn = (minibatch * a.n_layers + layer) * 2
    attn = batch(a.resid, b_attn)
    mlp = batch(a.resid, b_attn + 1)
    heads = [batch(a.head, minibatch * a.n_layers + layer, problem=h) for h in range(a.n_heads)]
    return {"attn": attn, "mlp": mlp, "o": np.concatenate(heads, axis=1)}


def site_initial_rotations(a: SiteModel):
    """(R_1 as d x d, R_2 as n_layers x n_heads x d_head x d_head), float32."""
    r1 = initial_rotation(a.resid)
    r2 = np.stack([np.stack([initial_rotation(a.head, problem=l * a.n_heads + h) for h in range(a.n_heads)])
                   for l in range(a.n_layers)])
    return r1, r2


def random_weight(seed: int, rows: int, cols: int) -> np.ndarray:
    """A linear layer's weight (rows = outputs, cols = inputs), float32, N(0, 1/cols) entries."""
    rng = np.random.Generator(np.random.PCG64(9_000_000 + seed))
    return (rng.standard_normal((rows, cols)) / np.sqrt(cols)).astype(np.float32)
