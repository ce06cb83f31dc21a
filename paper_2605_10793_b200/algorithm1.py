"""Algorithm 1 (online calibration of the shared and the per-block rotations) as a sequence of library calls.

One context holds the shared rotation R_1: the attention-input and MLP-input activations of every block are
accumulated into it (`conqur_step`) and it is updated once per mini-batch (`conqur_update`).  One batched
context holds all L * n_heads diagonal blocks of the R_{2,l}: they are independent d_head x d_head problems; block l
feeds its n_heads problems from the head-interleaved o_proj input in one `conqur_step_batched_range` call.
Algorithm 1 updates R_{2,l} inside the loop over blocks; since R_{2,l} is not used again before the next
mini-batch and the problems are independent, all of them are updated here by ONE batched `conqur_update` at the
end of the mini-batch, which gives the same rotations with 1 instead of L latency-bound launches.

This file only sequences calls and moves pointers; all arithmetic runs in the library's kernels.  Weight
folding (Appendix A) for one transformer block is at the end.
"""
from __future__ import annotations

from typing import Dict, List, Optional

from . import binding as B


class Calibrator:
    def __init__(self, d: int, n_heads: int, d_head: int, n_layers: int, n_max: int, *, in_dtype="bf16", mode="tc",
                 quant_bits=0, quant_mode="sym", clip_ratio=0.0, prior_rel=0.0, record: Optional[str] = None,
                 queue_sites: bool = True):
        """n_max: most tokens in one activation matrix.  queue_sites (tensor-core mode): the R_1 context queues the 2L
        activation matrices of a mini-batch and runs its two products once over all of them (the statistics are sums
        over rows with R_1 fixed, Section 3.4); costs 4*d*n_max bytes of workspace per site.  record: None | "objective" | "full" (also keeps each
        cross-covariance, read before its update, and the sign decisions of every step; both synchronise and are
        meant for tests and logging)."""
        kw = dict(in_dtype=in_dtype, mode=mode, quant_bits=quant_bits, quant_mode=quant_mode, clip_ratio=clip_ratio,
                  prior_rel=prior_rel)
        self.d, self.n_heads, self.d_head, self.n_layers = d, n_heads, d_head, n_layers
        queue = min(64, 2 * n_layers) if (queue_sites and mode == "tc") else 0
        self.ctx1 = B.Context(d=d, n_max=n_max, defer_batches=queue, **kw)
        self.ctx2 = B.Context(d=d_head, n_max=n_max, batch=n_layers * n_heads, **kw)
        self.record = record
        self.log: List[Dict] = []
        self._cur: Dict = {}
        self._signs: Dict = {}
        self._capture = None
        if record == "full" and mode == "tc":
            # the fused per-head kernel keeps nothing of a step in memory: its sign decisions are captured as it runs
            import torch
            self._capture = torch.zeros((n_heads * n_max, d_head), dtype=torch.int8, device="cuda")
            self.ctx2.debug_capture_signs(self._capture)

    def set_rotations(self, r1, r2):
        """r1: (d, d); r2: (n_layers, n_heads, d_head, d_head); fp32 CUDA tensors."""
        self.ctx1.set_R(r1.contiguous())
        self.ctx2.set_R(r2.reshape(self.n_layers * self.n_heads, self.d_head, self.d_head).contiguous())

    def collect(self, layer: int, x_attn, x_mlp, x_o):
        """The body of Algorithm 1's loop over blocks for block `layer`: both residual-stream sites go into the R_1
        statistics, the o_proj input into the statistics of the block's n_heads problems.
        x_o: (n, n_heads*d_head), head h in columns h*d_head.."""
        full = self.record == "full"
        self.ctx1.step(x_attn)
        if full:
            self._signs[("attn", layer)] = self.ctx1.debug_get_signs(x_attn.shape[0]).cpu().numpy()
        self.ctx1.step(x_mlp)
        if full:
            self._signs[("mlp", layer)] = self.ctx1.debug_get_signs(x_mlp.shape[0]).cpu().numpy()
        assert x_o.shape[1] == self.n_heads * self.d_head and x_o.stride(1) == 1
        n = x_o.shape[0]
        self.ctx2.step_batched_range(x_o, n, x_o.stride(0), self.d_head, layer * self.n_heads, self.n_heads)
        if full:
            if self._capture is not None:
                self.ctx2.stream.synchronize()
                s2 = self._capture[: self.n_heads * n].reshape(self.n_heads, n, self.d_head).cpu().numpy()
            else:
                s2 = self.ctx2.debug_get_signs(n, problems=self.n_heads).cpu().numpy()
            self._signs[("o", layer)] = s2

    def end_minibatch(self):
        """R_{2,l} <- OPU(R_{2,l}, X_o^(l)) for every block, and R_1 <- OPU(R_1, X_1), with everything accumulated
        since the last call."""
        if self.record:
            L, H, dh = self.n_layers, self.n_heads, self.d_head
            j, n = self.ctx1.get_objective()
            j2, n2 = self.ctx2.get_objective()
            self._cur = {"J1": j, "N1": n, "J2": j2.reshape(L, H).copy(), "N2": n2.reshape(L, H).copy()}
            if self.record == "full":
                self._cur["M1"] = self.ctx1.get_M().cpu().numpy()
                self._cur["M2"] = self.ctx2.get_M().cpu().numpy().reshape(L, H, dh, dh)
                self._cur["signs"] = self._signs
                self._signs = {}
            self.log.append(self._cur)
            self._cur = {}
        self.ctx2.update()
        self.ctx1.update()

    def rotations(self):
        """(R_1 (d, d), R_2 (n_layers, n_heads, d_head, d_head)) as fp32 CUDA tensors."""
        return self.ctx1.get_R(), self.ctx2.get_R().reshape(self.n_layers, self.n_heads, self.d_head, self.d_head)

    def close(self):
        self.ctx1.close()
        self.ctx2.close()


# which side of which projection absorbs which rotation (Appendix A)
FOLD_PLAN = {
    "q": [("input", "r1")], "k": [("input", "r1")], "up": [("input", "r1")], "gate": [("input", "r1")],
    "v": [("input", "r1"), ("output", "r2")],
    "o": [("input", "r2"), ("output", "r1")],
    "down": [("output", "r1")],
}


def fold_block(weights: Dict[str, "object"], r1, r2_layer, mode: str = "tc") -> Dict[str, "object"]:
    """Fold R_1 and one block's R_2 into that block's projection weights.

    weights: name -> fp32 CUDA tensor (out_features, in_features) for any of q, k, v, o, up, gate, down (the RMSNorm
    scales already merged into the projections that follow them).  r2_layer: (n_heads, d_head, d_head)."""
    out = {}
    for name, w in weights.items():
        for side, which in FOLD_PLAN[name]:
            w = B.conqur_fold_weight(w, r1 if which == "r1" else r2_layer, side, mode)
        out[name] = w
    return out
