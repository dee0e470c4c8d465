"""One ATP layer as a sequence of C-ABI calls (Fig. 3): Norm -> basis -> attention on r principal
keys -> output projection and FeedForward through the low-rank representation.

The composition for the linear layers follows the paper's remark that the next stage "first attains
principal components" of its input: every linear layer sees (U_r, X_r) of its own input, with the
same rank r. All buffers are allocated once, here; forward() only issues library calls.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import torch

from . import binding as B


class AtpLayer:
    def __init__(self, ctx: B.Context, weights: Dict[str, torch.Tensor], lengths: Sequence[int], ranks: Sequence[int],
                 heads: int, ffn: Optional[str] = None, input_norm: Optional[str] = None, post_norm: str = "layer",
                 power_iters: int = -1, oversample: int = -1, seed: int = 0, basis_kwargs: Optional[dict] = None,
                 q_mode: str = "lowrank", rope_base: float = 0.0):
        self.ctx, self.w = ctx, weights
        self.lengths, self.ranks = [int(x) for x in lengths], [int(x) for x in ranks]
        self.heads, self.ffn, self.input_norm, self.post_norm = heads, ffn, input_norm, post_norm
        self.power_iters, self.oversample, self.seed = power_iters, oversample, seed
        self.basis_kwargs = dict(basis_kwargs or {})
        self.q_mode, self.rope_base = q_mode, rope_base
        self.has_wo = "W_O" in weights
        self.dtype = weights["W_Q"].dtype
        self.device = weights["W_Q"].device
        self.d = weights["W_Q"].shape[0]
        self.dp = weights["W_Q"].shape[1]
        self.d_ff = 0
        if ffn == "gelu":
            self.d_ff = weights["W_1"].shape[1]
        elif ffn == "swiglu":
            self.d_ff = weights["W_up"].shape[1]
        rows, tr, maxr = sum(self.lengths), sum(self.ranks), max(self.ranks)
        ldu = (maxr + 7) // 8 * 8

        def buf(r, c):
            return torch.empty((r, (c + 7) // 8 * 8), dtype=self.dtype, device=self.device)[:, :c]

        def basis_out(cols):
            return (torch.zeros((rows, ldu), dtype=self.dtype, device=self.device)[:, :maxr], buf(tr, cols),
                    torch.empty(tr, dtype=torch.float32, device=self.device))

        self.Xn = buf(rows, self.d) if input_norm else None
        self.bX = basis_out(self.d)
        self.O = buf(rows, self.dp)
        if self.has_wo:
            self.bO = basis_out(self.dp)
            self.A = buf(rows, self.d)
        if ffn:
            self.H = buf(rows, self.d)
            self.bH = basis_out(self.d)
            self.F = buf(rows, self.d_ff)
            self.bF = basis_out(self.d_ff)
            self.Y = buf(rows, self.d)
        # one workspace large enough for every call of the layer
        sd = B.SeqDesc(self.lengths, self.ranks)
        dt = B._dt(weights["W_Q"])
        need = max(ctx.workspace_bytes(B.OP_BASIS, sd, max(self.d, self.dp, self.d_ff), 0, dt),
                   ctx.workspace_bytes(B.OP_ATTENTION, sd, self.d, self.dp, dt),
                   ctx.workspace_bytes(B.OP_LINEAR, sd, max(self.d, self.d_ff), max(self.d, self.d_ff), dt))
        ctx.ensure_workspace(need)

    def _basis(self, X, out):
        return B.atp_principal_basis(self.ctx, X, self.lengths, self.ranks, oversample=self.oversample,
                                     power_iters=self.power_iters, seed=self.seed, out=out, auto_workspace=False,
                                     **self.basis_kwargs)

    def _linear(self, basis, W, out, act=None, W_gate=None):
        return B.atp_lowrank_linear(self.ctx, basis[0], basis[1], W, self.lengths, self.ranks, act=act, W_gate=W_gate,
                                    out=out, auto_workspace=False)

    def forward(self, X: torch.Tensor, stage_events: Optional[list] = None) -> torch.Tensor:
        """Returns the layer output (Y with an FFN, else the projected attention output, else O).
        stage_events: a list that receives (stage name, start event, end event) per library call, recorded on
        the current stream (for per-stage timing; None: nothing is recorded)."""
        c, w = self.ctx, self.w

        def timed(name, fn):
            if stage_events is None:
                return fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            out = fn()
            b.record()
            stage_events.append((name, a, b))
            return out

        Xin = X
        if self.input_norm:
            Xin = timed("norm_in", lambda: B.atp_input_norm(c, X, None, kind=self.input_norm, out=self.Xn))
        timed("basis_X", lambda: self._basis(Xin, self.bX))
        timed("attention", lambda: B.atp_attention(c, Xin, self.bX[0], self.bX[1], w["W_Q"], w["W_K"], w["W_V"], self.heads,
                                                   self.lengths, self.ranks, out=self.O, auto_workspace=False,
                                                   q_mode=self.q_mode, rope_base=self.rope_base))
        if not self.has_wo:
            return self.O
        timed("basis_O", lambda: self._basis(self.O, self.bO))
        timed("linear_WO", lambda: self._linear(self.bO, w["W_O"], self.A))
        if not self.ffn:
            return self.A
        timed("norm_post", lambda: B.atp_input_norm(c, X, self.A, kind=self.post_norm, out=self.H))   # H = Norm(X + A)
        timed("basis_H", lambda: self._basis(self.H, self.bH))
        if self.ffn == "gelu":
            timed("linear_ffn_in", lambda: self._linear(self.bH, w["W_1"], self.F, act="gelu"))
            timed("basis_F", lambda: self._basis(self.F, self.bF))
            timed("linear_ffn_out", lambda: self._linear(self.bF, w["W_2"], self.Y))
        else:
            timed("linear_ffn_in", lambda: self._linear(self.bH, w["W_up"], self.F, act="swiglu", W_gate=w["W_gate"]))
            timed("basis_F", lambda: self._basis(self.F, self.bF))
            timed("linear_ffn_out", lambda: self._linear(self.bF, w["W_down"], self.Y))
        return self.Y


class AtpStack:
    """A chain of ATP layers (Sec. 4.2: the next encoder/decoder layer first attains the principal components
    of the previous layer's output). Layer l maps X_l to Y_l = FFN(H_l) with H_l = Norm(X_l + A_l); the stack
    closes the block the usual post-norm way, X_{l+1} = Norm(H_l + Y_l). Layers without an FFN pass their
    output on unchanged. Every layer has its own weights; lengths, ranks and options are shared."""

    def __init__(self, ctx: B.Context, layer_weights: Sequence[Dict[str, torch.Tensor]], lengths: Sequence[int],
                 ranks: Sequence[int], heads: int, **layer_kwargs):
        self.ctx = ctx
        self.layers = [AtpLayer(ctx, w, lengths, ranks, heads, **layer_kwargs) for w in layer_weights]
        first = self.layers[0]
        rows = sum(first.lengths)
        self.Xnext = [torch.empty((rows, (first.d + 7) // 8 * 8), dtype=first.dtype, device=first.device)[:, :first.d]
                      for _ in self.layers]

    def forward(self, X: torch.Tensor) -> torch.Tensor:
        for layer, xn in zip(self.layers, self.Xnext):
            Y = layer.forward(X)
            X = B.atp_input_norm(self.ctx, layer.H, Y, kind=layer.post_norm, out=xn) if layer.ffn else Y
        return X
