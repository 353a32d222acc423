"""`torch.autograd` front end of the MoC FFN operator: marshalling only, every step runs in the CUDA library.

`moc_ffn(x, w_gate, w_up, w_down, k)` is the layer of Section 3.2 (Eq. (Moc-1), the Top-K mask, Eq. (MoC-2)) with the
backward of Section 4 (Eqs. (bp-1)..(bp-5)); between forward and backward only the compact Top-K activations are kept alive
(int16 channel indices and the gate / up values of the K selected channels per token: Section 4, Table 1, column "MoC+GCP"),
plus `x` for the weight gradients.
`MoCFFN` is a drop-in module holding the three weight matrices channel-major (`[d_ff, d_model]` each, the layout of
`nn.Linear.weight` for gate / up and of its transpose for down).

No gradient flows through the choice of channels (the mask is a constant in the backward equations).
"""
from __future__ import annotations

import torch

from . import binding as B


class _MoCFFNFunction(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, w_gate, w_up, w_down, k, d_ff, grouped, recompute_up, post_silu=False):
        shape = x.shape
        x2 = x.reshape(-1, shape[-1]).contiguous()
        save = any(ctx.needs_input_grad[:4])
        out, idx, tg, tu = B.moc_ffn_forward(x2, w_gate, w_up, w_down, None if k is None else int(k), d_ff=d_ff,
                                             save=save, grouped=bool(grouped), post_silu=bool(post_silu))
        if save:
            # recompute_up: the up values are dropped here and formed again in backward from x, w_up and the indices
            ctx.save_for_backward(x2, w_gate, w_up, w_down, idx, tg, *(() if recompute_up else (tu,)))
            ctx.d_ff = d_ff
            ctx.grouped = bool(grouped)
            ctx.x_shape = shape
        return out.reshape(shape)

    @staticmethod
    def backward(ctx, grad_out):
        x2, w_gate, w_up, w_down, idx, tg, *rest = ctx.saved_tensors
        names = ("x", "w_gate", "w_up", "w_down")
        want = tuple(n for n, need in zip(names, ctx.needs_input_grad[:4]) if need)
        go = grad_out.reshape(-1, grad_out.shape[-1]).contiguous()
        tu = rest[0] if rest else B.moc_ffn_recompute_up(x2, w_up, idx, d_ff=ctx.d_ff)
        res = B.moc_ffn_backward(x2, w_gate, w_up, w_down, idx, tg, tu, go, d_ff=ctx.d_ff, want=want,
                                 grouped=ctx.grouped)
        gx = res["grad_x"]
        return (None if gx is None else gx.reshape(ctx.x_shape), res["grad_w_gate"], res["grad_w_up"],
                res["grad_w_down"], None, None, None, None, None)


def moc_ffn(x: torch.Tensor, w_gate: torch.Tensor, w_up: torch.Tensor, w_down: torch.Tensor, k: int | None,
            d_ff: int | None = None, grouped: bool = False, recompute_up: bool = False,
            post_silu: bool = False) -> torch.Tensor:
    """out[..., :] = sum over the k channels j with the largest pre-SiLU gate value x.w_gate[j] of
    SiLU(x.w_gate[j]) * (x.w_up[j]) * w_down[j, :].  `x` is `[..., d_model]`, the weights `[d_ff_ld, d_model]` (rows at and
    past `d_ff`, when given, are padding and never selected).  grouped=True: the 2-of-8 mask of MoC 2:8 (Section 4)
    instead of the row Top-K: the 2 largest of every 8 consecutive channels, k = d_ff / 4.  recompute_up=True keeps only
    the indices and the gate values between forward and backward (k * (2 + e) instead of k * (2 + 2 e) bytes per token)
    and pays one more up projection in backward.  post_silu=True ranks the channels by SiLU(gate value) instead of the
    gate value (the paper's ablation of the Top-K position, Section 6.5; exact but slow kernels)."""
    return _MoCFFNFunction.apply(x, w_gate, w_up, w_down, k, d_ff, grouped, recompute_up, post_silu)


class MoCFFN(torch.nn.Module):
    """SwiGLU feed-forward block with Top-K channel selection on the gate (Section 3.2)."""

    def __init__(self, d_model: int, d_ff: int, k: int | None, dtype=torch.bfloat16, device="cuda", init_std: float = 0.02,
                 grouped: bool = False, recompute_up: bool = False, post_silu: bool = False):
        super().__init__()
        if grouped:
            k = B._grouped_k(k, d_ff)
        if not 1 <= k <= d_ff:
            raise ValueError("k must be in [1, d_ff]")
        self.d_model, self.d_ff, self.k, self.grouped = int(d_model), int(d_ff), int(k), bool(grouped)
        self.recompute_up = bool(recompute_up)
        self.post_silu = bool(post_silu)
        mk = lambda: torch.nn.Parameter(torch.empty(d_ff, d_model, dtype=dtype, device=device))
        self.w_gate, self.w_up, self.w_down = mk(), mk(), mk()
        self.reset_parameters(init_std)

    def reset_parameters(self, std: float = 0.02) -> None:
        for p in (self.w_gate, self.w_up, self.w_down):
            torch.nn.init.normal_(p, mean=0.0, std=std)

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return moc_ffn(x, self.w_gate, self.w_up, self.w_down, self.k, grouped=self.grouped,
                       recompute_up=self.recompute_up, post_silu=self.post_silu)

    def saved_bytes_per_token(self) -> int:
        """Bytes of activations alive between forward and backward per token, besides x and the output."""
        e = torch.empty((), dtype=self.w_gate.dtype).element_size()
        return self.k * (2 + (1 if self.recompute_up else 2) * e)

    def extra_repr(self) -> str:
        rule = "2 of every 8" if self.grouped else "row Top-K after SiLU" if self.post_silu else "row Top-K"
        return f"d_model={self.d_model}, d_ff={self.d_ff}, k={self.k} ({100.0 * self.k / self.d_ff:.1f} % of channels, {rule})"


__all__ = ["moc_ffn", "MoCFFN"]
