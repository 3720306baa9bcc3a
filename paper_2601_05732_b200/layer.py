"""Device buffers of one Hyper-Connections layer and the call sequences around the caller's sublayer.

Plumbing only: tensors are allocated with PyTorch and handed to the C ABI through
:class:`~paper_2601_05732_b200.binding.MhcLite`; every step of the path runs in the
library's kernels.

Forward (paper Eq. (1), (4), (5)):   pre  -> [sublayer f: the caller's] -> post
Backward:                            post_bwd -> [f's backward]        -> tail
"""
from __future__ import annotations

import numpy as np
import torch

from .binding import MhcLite


def to_device_bf16(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 tensor on the device (no value conversion)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_to_host_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


class LayerParams:
    def __init__(self, W, b, alpha, gain, device):
        f = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
        self.W, self.b, self.alpha, self.gain = f(W), f(b), f(alpha), f(gain)


class LayerBuffers:
    """Outputs and saved tensors of one layer for T tokens (kind 'lite' or 'sk')."""

    def __init__(self, ctx: MhcLite, T: int, kind: str = "lite"):
        n, C, dev = ctx.n, ctx.C, f"cuda:{ctx.device}"
        self.kind = kind
        N = ctx.n_cols(0 if kind == "lite" else 1)
        f32 = lambda *s: torch.empty(*s, dtype=torch.float32, device=dev)
        bf = lambda *s: torch.empty(*s, dtype=torch.bfloat16, device=dev)
        self.H_res, self.H_pre, self.H_post = f32(T, n, n), f32(T, n), f32(T, n)
        self.a_saved = f32(T, ctx.nfact) if kind == "lite" else None
        self.p_saved, self.rstd = f32(T, N), f32(T)
        self.u, self.x_next = bf(T, C), bf(T, n, C)
        self.dy, self.dx = bf(T, C), bf(T, n, C)
        self.dH_res, self.dH_post, self.dH_pre = f32(T, n, n), f32(T, n), f32(T, n)
        self.dW, self.db, self.dalpha, self.dgain = f32(n * C, N), f32(N), f32(4)[:3], f32(n * C)
        ctx.ensure_workspace(T, 0 if kind == "lite" else 1)


def pre_fwd(ctx: MhcLite, P: LayerParams, B: LayerBuffers, x, eps=1e-6, fused=True, iters=20, u_rstd=None, eps_u=1e-6):
    """Mappings + stream pre-mix: everything before the sublayer. Result: B.u (and the coefficients).  With u_rstd
    (fp32 [T], fused lite path only) the call also leaves the RMSNorm row statistic of the stored u there."""
    if u_rstd is not None:
        if B.kind != "lite" or not fused:
            raise ValueError("u_rstd is produced by the fused mHC-lite call only")
        ctx.pre_fwd_fused_ustat(x, P.W, P.b, P.alpha, P.gain, eps, B.H_res, B.H_pre, B.H_post, B.a_saved, B.p_saved,
                                B.rstd, B.u, u_rstd, eps_u)
        return
    if B.kind == "sk" and fused:
        ctx.sk20_pre_fwd_fused(x, P.W, P.b, P.alpha, P.gain, eps, iters, B.H_res, B.H_pre, B.H_post, B.p_saved, B.rstd,
                               B.u)
    elif B.kind == "sk":
        ctx.sk20_coeffs_fwd(x, P.W, P.b, P.alpha, P.gain, eps, iters, B.H_res, B.H_pre, B.H_post, B.p_saved, B.rstd)
        ctx.premix_fwd(x, B.H_pre, B.u)
    elif fused:
        ctx.pre_fwd_fused(x, P.W, P.b, P.alpha, P.gain, eps, B.H_res, B.H_pre, B.H_post, B.a_saved, B.p_saved,
                          B.rstd, B.u)
    else:
        ctx.coeffs_fwd(x, P.W, P.b, P.alpha, P.gain, eps, B.H_res, B.H_pre, B.H_post, B.a_saved, B.p_saved, B.rstd)
        ctx.premix_fwd(x, B.H_pre, B.u)


def post_fwd(ctx: MhcLite, B: LayerBuffers, x, y):
    """Residual mixing + merge of the sublayer output: B.x_next."""
    ctx.postres_fwd(x, y, B.H_res, B.H_post, B.x_next)


def post_bwd(ctx: MhcLite, B: LayerBuffers, x, y, g, fused=True):
    """Backward of the merge: B.dy, B.dH_res, B.dH_post (and, unfused, the H_res^T g part of B.dx)."""
    skip_dx = fused                                # the fused tail recomputes H_res^T g from g
    ctx.postres_bwd(x, y, B.H_res, B.H_post, g, B.dy, B.dH_res, B.dH_post, None if skip_dx else B.dx, False)


def tail_bwd(ctx: MhcLite, P: LayerParams, B: LayerBuffers, x, g, du, eps=1e-6, fused=True, iters=20,
             accumulate_params=False):
    """Everything after the sublayer's backward: B.dx and the parameter gradients."""
    if B.kind == "sk" and fused:
        ctx.sk20_tail_bwd_fused(x, P.W, P.b, P.alpha, P.gain, eps, iters, B.p_saved, B.rstd, B.H_res, B.H_pre, B.H_post,
                                g, du, B.dH_res, B.dH_post, B.dx, B.dW, B.db, B.dalpha, B.dgain, accumulate_params)
    elif B.kind == "sk":
        ctx.premix_bwd(x, B.H_pre, du, B.dH_pre, B.dx, True)
        ctx.sk20_coeffs_bwd(x, P.W, P.b, P.alpha, P.gain, eps, iters, B.p_saved, B.rstd, B.H_pre, B.H_post,
                            B.dH_res, B.dH_pre, B.dH_post, B.dx, True, B.dW, B.db, B.dalpha, B.dgain,
                            accumulate_params)
    elif fused:
        ctx.tail_bwd_fused(x, P.W, P.alpha, P.gain, eps, B.a_saved, B.p_saved, B.rstd, B.H_res, B.H_pre, B.H_post,
                           g, du, B.dH_res, B.dH_post, B.dx, B.dW, B.db, B.dalpha, B.dgain, accumulate_params)
    else:
        ctx.premix_bwd(x, B.H_pre, du, B.dH_pre, B.dx, True)
        ctx.coeffs_bwd(x, P.W, P.alpha, P.gain, eps, B.a_saved, B.p_saved, B.rstd, B.H_pre, B.H_post,
                       B.dH_res, B.dH_pre, B.dH_post, B.dx, True, B.dW, B.db, B.dalpha, B.dgain, accumulate_params)


def stack_fwd(ctx: MhcLite, Ps, Bs, x0, sublayer, eps=1e-6, fuse_layers=True):
    """Forward through len(Ps) layers (the paper's models are 6, 12 or 24 of them back to back): layer l reads the
    x_next of layer l - 1.  `sublayer(l, u)` is the caller's f and returns y [T,C] bf16.  Each layer's input, y
    and outputs stay in its LayerBuffers for the backward.  With fuse_layers the merge of layer l also produces the
    projection of layer l + 1 (mhclite_postres_fwd_next_proj / mhclite_pre_fwd_resume), so x_{l+1} is read once less.
    The sublayer must not call workspace-using entry points of `ctx` in between.  Returns the last layer's x_next."""
    x = x0
    resumed = False
    for l, (P, B) in enumerate(zip(Ps, Bs)):
        B.x_in = x
        if resumed:       # this layer's projection came out of the merge kernel of the layer before
            ctx.pre_fwd_resume(x, P.b, P.alpha, eps, B.H_res, B.H_pre, B.H_post, B.a_saved, B.p_saved, B.rstd, B.u)
        else:
            pre_fwd(ctx, P, B, x, eps, True)
        B.y = sublayer(l, B.u)
        resumed = fuse_layers and l + 1 < len(Ps) and B.kind == "lite"
        if resumed:
            ctx.postres_fwd_next_proj(x, B.y, B.H_res, B.H_post, B.x_next, Ps[l + 1].W, Ps[l + 1].gain)
        else:
            post_fwd(ctx, B, x, B.y)
        x = B.x_next
    return x


def stack_bwd(ctx: MhcLite, Ps, Bs, g_top, sublayer_bwd, eps=1e-6):
    """Backward through the stack: `sublayer_bwd(l, u, dy)` is the caller's backward of f and returns du [T,C] bf16.
    Returns dL/dx_0; each layer's parameter gradients are in its LayerBuffers."""
    g = g_top
    for l in reversed(range(len(Ps))):
        P, B = Ps[l], Bs[l]
        B.g_in = g
        post_bwd(ctx, B, B.x_in, B.y, g, True)
        B.du = sublayer_bwd(l, B.u, B.dy)
        tail_bwd(ctx, P, B, B.x_in, g, B.du, eps, True)
        g = B.dx
    return g
