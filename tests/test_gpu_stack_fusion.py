"""Layer-to-layer fusion: the merge of layer l (Eq. (1)) fused with the RMSNorm statistics and projection of
layer l+1 (Eq. (4)), mhclite_postres_fwd_next_proj + mhclite_pre_fwd_resume, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import mhclite_oracle as O
from paper_2601_05732_b200 import synth
from paper_2601_05732_b200 import layer as L
from paper_2601_05732_b200.binding import MhcLite, ERR_BAD_ARG
from parity_utils import DEV, check_bf16, check_f32, host, p_tolerance

pytestmark = pytest.mark.gpu

# (n, C, T): tiles of fewer than 128 tokens, ragged last tiles, several tiles per CTA (T > 148 * 128), one
# channel block, and shapes the fused kernel does not take (n = 5, C not a multiple of 64: the un-fused route)
CASES = [(4, 256, 333), (3, 192, 700), (2, 128, 300), (4, 2048, 1100), (4, 64, 20000), (4, 1024, 257),
         (5, 136, 161), (4, 264, 130)]


@pytest.mark.parametrize("n,C,T", CASES)
def test_merge_with_next_projection(n, C, T):
    eps = 1e-6
    a = synth.make_layer_inputs(n, C, T, seed=50 + n, bias_std=0.5, alpha=[1.0, 0.7, 1.3], w_std=0.05, gain_std=0.1)
    nxt = synth.make_layer_params(n, C, seed=51 + n, layer=1, bias_std=0.5, alpha=[1.0, 0.7, 1.3], w_std=0.05, gain_std=0.2)
    ctx = MhcLite(n, C, 0)
    P0 = L.LayerParams(a["W"], a["b"], a["alpha"], a["gain"], DEV)
    P1 = L.LayerParams(nxt["W"], nxt["b"], nxt["alpha"], nxt["gain"], DEV)
    B0, B1 = L.LayerBuffers(ctx, T), L.LayerBuffers(ctx, T)
    x = L.to_device_bf16(a["x"], DEV); y = L.to_device_bf16(a["y"], DEV)
    L.pre_fwd(ctx, P0, B0, x, eps, True)
    ctx.postres_fwd_next_proj(x, y, B0.H_res, B0.H_post, B0.x_next, P1.W, P1.gain)
    ctx.pre_fwd_resume(B0.x_next, P1.b, P1.alpha, eps, B1.H_res, B1.H_pre, B1.H_post, B1.a_saved, B1.p_saved, B1.rstd, B1.u)
    torch.cuda.synchronize()
    ctx.device_status()
    f = synth.bf16_bits_to_f64
    w0 = [a[k].astype(np.float64) for k in ("W", "b", "alpha", "gain")]
    fw0 = O.layer_fwd(f(a["x"]), f(a["y"]), *w0, eps)
    check_bf16("x_next", host(B0.x_next), fw0["x_next"])
    # layer 1 on the x_next the GPU stored (teacher-forced: bf16 storage between the layers)
    xn = host(B0.x_next)
    w1 = [nxt[k].astype(np.float64) for k in ("W", "b", "alpha", "gain")]
    co = O.coeffs_fwd(xn, *w1, eps)
    check_f32("rstd", host(B1.rstd), co["rstd"], 1e-5)
    check_f32("p_saved", host(B1.p_saved), co["p"], 2e-4)
    check_f32("p_saved", host(B1.p_saved), co["p"], max(2e-5, p_tolerance(n * C)))
    for k, got in (("H_res", B1.H_res), ("H_pre", B1.H_pre), ("H_post", B1.H_post), ("a_saved", B1.a_saved)):
        check_f32(k, host(got), co["a" if k == "a_saved" else k], 2e-4)
    check_bf16("u", host(B1.u), O.premix_fwd(xn, co["H_pre"]))
    # same results as the un-fused sequence on the same x_next, up to the summation order of the contraction (these
    # logits are sharp: alpha = 1, so 1e-5 in a logit shows at that size in the mappings)
    B2 = L.LayerBuffers(ctx, T)
    L.pre_fwd(ctx, P1, B2, B0.x_next, eps, True)
    torch.cuda.synchronize()
    assert float((B2.H_res - B1.H_res).abs().max()) < 5e-5 and float((B2.rstd - B1.rstd).abs().max()) < 1e-5 * float(B2.rstd.max())


def test_resume_needs_pending_partials():
    n, C, T = 4, 64, 16
    a = synth.make_layer_inputs(n, C, T, seed=5)
    ctx = MhcLite(n, C, 0)
    P = L.LayerParams(a["W"], a["b"], a["alpha"], a["gain"], DEV)
    B = L.LayerBuffers(ctx, T)
    x = L.to_device_bf16(a["x"], DEV); y = L.to_device_bf16(a["y"], DEV)
    args = lambda xx: (ctx._h, T, xx.data_ptr(), P.b.data_ptr(), P.alpha.data_ptr(), 1e-6, B.H_res.data_ptr(), B.H_pre.data_ptr(),
                       B.H_post.data_ptr(), B.a_saved.data_ptr(), B.p_saved.data_ptr(), B.rstd.data_ptr(), B.u.data_ptr(), None)
    assert ctx.lib.mhclite_pre_fwd_resume(*args(x)) == ERR_BAD_ARG            # nothing pending
    L.pre_fwd(ctx, P, B, x)
    ctx.postres_fwd_next_proj(x, y, B.H_res, B.H_post, B.x_next, P.W, P.gain)
    assert ctx.lib.mhclite_pre_fwd_resume(*args(x)) == ERR_BAD_ARG            # pending for x_next, not for x
    assert ctx.lib.mhclite_pre_fwd_resume(*args(B.x_next)) == 0
    assert ctx.lib.mhclite_pre_fwd_resume(*args(B.x_next)) == ERR_BAD_ARG     # consumed
    # in-place merge is refused
    assert ctx.lib.mhclite_postres_fwd_next_proj(ctx._h, T, x.data_ptr(), y.data_ptr(), B.H_res.data_ptr(), B.H_post.data_ptr(),
                                                 x.data_ptr(), P.W.data_ptr(), P.gain.data_ptr(), None) == ERR_BAD_ARG
    torch.cuda.synchronize()


@pytest.mark.parametrize("Ld", [2, 5])
def test_fused_stack_matches_oracle_stack(Ld):
    # a small stack through layer.stack_fwd / stack_bwd with the fusion on, against the oracle's stack (bf16 storage)
    n, C, T, eps = 4, 128, 300, 1e-6
    params = [synth.make_layer_params(n, C, 7, layer=l, bias_std=0.3, alpha=[0.5, 0.5, 0.5], w_std=0.05) for l in range(Ld)]
    Ps = [L.LayerParams(p["W"], p["b"], p["alpha"], p["gain"], DEV) for p in params]
    ctx = MhcLite(n, C, 0)
    Bs = [L.LayerBuffers(ctx, T) for _ in range(Ld)]
    x0 = synth.normal_bf16(7, 0, (T, n, C)); gtop = synth.normal_bf16(7, 2, (T, n, C))

    def standin(u):
        uf = u.float()
        return (uf * torch.rsqrt(uf.pow(2).mean(-1, keepdim=True) + eps)).to(torch.bfloat16)

    def standin_bwd(u, dy):
        uf, d = u.float(), dy.float()
        r = torch.rsqrt(uf.pow(2).mean(-1, keepdim=True) + eps)
        return (r * d - uf * r.pow(3) * (uf * d).sum(-1, keepdim=True) / C).to(torch.bfloat16)

    out = L.stack_fwd(ctx, Ps, Bs, L.to_device_bf16(x0, DEV), lambda l, u: standin(u), eps, fuse_layers=True)
    dx0 = L.stack_bwd(ctx, Ps, Bs, L.to_device_bf16(gtop, DEV), lambda l, u, dy: standin_bwd(u, dy), eps)
    torch.cuda.synchronize()
    ctx.device_status()
    f = synth.bf16_bits_to_f64
    st = O.stack_fwd_bwd(f(x0), [tuple(p[k].astype(np.float64) for k in ("W", "b", "alpha", "gain")) for p in params],
                         f(gtop), eps, bf16_storage=True)
    # single bf16 rounding flips compound from layer to layer: rms-level agreement end to end ...
    rms = lambda v: float(np.sqrt(np.mean(v * v)))
    assert rms(host(out) - st["xs"][Ld]) <= 0.01 * rms(st["xs"][Ld])
    assert rms(host(dx0) - st["dx0"]) <= 0.02 * rms(st["dx0"])
    # ... and element by element for every layer when the oracle is fed what the GPU layer was fed
    for l in range(Ld):
        p = [params[l][k].astype(np.float64) for k in ("W", "b", "alpha", "gain")]
        fw = O.layer_fwd(host(Bs[l].x_in), host(Bs[l].y), *p, eps)
        check_f32(f"H_res[{l}]", host(Bs[l].H_res), fw["H_res"], 1e-4)
        check_bf16(f"u[{l}]", host(Bs[l].u), fw["u"])
        check_bf16(f"x_next[{l}]", host(Bs[l].x_next), fw["x_next"])
