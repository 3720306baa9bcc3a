"""The allocation-free entry point, mhclite_coeffs_bwd_static, against mhclite_coeffs_bwd.

Some users of the library cannot allocate device memory where they call it (inside an allocator
callback, under a fixed memory budget, as a plug-in that only sees inputs and outputs), so they cannot
attach a workspace.  This entry point keeps its scratch in a fixed array inside the library instead.
The test calls it through the C ABI on a context that never had a workspace, twice in a row (the array
keeps the first call's contents: the second call must not be disturbed by them), and compares every
output with the workspace-based entry point within the tolerances the other GPU tests use.  It also
checks that a problem too large for the array is refused with a clear message and no launch.

This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2601_05732_b200 import synth
from paper_2601_05732_b200.binding import MhcLite, ERR_WORKSPACE, load
from oracle import mhclite_oracle as O
from parity_utils import DEV, GpuLayer, check_bf16, check_f32, dxhat_allowance, host, oracle_inputs

pytestmark = pytest.mark.gpu


def _scratch_need(n, C, T):
    """Scratch the static entry point takes from its array (the formula of its header comment)."""
    import math
    Np = (math.factorial(n) + 2 * n + 7) // 8 * 8
    return 4 * (T * Np + T + n * C * Np) + 3 * 256


def _upstream(G, seed):
    """Synthetic upstream gradients of the mappings (what postres_bwd / premix_bwd would hand over)."""
    n, T = G.ctx.n, G.inp["T"]
    f = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV)
    return (f(synth.normal(seed, 50, (T, n, n), 8.0)), f(synth.normal(seed, 51, (T, n), 8.0)),
            f(synth.normal(seed, 52, (T, n), 8.0)))


@pytest.mark.parametrize("n,C,T", [(4, 256, 700), (3, 72, 130), (5, 40, 70)])
def test_static_scratch_matches_workspace_entry_point_twice(n, C, T):
    assert _scratch_need(n, C, T) <= load().mhclite_static_scratch_bytes()
    outs = []
    for call, seed in enumerate((61, 62)):           # two calls in a row, different data
        inp = synth.make_layer_inputs(n, C, T, seed=seed, bias_std=0.5, alpha=[1.0, 1.0, 1.0], w_std=0.05)
        G = GpuLayer(inp)                             # reference context: has a workspace
        G.forward(False)
        B, P = G.B, G.P
        dHr, dHp, dHo = _upstream(G, seed)
        ref = {}
        G.ctx.coeffs_bwd(G.x, P.W, P.alpha, P.gain, 1e-6, B.a_saved, B.p_saved, B.rstd, B.H_pre, B.H_post,
                         dHr, dHp, dHo, B.dx, False, B.dW, B.db, B.dalpha, B.dgain, False)
        torch.cuda.synchronize()
        for k in ("dx", "dW", "db", "dalpha", "dgain"):
            ref[k] = host(getattr(B, k)).copy()

        bare = MhcLite(n, C)                          # never given a workspace
        dx = torch.full_like(B.dx, float("nan")); dW = torch.full_like(B.dW, float("nan"))
        db = torch.full_like(B.db, float("nan")); dal = torch.full((4,), float("nan"), device=DEV)[:3]
        dg = torch.full_like(B.dgain, float("nan"))
        args = (G.x, P.W, P.alpha, P.gain, 1e-6, B.a_saved, B.p_saved, B.rstd, B.H_pre, B.H_post, dHr, dHp, dHo)
        bare.coeffs_bwd_static(*args, dx, False, dW, db, dal, dg, False)
        torch.cuda.synchronize()
        assert bare._ws is None
        # against the workspace entry point: that one rounds the operands of sum_c e W' to bf16 (tensor
        # cores), this one keeps them in fp32; allow for that rounding exactly as the parity tests do
        o = oracle_inputs(inp)
        orc = O.coeffs_bwd(o["x"], o["W"], o["b"], o["alpha"], o["gain"], 1e-6, host(dHr), host(dHp), host(dHo))
        check_bf16(f"dx vs workspace call (call {call})", host(dx), ref["dx"], extra=dxhat_allowance(inp, orc["dz"]))
        check_f32(f"dW vs workspace call (call {call})", host(dW), ref["dW"], 1e-3)
        check_f32(f"db vs workspace call (call {call})", host(db), ref["db"], 1e-3)
        check_f32(f"dalpha vs workspace call (call {call})", host(dal), ref["dalpha"], 1e-3)
        check_f32(f"dgain vs workspace call (call {call})", host(dg), ref["dgain"], 1e-3)
        # and against the oracle's gradient of the mappings itself (no allowance: fp32 operands here)
        check_bf16(f"dx vs oracle (call {call})", host(dx), orc["dx"])
        for k, got in (("dW", dW), ("db", db), ("dalpha", dal), ("dgain", dg)):
            check_f32(f"{k} vs oracle (call {call})", host(got), orc[k], 1e-3)
        assert np.abs(ref["dW"]).max() > 0 and np.isfinite(host(dx)).all()
        # both accumulate flags: a second call adds the same gradients on top
        bare.coeffs_bwd_static(*args, dx, True, dW, db, dal, dg, True)
        torch.cuda.synchronize()
        check_bf16(f"dx x2 (call {call})", host(dx), 2 * orc["dx"], rel=3e-2)
        for k, got in (("dW", dW), ("db", db), ("dalpha", dal), ("dgain", dg)):
            check_f32(f"{k} x2 (call {call})", host(got), 2 * orc[k], 1e-3)
        outs.append(ref["dW"])
    assert np.abs(outs[0] - outs[1]).max() > 0        # the two calls really computed different things


def test_static_scratch_rejects_oversized_problem():
    n, C, T = 4, 1024, 65536
    assert _scratch_need(n, C, T) > load().mhclite_static_scratch_bytes()
    ctx = MhcLite(n, C)
    z = torch.zeros(64, device=DEV)
    zb = torch.zeros(64, device=DEV, dtype=torch.bfloat16)
    p = z.data_ptr()
    rc = ctx.lib.mhclite_coeffs_bwd_static(ctx._h, T, zb.data_ptr(), p, p, p, 1e-6, p, p, p, p, p, p, p, p,
                                           zb.data_ptr(), 0, p, p, p, p, 0, None)
    assert rc == ERR_WORKSPACE
    msg = ctx.lib.mhclite_last_error(ctx._h).decode()
    assert "scratch" in msg and "mhclite_coeffs_bwd" in msg
    torch.cuda.synchronize()
