"""Helpers of the GPU parity tests: run the CUDA path through the C ABI, run the oracle on the same host
inputs, and compare element by element with the stated tolerances.

Tolerances (they follow the arithmetic: bf16 storage rounds to 2^-9 relative, fp32 accumulation over
n*C <= 2^15 terms leaves ~1e-6 relative):
  bf16 tensors : |gpu - ref| <= 2e-2 |ref| + 1e-3 rms(ref)          for every element
  fp32 mappings: |gpu - ref| <= 1e-5 max(|ref|, rms(ref))           (H_res, H_pre, H_post, a, rstd)
  saved projection p = x' W: p_tolerance(nC) max(|ref|, rms(ref)) = 2^-16 + (nC / 16) 2^-24 -- W' enters the
                tensor cores as a bf16 pair hi + lo (16 mantissa bits: 2^-17 relative per weight) and the
                tensor cores add each 16-deep k-step to the fp32 accumulator with up to one unit in the last
                place lost (nC / 16 steps).  Measured: 1.0e-5 at nC = 4096, 3.8e-5 at nC = 7680, 4.9e-5 at
                nC = 16384.  alpha scales this down by 100x before it reaches the mappings, checked at 1e-5
  fp32 parameter gradients: |gpu - ref| <= 1e-3 max(|ref|, rms(ref)) (the binding tolerance is 2e-2)
"""
import numpy as np
import torch

from oracle import mhclite_oracle as O
from paper_2601_05732_b200 import synth
from paper_2601_05732_b200.binding import MhcLite
from paper_2601_05732_b200 import layer as L

DEV = "cuda:0"


def p_tolerance(nC):
    """Relative tolerance of the saved projection for a contraction over nC terms (see the module docstring)."""
    return 2.0 ** -16 + (nC / 16) * 2.0 ** -24


def rms(a):
    a = np.asarray(a, dtype=np.float64)
    return float(np.sqrt(np.mean(a * a))) if a.size else 0.0


RECORDS = []     # raw error figures of every comparison made in this session (written out by conftest.py)


def _record(name, kind, got, ref, tol, tol_plain):
    """Raw figures of one comparison: max relative error over the elements with |ref| >= rms/16, max
    absolute error over rms, and the worst error as a fraction of the tolerance, with and without the
    per-element allowance (`extra`) -- so that neither the floor term nor an allowance can hide anything."""
    import os
    err = np.abs(got - ref)
    r = rms(ref)
    big = np.abs(ref) >= r / 16 if r > 0 else np.zeros(ref.shape, dtype=bool)
    rec = dict(test=os.environ.get("PYTEST_CURRENT_TEST", "").split(" ")[0], tensor=name, kind=kind, size=int(ref.size),
               rms=r, max_abs_err=float(err.max()) if err.size else 0.0,
               max_abs_err_over_rms=float(err.max() / r) if (err.size and r > 0) else 0.0,
               max_rel_err_big=float((err[big] / np.abs(ref[big])).max()) if big.any() else 0.0,
               worst_over_tol=float((err / tol).max()) if err.size else 0.0,
               worst_over_tol_no_extra=float((err / tol_plain).max()) if err.size else 0.0)
    RECORDS.append(rec)
    return rec


def check_bf16(name, got, ref, rel=2e-2, floor=1e-3, extra=0.0):
    """`extra` (per element) allows for a tensor that was stored in bf16 on the way: one rounding of
    an intermediate v moves the result by up to 2^-8 |v|, whatever the size of the final value."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    plain = rel * np.abs(ref) + floor * rms(ref) + 1e-300
    tol = plain + extra
    rec = _record(name, "bf16", got, ref, tol, plain)
    bad = np.abs(got - ref) > tol
    assert not bad.any(), f"{name}: {bad.sum()} of {bad.size} elements off; worst {np.abs(got - ref).max():.3e} (rms {rms(ref):.3e})"
    return rec


def check_f32(name, got, ref, rel=1e-5):
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    tol = rel * np.maximum(np.abs(ref), rms(ref)) + 1e-30
    err = np.abs(got - ref)
    rec = _record(name, "f32@%g" % rel, got, ref, tol, tol)
    assert (err <= tol).all(), f"{name}: worst err/tol {np.max(err / tol):.2f}, max abs err {err.max():.3e}, rms {rms(ref):.3e}"
    return rec


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


class GpuLayer:
    """Uploads one layer's host inputs and runs the library's call sequence on them."""

    def __init__(self, inp, eps=1e-6, kind="lite", iters=20, table=None):
        self.inp, self.eps, self.kind, self.iters = inp, eps, kind, iters
        n, C, T = inp["n"], inp["C"], inp["T"]
        self.ctx = MhcLite(n, C, 0)
        if table is not None:                       # a subset of the permutations (paper Section 5)
            self.table = torch.from_numpy(np.ascontiguousarray(table, dtype=np.uint8)).to(DEV)
            self.ctx.set_perm_subset(self.table)
        self.P = L.LayerParams(inp["W"], inp["b"], inp["alpha"], inp["gain"], DEV)
        self.B = L.LayerBuffers(self.ctx, T, kind)
        self.x = L.to_device_bf16(inp["x"], DEV); self.y = L.to_device_bf16(inp["y"], DEV)
        self.g = L.to_device_bf16(inp["g"], DEV); self.du = L.to_device_bf16(inp["du"], DEV)

    def forward(self, fused=True):
        L.pre_fwd(self.ctx, self.P, self.B, self.x, self.eps, fused, self.iters)
        L.post_fwd(self.ctx, self.B, self.x, self.y)
        torch.cuda.synchronize()

    def backward(self, fused=True, accumulate_params=False):
        L.post_bwd(self.ctx, self.B, self.x, self.y, self.g, fused)
        L.tail_bwd(self.ctx, self.P, self.B, self.x, self.g, self.du, self.eps, fused, self.iters, accumulate_params)
        torch.cuda.synchronize()


def oracle_inputs(inp):
    f = synth.bf16_bits_to_f64
    return dict(x=f(inp["x"]), y=f(inp["y"]), g=f(inp["g"]), du=f(inp["du"]),
                W=inp["W"].astype(np.float64), b=inp["b"].astype(np.float64),
                alpha=inp["alpha"].astype(np.float64), gain=inp["gain"].astype(np.float64))


def oracle_fwd(inp, eps=1e-6, kind="lite", iters=20, table=None):
    o = oracle_inputs(inp)
    return O.layer_fwd(o["x"], o["y"], o["W"], o["b"], o["alpha"], o["gain"], eps, kind=kind, iters=iters, table=table)


def oracle_bwd(inp, eps=1e-6, kind="lite", iters=20, table=None):
    o = oracle_inputs(inp)
    return O.layer_bwd(o["x"], o["y"], o["W"], o["b"], o["alpha"], o["gain"], eps, o["g"], o["du"], kind=kind, iters=iters,
                       table=table)


def compare_forward(G, ref, coeff_rel=1e-5):
    B = G.B
    check_f32("rstd", host(B.rstd), ref["rstd"], coeff_rel)
    check_f32("p_saved", host(B.p_saved), ref["p"], max(coeff_rel, p_tolerance(G.ctx.n * G.ctx.C)))
    if G.kind == "lite":
        check_f32("a_saved", host(B.a_saved), ref["a"], coeff_rel)
    check_f32("H_res", host(B.H_res), ref["H_res"], coeff_rel)
    check_f32("H_pre", host(B.H_pre), ref["H_pre"], coeff_rel)
    check_f32("H_post", host(B.H_post), ref["H_post"], coeff_rel)
    check_bf16("u", host(B.u), ref["u"])
    check_bf16("x_next", host(B.x_next), ref["x_next"])


def staged_dx_allowance(ref, fused):
    """dx is stored in bf16 between the calls that add to it: each stored intermediate v may round
    the other way on the GPU (fp32 sums) than in fp64, which moves dx by up to 2^-8 |v|."""
    d2 = ref["dx"] - ref["dx_coeffs"]                     # after H_res^T g + H_pre du
    if fused:
        return 0.0                                        # the fused tail writes dx once
    d1 = d2 - ref["dx_premix"]                            # after H_res^T g
    return 2.0 ** -8 * (np.abs(d1) + np.abs(d2))


def dxhat_allowance_f(x, W, alpha, gain, dz, eps=1e-6):
    """Allowance for the projection-backward term of dx, sum_c e[t,c] W'[m,c]: the tensor-core kernel
    rounds both operands to bf16 (as bf16 mixed-precision training does for this matmul).  bf16 keeps 8
    significant bits, so rounding to nearest moves an operand by up to 2^-8 of its size and a product of
    two rounded operands by up to 2^-7: |error| <= 2^-7 sum_c |e[t,c]| |W'[m,c]|.  Only the stress cases
    (sharp logits, the mappings' gradient in isolation) use it; the five workloads pass without."""
    T, n, C = x.shape
    xh = x.reshape(T, n * C)
    rstd = 1.0 / np.sqrt((xh * xh).mean(axis=1) + eps)
    n_res = dz.shape[1] - 2 * n
    av = np.concatenate([np.full(n_res, alpha[0]), np.full(n, alpha[1]), np.full(n, alpha[2])])
    e = np.abs(rstd[:, None] * av * dz)
    Wp = np.abs(gain[:, None] * W)
    return 2.0 ** -7 * (e @ Wp.T).reshape(T, n, C)


def dxhat_allowance(inp, dz, eps=1e-6):
    o = oracle_inputs(inp)
    return dxhat_allowance_f(o["x"], o["W"], o["alpha"], o["gain"], dz, eps)


def compare_backward(G, ref, grad_rel=1e-3, fused=True):
    B = G.B
    check_bf16("dy", host(B.dy), ref["dy"])
    check_f32("dH_res", host(B.dH_res), ref["dH_res"], 2e-5)
    check_f32("dH_post", host(B.dH_post), ref["dH_post"], 2e-5)
    check_bf16("dx", host(B.dx), ref["dx"], extra=staged_dx_allowance(ref, fused) + dxhat_allowance(G.inp, ref["dz"], G.eps))
    check_f32("dW", host(B.dW), ref["dW"], grad_rel)
    check_f32("db", host(B.db), ref["db"], grad_rel)
    check_f32("dalpha", host(B.dalpha), ref["dalpha"], grad_rel)
    check_f32("dgain", host(B.dgain), ref["dgain"], grad_rel)
