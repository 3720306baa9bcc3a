"""Element-by-element parity of the CUDA path (through the C ABI) with the fp64 oracle on the same
seeded inputs: sizes that span several tiles with ragged tails, every n, both call sequences."""
import math

import numpy as np
import pytest
import torch

from oracle import mhclite_oracle as O
from paper_2601_05732_b200 import synth
from paper_2601_05732_b200 import layer as L
from parity_utils import (DEV, GpuLayer, check_bf16, check_f32, compare_backward, compare_forward, dxhat_allowance,
                          host, oracle_bwd, oracle_fwd, oracle_inputs)

pytestmark = pytest.mark.gpu

CASES = [  # (n, C, T): ragged token tails (T not a multiple of 32/64/128) and ragged channel tails
    (4, 256, 333), (4, 264, 130), (2, 8, 77), (3, 72, 200), (5, 136, 161), (4, 1024, 257), (3, 1536, 65),
    (5, 320, 700),
    # fused tcgen05 tail (C a multiple of 64): n = 2, and several 128-token tiles per CTA with a ragged last tile
    (2, 128, 300), (4, 2048, 1100), (3, 1536, 2000),
]


@pytest.mark.parametrize("n,C,T", CASES)
@pytest.mark.parametrize("fused", [True, False])
def test_layer_parity(n, C, T, fused):
    inp = synth.make_layer_inputs(n, C, T, seed=10 + n, bias_std=0.1, gain_std=0.1)
    G = GpuLayer(inp)
    G.forward(fused)
    compare_forward(G, oracle_fwd(inp))
    G.backward(fused)
    compare_backward(G, oracle_bwd(inp), fused=fused)


@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_permutation_table_on_device_bit_exact(n):
    from paper_2601_05732_b200.binding import MhcLite
    got = MhcLite(n, 8).perm_table_device()
    assert (got == O.perm_table(n)).all()


@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_one_hot_weight_selects_each_permutation(n):
    # W = 0, b_res = 0 at k and -200 elsewhere: a = e_k and H_res = P_k exactly (fp32 exp underflows to 0)
    C, T = 64, 5
    nf = math.factorial(n)
    tab = O.perm_table(n)
    for k in range(nf):
        inp = synth.make_layer_inputs(n, C, T, seed=3)
        inp["W"][:] = 0
        inp["b"][:nf] = -200.0
        inp["b"][k] = 0.0
        G = GpuLayer(inp)
        G.forward()
        H = host(G.B.H_res)
        expect = np.zeros((n, n)); expect[np.arange(n), tab[k]] = 1.0
        assert (H == expect[None]).all(), k
        # x_next = P_k x + H_post y with H_post = 1 (b_post = 0): row i takes stream sigma_k(i)
        ref = oracle_fwd(inp)
        check_bf16("x_next", host(G.B.x_next), ref["x_next"])


def test_paper_initialisation_is_near_identity():
    n, C, T = 4, 128, 64
    inp = synth.make_layer_inputs(n, C, T, seed=4)
    inp["W"][:] = 0
    inp["b"][:] = synth.paper_init_bias(n)
    G = GpuLayer(inp); G.forward()
    ref = oracle_fwd(inp)
    compare_forward(G, ref)
    H = host(G.B.H_res)
    assert np.abs(H - np.eye(4)).max() < 24 * math.exp(-8.0)


@pytest.mark.parametrize("n", [3, 4, 5])
def test_sharp_logits(n):
    # alpha = 1 and a wide bias: the softmax is far from uniform, so a wrong permutation mapping or
    # a wrong column group shows at first order.  fp32 accumulation over n*C terms of |p| ~ 5 leaves
    # ~1e-5 absolute in the logits, hence the looser coefficient tolerance here.
    C, T = 256, 150
    inp = synth.make_layer_inputs(n, C, T, seed=20 + n, bias_std=2.0, alpha=[1.0, 0.7, 1.3], w_std=0.05, gain_std=0.2)
    G = GpuLayer(inp)
    G.forward(); compare_forward(G, oracle_fwd(inp), coeff_rel=2e-4)
    G.backward(); compare_backward(G, oracle_bwd(inp), grad_rel=2e-3)
    Hr = host(G.B.H_res)
    assert np.abs(Hr.sum(1) - 1).max() < 1e-6 and np.abs(Hr.sum(2) - 1).max() < 1e-6 and Hr.min() >= 0
    assert Hr.std() > 0.05     # genuinely non-uniform


def test_coeffs_bwd_in_isolation():
    # the gradient through the mappings is ~0.5 % of dx at the benchmark's distributions: check it alone
    n, C, T = 4, 256, 200
    inp = synth.make_layer_inputs(n, C, T, seed=31, bias_std=0.5, alpha=[1.0, 1.0, 1.0], w_std=0.05)
    G = GpuLayer(inp); G.forward(False)
    ref = oracle_bwd(inp)
    B, P = G.B, G.P
    f = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV)
    dHr, dHp, dHo = f(ref["dH_res"]), f(ref["dH_pre"]), f(ref["dH_post"])
    G.ctx.coeffs_bwd(G.x, P.W, P.alpha, P.gain, 1e-6, B.a_saved, B.p_saved, B.rstd, B.H_pre, B.H_post,
                     dHr, dHp, dHo, B.dx, False, B.dW, B.db, B.dalpha, B.dgain, False)
    torch.cuda.synchronize()
    allow = dxhat_allowance(inp, ref["dz"])
    check_bf16("dx_coeffs", host(B.dx), ref["dx_coeffs"], extra=allow)
    check_f32("dW", host(B.dW), ref["dW"], 1e-3)
    check_f32("dgain", host(B.dgain), ref["dgain"], 1e-3)
    check_f32("db", host(B.db), ref["db"], 1e-3)
    check_f32("dalpha", host(B.dalpha), ref["dalpha"], 1e-3)
    # accumulate_params adds to what is there
    G.ctx.coeffs_bwd(G.x, P.W, P.alpha, P.gain, 1e-6, B.a_saved, B.p_saved, B.rstd, B.H_pre, B.H_post,
                     dHr, dHp, dHo, B.dx, True, B.dW, B.db, B.dalpha, B.dgain, True)
    torch.cuda.synchronize()
    check_f32("dW x2", host(B.dW), 2 * ref["dW"], 1e-3)
    check_f32("db x2", host(B.db), 2 * ref["db"], 1e-3)
    check_f32("dalpha x2", host(B.dalpha), 2 * ref["dalpha"], 1e-3)
    check_f32("dgain x2", host(B.dgain), 2 * ref["dgain"], 1e-3)
    check_bf16("dx x2", host(B.dx), 2 * ref["dx_coeffs"], rel=3e-2, extra=2 * allow)


@pytest.mark.parametrize("T", [0, 1, 2, 31, 33])
def test_tiny_and_empty_token_counts(T):
    n, C = 4, 64
    inp = synth.make_layer_inputs(n, C, max(T, 1), seed=5, bias_std=0.1)
    if T == 0:
        from paper_2601_05732_b200.binding import MhcLite
        ctx = MhcLite(n, C)
        e = torch.empty(0, device=DEV)
        # T = 0 is a valid no-op: pointers are not even inspected
        assert ctx.lib.mhclite_premix_fwd(ctx._h, 0, None, None, None, None) == 0
        assert ctx.lib.mhclite_postres_fwd(ctx._h, 0, None, None, None, None, None, None) == 0
        return
    G = GpuLayer(inp)
    G.forward(); compare_forward(G, oracle_fwd(inp))
    G.backward(); compare_backward(G, oracle_bwd(inp))


def test_bad_arguments_are_rejected_without_launch():
    from paper_2601_05732_b200.binding import MhcLite, MhcLiteError, ERR_BAD_ARG, ERR_WORKSPACE
    n, C, T = 4, 64, 16
    inp = synth.make_layer_inputs(n, C, T, seed=5)
    G = GpuLayer(inp)
    lib, h = G.ctx.lib, G.ctx._h
    x = G.x.data_ptr()
    assert lib.mhclite_premix_fwd(h, -1, x, G.B.H_pre.data_ptr(), G.B.u.data_ptr(), None) == ERR_BAD_ARG
    assert lib.mhclite_premix_fwd(h, T, None, G.B.H_pre.data_ptr(), G.B.u.data_ptr(), None) == ERR_BAD_ARG
    assert lib.mhclite_premix_fwd(h, T, x + 2, G.B.H_pre.data_ptr(), G.B.u.data_ptr(), None) == ERR_BAD_ARG
    assert b"aligned" in lib.mhclite_last_error(h)
    # in-place use is refused (outputs must not alias inputs)
    assert lib.mhclite_postres_fwd(h, T, x, G.y.data_ptr(), G.B.H_res.data_ptr(), G.B.H_post.data_ptr(), x, None) == ERR_BAD_ARG
    assert b"alias" in lib.mhclite_last_error(h)
    assert lib.mhclite_postres_bwd(h, T, x, G.y.data_ptr(), G.B.H_res.data_ptr(), G.B.H_post.data_ptr(), G.g.data_ptr(),
                                   G.B.dy.data_ptr(), G.B.dH_res.data_ptr(), G.B.dH_post.data_ptr(), G.g.data_ptr(), 0, None) == ERR_BAD_ARG
    # a context without workspace refuses the calls that need one
    ctx2 = MhcLite(n, C)
    B = G.B
    with pytest.raises(MhcLiteError) as ei:
        ctx2._check(ctx2.lib.mhclite_coeffs_bwd(
            ctx2._h, T, x, G.P.W.data_ptr(), G.P.alpha.data_ptr(), G.P.gain.data_ptr(), 1e-6, B.a_saved.data_ptr(),
            B.p_saved.data_ptr(), B.rstd.data_ptr(), B.H_pre.data_ptr(), B.H_post.data_ptr(), B.dH_res.data_ptr(),
            B.dH_pre.data_ptr(), B.dH_post.data_ptr(), B.dx.data_ptr(), 0, B.dW.data_ptr(), B.db.data_ptr(),
            B.dalpha.data_ptr(), B.dgain.data_ptr(), 0, None), "coeffs_bwd")
    assert ei.value.status == ERR_WORKSPACE
    torch.cuda.synchronize()


# ------------------------------------------------------------------ SK comparison path (Eq. (2))
@pytest.mark.parametrize("n,C,T", [(4, 256, 300), (3, 72, 100), (2, 64, 50), (5, 40, 70)])
@pytest.mark.parametrize("fused", [True, False])
def test_sk_path_parity(n, C, T, fused):
    inp = synth.make_layer_inputs(n, C, T, seed=40 + n, bias_std=0.5, alpha=[1.0, 1.0, 1.0], w_std=0.05, kind="sk")
    G = GpuLayer(inp, kind="sk")
    G.forward(fused); compare_forward(G, oracle_fwd(inp, kind="sk"), coeff_rel=1e-4)
    G.backward(fused); compare_backward(G, oracle_bwd(inp, kind="sk"), grad_rel=2e-3, fused=fused)


def test_sk_gap_vs_lite_on_ill_conditioned_logits():
    # paper Section 3.1: with a large relative range 1/nu, 20 iterations leave a visible gap; mHC-lite none
    n, C, T = 4, 256, 4096
    sk = synth.make_layer_inputs(n, C, T, seed=6, kind="sk")
    sk["b"][:16] = synth.normal(6, 99, (16,), 10.0).astype(np.float32)
    G = GpuLayer(sk, kind="sk"); G.forward()
    ref = oracle_fwd(sk, kind="sk")
    l1 = torch.empty(T, device=DEV); cd = torch.empty(T, device=DEV)
    G.ctx.ds_gap(G.B.H_res, l1, cd); torch.cuda.synchronize()
    gap_ref = O.l1_error(ref["H_res"])
    assert gap_ref.max() > 1e-3                                   # the oracle sees the gap ...
    check_f32("l1 gap", host(l1), gap_ref, 1e-2)                  # ... and the GPU path reproduces it
    check_f32("colsum dev", host(cd), np.abs(O.column_sums(ref["H_res"]) - 1).max(axis=1), 1e-2)
    lite = synth.make_layer_inputs(n, C, T, seed=6)
    lite["b"][:24] = synth.normal(6, 98, (24,), 10.0).astype(np.float32)
    GL = GpuLayer(lite); GL.forward()
    GL.ctx.ds_gap(GL.B.H_res, l1, cd); torch.cuda.synchronize()
    assert float(l1.max()) < 4e-6 and float(cd.max()) < 1e-6


def test_sk_gap_with_the_papers_initialisation_bias():
    # Section 4, "Initialization": b_res = -8 off the diagonal, 0 on it (mHC); -8 / 0 at the identity (mHC-lite).
    # With W != 0 at alpha = 1 the logits spread around that pattern; the SK path's gap must match the oracle's,
    # mHC-lite has none.
    n, C, T = 4, 256, 4096
    sk = synth.make_layer_inputs(n, C, T, seed=6, kind="sk", alpha=[1.0, 1.0, 1.0], w_std=0.1)
    sk["b"][:] = synth.paper_init_bias(n, "sk")
    G = GpuLayer(sk, kind="sk"); G.forward()
    ref = oracle_fwd(sk, kind="sk")
    compare_forward(G, ref, coeff_rel=1e-4)
    l1 = torch.empty(T, device=DEV); cd = torch.empty(T, device=DEV)
    G.ctx.ds_gap(G.B.H_res, l1, cd); torch.cuda.synchronize()
    gap_ref = O.l1_error(ref["H_res"])
    assert np.abs(host(l1) - gap_ref).max() <= 1e-2 * gap_ref.max() + 4e-6
    assert np.abs(host(cd) - np.abs(O.column_sums(ref["H_res"]) - 1).max(axis=1)).max() <= 1e-2 * gap_ref.max() + 4e-6
    nu = torch.empty(T, device=DEV)
    M0 = torch.from_numpy(np.ascontiguousarray(ref["M0"], dtype=np.float32)).to(DEV)
    G.ctx.relative_range(M0, nu); torch.cuda.synchronize()
    np.testing.assert_allclose(host(nu), O.relative_range(ref["M0"].astype(np.float32).astype(np.float64)), rtol=1e-6)
    lite = synth.make_layer_inputs(n, C, T, seed=6, alpha=[1.0, 1.0, 1.0], w_std=0.1)
    lite["b"][:] = synth.paper_init_bias(n)
    GL = GpuLayer(lite); GL.forward()
    compare_forward(GL, oracle_fwd(lite), coeff_rel=2e-4)
    GL.ctx.ds_gap(GL.B.H_res, l1, cd); torch.cuda.synchronize()
    assert float(cd.max()) < 1e-6 and float(l1.max()) < 2 * n * 1e-6       # 2n row / column sums, each within 1e-6


def test_kernel_timing_and_device_status():
    # the library's own per-kernel events and its device status word (bounded waits record a status there)
    n, C, T = 4, 256, 2048
    inp = synth.make_layer_inputs(n, C, T, seed=8, bias_std=0.1)
    G = GpuLayer(inp)
    G.ctx.set_kernel_timing(True)
    G.forward(True); G.backward(True)
    torch.cuda.synchronize()
    times = [G.ctx.kernel_time_ms(i) for i in range(len(G.ctx.KERNELS))]
    assert all(0.0 < t < 50.0 for t in times), times
    G.ctx.set_kernel_timing(False)
    G.ctx.device_status()                      # raises if any kernel gave up on a wait
    compare_forward(G, oracle_fwd(inp))


def test_kernel_timing_of_a_kernel_off_the_path_is_an_argument_error():
    # only the forward has run: the time of the backward tail is refused cleanly and later calls still work
    from paper_2601_05732_b200.binding import MhcLiteError
    n, C, T = 5, 64, 200
    inp = synth.make_layer_inputs(n, C, T, seed=9, bias_std=0.1)
    G = GpuLayer(inp)
    G.ctx.set_kernel_timing(True)
    G.forward(True)
    torch.cuda.synchronize()
    tail = G.ctx.KERNELS.index("tail_dx")
    with pytest.raises(MhcLiteError) as ei:
        G.ctx.kernel_time_ms(tail)
    assert ei.value.status == -1
    assert G.ctx.kernel_time_ms(0) > 0.0
    G.forward(True); torch.cuda.synchronize()
    compare_forward(G, oracle_fwd(inp))


@pytest.mark.parametrize("n,C,T", [(4, 128, 700), (3, 72, 130)])
def test_step_from_host_buffers(n, C, T):
    # the whole step through mhclite_step_host: pinned host activations in, host activations out, in chunks of
    # tokens whose copies and kernels overlap (700 tokens = three chunks, the last one ragged)
    inp = synth.make_layer_inputs(n, C, T, seed=40 + n, bias_std=0.1, gain_std=0.1)
    G = GpuLayer(inp)
    B, P = G.B, G.P
    pin = lambda t: t.cpu().pin_memory()
    hx, hy, hg, hdu = pin(G.x), pin(G.y), pin(G.g), pin(G.du)
    hu, hxn, hdy, hdx = (torch.zeros_like(t, device="cpu").pin_memory() for t in (B.u, B.x_next, B.dy, B.dx))
    run = lambda acc: G.ctx.step_host(hx, hy, hg, hdu, P.W, P.b, P.alpha, P.gain, 1e-6, hu, hxn, hdy, hdx,
                                      B.dW, B.db, B.dalpha, B.dgain, acc)
    run(False)
    torch.cuda.synchronize()
    fw, bw = oracle_fwd(inp), oracle_bwd(inp)
    f64 = lambda t: t.float().numpy().astype(np.float64)
    check_bf16("u", f64(hu), fw["u"])
    check_bf16("x_next", f64(hxn), fw["x_next"])
    check_bf16("dy", f64(hdy), bw["dy"])
    check_bf16("dx", f64(hdx), bw["dx"], extra=dxhat_allowance(inp, bw["dz"]))
    for name, got in (("dW", B.dW), ("db", B.db), ("dalpha", B.dalpha), ("dgain", B.dgain)):
        check_f32(name, host(got), bw[name], 1e-3)
    run(True)                                       # accumulate_params adds a second copy of the gradients
    torch.cuda.synchronize()
    for name, got in (("dW", B.dW), ("db", B.db), ("dalpha", B.dalpha), ("dgain", B.dgain)):
        check_f32(name + " x2", host(got), 2 * bw[name], 1e-3)
    check_bf16("dx again", f64(hdx), bw["dx"], extra=dxhat_allowance(inp, bw["dz"]))
    G.ctx.device_status()


@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_depth_product_and_relative_range(n):
    # Section 3.1 diagnostics in the library's kernels: prod_l H_l per token (later layers on the left) and
    # Eq. (3)'s nu, against the oracle on random doubly stochastic and random positive matrices
    T, depth = 300, 6
    rng = np.random.default_rng(60 + n)
    nf = math.factorial(n)
    Hs = [O.hres_from_weights(rng.dirichlet(np.ones(nf) * 0.3, size=T), n).astype(np.float32) for _ in range(depth)]
    ctx = GpuLayer(synth.make_layer_inputs(n, 8, 4, seed=1)).ctx
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV)
    P = torch.empty(T, n, n, device=DEV)
    for l, H in enumerate(Hs):
        ctx.depth_product(dev(H), P, first=(l == 0))
    torch.cuda.synchronize()
    ref = O.depth_product([H.astype(np.float64) for H in Hs])
    assert np.abs(host(P) - ref).max() < 1e-6
    l1 = torch.empty(T, device=DEV); ctx.ds_gap(P, l1, None); torch.cuda.synchronize()
    assert float(l1.max()) < depth * 4e-6                      # products of doubly stochastic matrices stay so
    X = rng.uniform(0.0, 1.0, size=(T, n, n)).astype(np.float32)
    X[rng.uniform(size=X.shape) < 0.2] = 0.0                   # zeros are skipped by Eq. (3)
    X[0] = 0.0                                                 # degenerate: no positive entry
    nu = torch.empty(T, device=DEV); ctx.relative_range(dev(X), nu); torch.cuda.synchronize()
    ok = X.reshape(T, -1).max(axis=1) > 0
    ref_nu = O.relative_range(X[ok].astype(np.float64))
    np.testing.assert_allclose(host(nu)[ok], ref_nu, rtol=1e-6)
    assert float(nu[0]) == 0.0


def test_gap_statistics_and_relative_range_histogram():
    # Section 3.1's population figures in one pass each: gap statistics of an SK output (Fig. 3's procedure) and the
    # histogram of log10(1/nu) of the SK input (Fig. 4's), against the oracle's per-token values
    n, C, T = 4, 64, 5000
    sk = synth.make_layer_inputs(n, C, T, seed=16, kind="sk", alpha=[1.0, 1.0, 1.0], w_std=0.3)
    sk["b"][:16] = synth.normal(16, 99, (16,), 6.0).astype(np.float32)
    G = GpuLayer(sk, kind="sk"); G.forward()
    ref = oracle_fwd(sk, kind="sk")
    stats = torch.empty(4, device=DEV)
    G.ctx.ds_gap_stats(G.B.H_res, stats); torch.cuda.synchronize()
    Hg = host(G.B.H_res)                                   # the statistics of the matrices the GPU produced
    l1 = O.l1_error(Hg); cd = np.abs(O.column_sums(Hg) - 1).max(axis=1)
    got = host(stats)
    np.testing.assert_allclose(got, [l1.max(), l1.sum(), cd.max(), cd.sum()], rtol=2e-4, atol=1e-5)
    assert abs(got[0] - O.l1_error(ref["H_res"]).max()) <= 1e-2 * O.l1_error(ref["H_res"]).max() + 1e-5
    M0 = np.ascontiguousarray(ref["M0"], dtype=np.float32)
    M0[7] = 0.0                                            # a matrix without a positive entry
    bins, lo, hi = 20, 0.0, 10.0
    hist = torch.empty(bins + 1, dtype=torch.int64, device=DEV)
    G.ctx.log_inv_nu_histogram(torch.from_numpy(M0).to(DEV), bins, lo, hi, hist); torch.cuda.synchronize()
    nu = O.relative_range(M0.astype(np.float64))
    ok = nu > 0
    l = np.log10(1.0 / nu[ok])
    idx = np.clip(np.floor((l - lo) * bins / (hi - lo)).astype(int), 0, bins - 1)
    expect = np.bincount(idx, minlength=bins + 1); expect[bins] = int((~ok).sum())
    h = hist.cpu().numpy()
    assert h.sum() == T and h[bins] == 1
    # a value within rounding of a bin edge may fall either side: compare cumulative counts with a slack of a few
    assert np.abs(np.cumsum(h) - np.cumsum(expect)).max() <= 3


@pytest.mark.parametrize("kind", ["lite", "sk"])
def test_fused_tail_partials_accumulate_and_survive_a_graph(kind):
    """The fused backward tail on the tcgen05 path sums db / dalpha from per-block partials in a fixed order (no
    atomics on the lite path, nothing cleared beforehand): two runs give the same db, dalpha and dx bit for
    bit (dW and dgain agree to rounding: the order in which tensor memory accumulates a tile's four token quadrants
    follows the arrival of their data), an accumulating call doubles the parameter gradients, and the call sequence can
    be captured in a CUDA graph and replayed."""
    n, C, T = 4, 512, 1500
    inp = synth.make_layer_inputs(n, C, T, seed=77, bias_std=0.1, gain_std=0.1, kind=kind)
    G = GpuLayer(inp, kind=kind)
    G.forward(True)
    G.backward(True)
    torch.cuda.synchronize()
    names = ("db", "dalpha", "dW", "dgain", "dx")
    first = {k: getattr(G.B, k).clone() for k in names}
    ref = oracle_bwd(inp, kind=kind)
    check_f32("db", host(first["db"]), ref["db"], 1e-3)
    check_f32("dalpha", host(first["dalpha"]), ref["dalpha"], 1e-3)
    exact = ("db", "dalpha", "dx") if kind == "lite" else ("dx",)      # the SK kernel adds within a block by atomics

    def same_as_first(what):
        for k, v in first.items():
            got = getattr(G.B, k)
            if k in exact:
                assert torch.equal(got, v), f"{k} differs {what}"
            else:
                scale = v.float().pow(2).mean().sqrt()
                assert (got.float() - v.float()).abs().max() <= 1e-5 * scale, f"{k} differs {what}"

    G.backward(True)
    torch.cuda.synchronize()
    same_as_first("between two runs")
    G.backward(True, accumulate_params=True)
    torch.cuda.synchronize()
    for k in ("db", "dalpha", "dW", "dgain"):
        v = first[k]
        scale = v.float().pow(2).mean().sqrt()
        assert (getattr(G.B, k) - 2 * v).abs().max() <= 2e-5 * scale, f"{k} is not doubled by an accumulating call"
    # capture and replay
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        G.backward(True)
        st.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            L.post_bwd(G.ctx, G.B, G.x, G.y, G.g, True)
            L.tail_bwd(G.ctx, G.P, G.B, G.x, G.g, G.du, G.eps, True, G.iters, False)
        for k in names:
            getattr(G.B, k).zero_()
        graph.replay()
        st.synchronize()
    same_as_first("after a graph replay")
    G.ctx.device_status()


@pytest.mark.parametrize("n,C,T", [(4, 1024, 300), (4, 4096, 70), (3, 264, 257), (2, 64, 100), (5, 320, 130)])
def test_pre_fwd_with_the_row_statistic_of_u(n, C, T):
    """mhclite_pre_fwd_fused_ustat: the same outputs as mhclite_pre_fwd_fused, and u_rstd = the oracle's RMSNorm row
    statistic of the stored u (fused into the pre-mix kernel for n <= 4, a separate kernel for n = 5)."""
    inp = synth.make_layer_inputs(n, C, T, seed=40 + n, bias_std=0.1, gain_std=0.1)
    G = GpuLayer(inp)
    G.forward(True)
    torch.cuda.synchronize()
    base = {k: getattr(G.B, k).clone() for k in ("u", "H_res", "H_pre", "H_post", "a_saved", "p_saved", "rstd")}
    u_rstd = torch.full((T,), float("nan"), device=DEV)
    eps_u = 1e-5
    G.ctx.pre_fwd_fused_ustat(G.x, G.P.W, G.P.b, G.P.alpha, G.P.gain, G.eps, G.B.H_res, G.B.H_pre, G.B.H_post, G.B.a_saved,
                              G.B.p_saved, G.B.rstd, G.B.u, u_rstd, eps_u)
    torch.cuda.synchronize()
    for k, v in base.items():
        assert torch.equal(getattr(G.B, k), v), k
    ref = O.premix_row_rstd(host(G.B.u), eps_u)          # over the stored (rounded) u, as the header says
    check_f32("u_rstd", host(u_rstd), ref, 1e-5)
    # and against the oracle's own u: the statistic inherits only u's bf16 rounding
    ref_u = oracle_fwd(inp)["u"]
    assert np.abs(host(u_rstd) / O.premix_row_rstd(ref_u, eps_u) - 1.0).max() < 4e-3
    G.ctx.device_status()

