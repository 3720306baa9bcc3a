"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with itself: each checks a property,
a closed form, a printed value, a brute-force enumeration or a finite
difference that a plausible mistake in the oracle would break.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import mhclite_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def _rand_layer(T, n, C, kind="lite", alpha=(0.7, 1.1, 0.9), w_std=0.3, seed=0):
    r = np.random.default_rng(seed)
    N = (math.factorial(n) if kind == "lite" else n * n) + 2 * n
    return dict(x=r.standard_normal((T, n, C)), y=r.standard_normal((T, C)),
                W=r.standard_normal((n * C, N)) * w_std, b=r.standard_normal(N) * 0.5,
                alpha=np.array(alpha), gain=1.0 + 0.2 * r.standard_normal(n * C),
                g=r.standard_normal((T, n, C)), du=r.standard_normal((T, C)))


# ------------------------------------------------------------------ permutations (Theorem 3.1, Sec. 3.2)
@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_perm_table_bruteforce(n):
    # brute force: every index tuple of [0,n)^n that is a bijection, sorted
    brute = sorted(t for t in itertools.product(range(n), repeat=n) if len(set(t)) == n)
    tab = O.perm_table(n)
    assert tab.dtype == np.uint8 and tab.shape == (math.factorial(n), n)
    assert [tuple(int(v) for v in row) for row in tab] == brute
    assert len({tuple(r) for r in tab.tolist()}) == math.factorial(n)
    assert tab[0].tolist() == list(range(n))                     # index 0 = identity
    M = O.perm_matrices(n).reshape(-1, n * n)
    assert set(np.unique(M)) == {0.0, 1.0}
    assert (M.sum(axis=1) == n).all()                            # n ones per permutation
    assert (M.sum(axis=0) == math.factorial(n - 1)).all()        # (n-1)! permutations map i -> j
    P = O.perm_matrices(n)
    for k in range(P.shape[0]):                                  # P_k x permutes streams: row i takes sigma_k(i)
        v = np.arange(n, dtype=float)
        assert (P[k] @ v == tab[k]).all()


# ------------------------------------------------------------------ exact double stochasticity (Sec. 2, Theorem 3.1)
@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_hres_doubly_stochastic(n):
    L = _rand_layer(64, n, 8, alpha=(3.0, 1.0, 1.0), seed=n)
    co = O.coeffs_fwd(L["x"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6)
    H = co["H_res"]
    assert (H >= 0).all()
    assert np.abs(H.sum(axis=1) - 1).max() < 1e-14
    assert np.abs(H.sum(axis=2) - 1).max() < 1e-14
    assert np.abs(co["a"].sum(axis=1) - 1).max() < 1e-14 and (co["a"] >= 0).all()
    assert (O.l1_error(H) < 1e-13).all()
    # not a trivial matrix: weights are spread
    assert np.median(co["a"].max(axis=1)) < 0.999 and H.std() > 1e-3


@pytest.mark.parametrize("n", [2, 3, 4])
def test_one_hot_weight_gives_permutation(n):
    T, C = 3, 8
    L = _rand_layer(T, n, C, seed=7)
    N = math.factorial(n) + 2 * n
    tab = O.perm_table(n)
    for k in range(math.factorial(n)):
        b = np.zeros(N); b[:math.factorial(n)] = -800.0; b[k] = 0.0
        co = O.coeffs_fwd(L["x"], np.zeros((n * C, N)), b, L["alpha"], L["gain"], 1e-6)
        expect = np.zeros((n, n)); expect[np.arange(n), tab[k]] = 1.0
        assert (co["H_res"] == expect).all()
        if k == 0:
            assert (co["H_res"] == np.eye(n)).all()
        xn = O.postres_fwd(L["x"], 0 * L["y"], co["H_res"], co["H_post"])
        assert (xn == L["x"][:, tab[k], :]).all()                # row i takes stream sigma_k(i)


def test_paper_initialisation_closed_form():
    # Section 4, "Initialization": W = 0, b_res = -8 except 0 at the identity.
    n, C, T = 4, 8, 2
    L = _rand_layer(T, n, C, seed=3)
    N = 24 + 8
    b = np.concatenate([np.full(24, -8.0), [1, -1, -1, -1], [1, -1, -1, -1]]).astype(float); b[0] = 0.0
    co = O.coeffs_fwd(L["x"], np.zeros((n * C, N)), b, [0.01] * 3, np.ones(n * C), 1e-6)
    w = math.exp(-8.0)
    others = O.perm_matrices(4)[1:].sum(axis=0)
    expect = (np.eye(4) + w * others) / (1 + 23 * w)
    assert np.abs(co["H_res"] - expect).max() < 1e-15
    assert np.abs(co["H_pre"][0] - 1 / (1 + np.exp(-b[24:28]))).max() < 1e-15
    assert np.abs(co["H_post"][0] - 2 / (1 + np.exp(-b[28:32]))).max() < 1e-15


@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_uniform_weights(n):
    T, C = 2, 8
    L = _rand_layer(T, n, C, seed=5)
    N = math.factorial(n) + 2 * n
    co = O.coeffs_fwd(L["x"], np.zeros((n * C, N)), np.zeros(N), L["alpha"], L["gain"], 1e-6)
    assert np.abs(co["H_res"] - 1.0 / n).max() < 1e-15           # J/n
    assert (co["H_pre"] == 0.5).all() and (co["H_post"] == 1.0).all()


@pytest.mark.parametrize("n", [3, 4, 5])
def test_two_routes_to_hres(n):
    a = rng.random((50, math.factorial(n))); a /= a.sum(axis=1, keepdims=True)
    H1 = O.hres_from_weights(a, n)
    H2 = O.hres_from_weights_matmul(a, n)
    assert np.abs(H1 - H2).max() < 1e-15
    # brute-force definition of Eq. (5) for one token
    sig = list(itertools.permutations(range(n)))
    H = np.zeros((n, n))
    for k, s in enumerate(sig):
        Pk = np.zeros((n, n))
        for i in range(n):
            Pk[i, s[i]] = 1
        H += a[0, k] * Pk
    assert np.abs(H1[0] - H).max() < 1e-15


def test_n2_closed_form():
    # n = 2: H_res = [[a0, a1], [a1, a0]], a = softmax(z0, z1) = (sigmoid(z0 - z1), sigmoid(z1 - z0))
    T, n, C = 5, 2, 8
    L = _rand_layer(T, n, C, seed=11)
    co = O.coeffs_fwd(L["x"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6)
    z = co["z"]
    a0 = 1 / (1 + np.exp(-(z[:, 0] - z[:, 1])))
    assert np.abs(co["H_res"][:, 0, 0] - a0).max() < 1e-15
    assert np.abs(co["H_res"][:, 1, 1] - a0).max() < 1e-15
    assert np.abs(co["H_res"][:, 0, 1] - (1 - a0)).max() < 1e-15
    assert np.abs(co["H_res"][:, 1, 0] - (1 - a0)).max() < 1e-15


def test_products_over_depth_stay_doubly_stochastic():
    # Section 2 / 3.1: the Birkhoff polytope is closed under products; spectral norm <= 1
    T, n, C, Ld = 16, 4, 8, 24
    Hs = []
    for l in range(Ld):
        L = _rand_layer(T, n, C, alpha=(4.0, 1, 1), seed=100 + l)
        Hs.append(O.coeffs_fwd(L["x"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6)["H_res"])
    P = O.depth_product(Hs)
    assert (P >= 0).all()
    assert np.abs(P.sum(axis=1) - 1).max() < 1e-13 and np.abs(P.sum(axis=2) - 1).max() < 1e-13
    assert np.linalg.norm(P, ord=2, axis=(1, 2)).max() <= 1 + 1e-12
    # order of the product: later layers on the left
    ref = Hs[2][0] @ Hs[1][0] @ Hs[0][0]
    assert np.abs(O.depth_product(Hs[:3])[0] - ref).max() < 1e-15


# ------------------------------------------------------------------ textbook reductions of Eq. (4)
def test_rmsnorm_softmax_sigmoid_closed_forms():
    xn, rstd = O.rmsnorm_fwd(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), 0.0)
    # mean square = 12.5 -> rstd = 1/sqrt(12.5)
    assert abs(rstd[0] - 1 / math.sqrt(12.5)) < 1e-16
    assert np.abs(xn[0] - np.array([3 / math.sqrt(12.5), 8 / math.sqrt(12.5)])).max() < 1e-15
    xn, rstd = O.rmsnorm_fwd(np.array([[1.0, -1.0, 1.0, -1.0]]), np.ones(4), 3.0)
    assert abs(rstd[0] - 0.5) < 1e-16                           # 1/sqrt(1+3)
    # the normalisation runs over the whole flattened n*C vector, not per stream
    x = np.zeros((1, 2, 2)); x[0, 0] = [2.0, 2.0]
    W = np.zeros((4, 6)); W[0, 2] = 1.0                           # pre-gate 0 sees x'[0]
    co = O.coeffs_fwd(x, W, np.zeros(6), [1, 1, 1], np.ones(4), 0.0)
    # mean(x^2) over 4 entries = 2 -> x'[0] = 2/sqrt(2) = sqrt(2)
    assert abs(co["H_pre"][0, 0] - 1 / (1 + math.exp(-math.sqrt(2)))) < 1e-15
    assert abs(co["p"][0, 2] - math.sqrt(2)) < 1e-15
    # softmax of (0, ln 3) = (1/4, 3/4); sigmoid(ln 3) = 3/4; 2*sigmoid(0) = 1
    b = np.array([0.0, math.log(3.0), math.log(3.0), 0.0, 0.0, 0.0])
    co = O.coeffs_fwd(x, np.zeros((4, 6)), b, [1, 1, 1], np.ones(4), 0.0)
    assert np.abs(co["a"][0] - [0.25, 0.75]).max() < 1e-15
    assert abs(co["H_pre"][0, 0] - 0.75) < 1e-15 and co["H_post"][0, 0] == 1.0


def test_alpha_groups_and_column_order():
    # columns [res | pre | post] scaled by (alpha_res, alpha_pre, alpha_post)
    n, C = 2, 8
    x = rng.standard_normal((3, n, C)); W = rng.standard_normal((n * C, 6)); b = rng.standard_normal(6)
    co = O.coeffs_fwd(x, W, b, [2.0, 3.0, 5.0], np.ones(n * C), 1e-6)
    xh = x.reshape(3, -1); xn = xh / np.sqrt((xh ** 2).mean(1, keepdims=True) + 1e-6)
    p = xn @ W
    assert np.abs(co["z"][:, :2] - (2 * p[:, :2] + b[:2])).max() < 1e-13
    assert np.abs(co["z"][:, 2:4] - (3 * p[:, 2:4] + b[2:4])).max() < 1e-13
    assert np.abs(co["z"][:, 4:] - (5 * p[:, 4:] + b[4:])).max() < 1e-13


def test_eq1_by_loops():
    # Eq. (1) written out with python loops on a tiny case
    T, n, C = 2, 3, 4
    x = rng.standard_normal((T, n, C)); y = rng.standard_normal((T, C))
    Hr = rng.random((T, n, n)); Hp = rng.random((T, n)); Ho = rng.random((T, n))
    u = O.premix_fwd(x, Hp); xn = O.postres_fwd(x, y, Hr, Ho)
    for t in range(T):
        for c in range(C):
            assert abs(u[t, c] - sum(Hp[t, j] * x[t, j, c] for j in range(n))) < 1e-14
            for i in range(n):
                ref = sum(Hr[t, i, j] * x[t, j, c] for j in range(n)) + Ho[t, i] * y[t, c]
                assert abs(xn[t, i, c] - ref) < 1e-14


# ------------------------------------------------------------------ Sinkhorn-Knopp (Eq. (2), Section 1 example)
def _read_golden():
    txt = open(os.path.join(GOLDEN, "sk_example_3x3.txt")).read().splitlines()
    txt = [l for l in txt if l and not l.startswith("#")]
    alpha = float(txt[0].split()[1]); iters = int(txt[1].split()[1])
    i = txt.index("input")
    conv = lambda s: alpha if s == "alpha" else float(s)
    M = np.array([[conv(s) for s in txt[i + 1 + r].split()] for r in range(3)])
    o = txt.index("output_2sig")
    R = np.array([[float(s) for s in txt[o + 1 + r].split()] for r in range(3)])
    cs = np.array([float(s) for s in txt[o + 5].split()[1:]])
    return alpha, iters, M, R, cs


def test_sk_printed_example():
    alpha, iters, M, R, cs = _read_golden()
    out = O.sk_iterate(M[None], iters)[0]
    # printed to two significant digits
    assert np.abs(out - R).max() < 5e-3
    assert np.abs(out.sum(axis=1) - 1).max() < 1e-15              # rows are normalised last
    col = out.sum(axis=0)
    assert np.abs(col - cs).max() < 5e-3                          # 1.82, 0.59, 0.59
    # l1-error of Section 3.1's footnote on this matrix: 0.82 + 0.41 + 0.41
    assert abs(O.l1_error(out) - (abs(col - 1).sum())) < 1e-15 and abs(O.l1_error(out) - 1.64) < 5e-3
    # Eq. (3) on the input: nu = alpha / 1
    assert abs(O.relative_range(M[None])[0] - alpha) < 1e-28
    # the other order (rows first) does not reproduce the printed matrix
    M2 = M.copy()
    for _ in range(iters):
        M2 = M2 / M2.sum(1, keepdims=True); M2 = M2 / M2.sum(0, keepdims=True)
    assert np.abs(M2 - R).max() > 0.1


def test_sk_properties():
    n = 4
    # a doubly stochastic matrix is a fixed point
    a = rng.random((10, 24)); a /= a.sum(1, keepdims=True)
    H = O.hres_from_weights(a, n)
    assert np.abs(O.sk_iterate(H, 20) - H).max() < 1e-14
    # converged SK is invariant to row / column shifts of the logits
    Z = rng.standard_normal((10, n, n))
    r = rng.standard_normal((10, n, 1)); c = rng.standard_normal((10, 1, n))
    A = O.sk_iterate(np.exp(Z), 400); B = O.sk_iterate(np.exp(Z + r + c), 400)
    assert np.abs(A - B).max() < 1e-12
    assert np.abs(A.sum(1) - 1).max() < 1e-12 and np.abs(A.sum(2) - 1).max() < 1e-12
    # rows sum to one after every iteration; columns need not
    for it in (1, 2, 5):
        M = O.sk_iterate(np.exp(3 * Z), it)
        assert np.abs(M.sum(2) - 1).max() < 1e-14
    # ill-conditioned inputs (large 1/nu) leave a gap after 20 iterations, mHC-lite none
    Zbad = 12.0 * rng.standard_normal((200, n, n))
    gap = O.l1_error(O.sk_iterate(np.exp(Zbad - Zbad.max(axis=(1, 2), keepdims=True)), 20))
    assert gap.max() > 1e-2
    L = _rand_layer(8, n, 8, kind="sk", seed=2)
    co = O.sk_coeffs_fwd(L["x"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6, 20)
    assert np.abs(co["H_res"].sum(2) - 1).max() < 1e-14
    # mat() is row-major: logits favouring entry (0,1) raise H_res[0,1]
    b = np.zeros(n * n + 2 * n); b[1] = 5.0
    co = O.sk_coeffs_fwd(L["x"], 0 * L["W"], b, L["alpha"], L["gain"], 1e-6, 20)
    assert co["H_res"][0, 0, 1] > 0.8 and co["H_res"][0, 1, 0] < 0.4


# ------------------------------------------------------------------ gradients: central finite differences
def _loss(L, kind, R1, R2, **over):
    p = {**L, **over}
    o = O.layer_fwd(p["x"], p["y"], p["W"], p["b"], p["alpha"], p["gain"], 1e-6, kind=kind)
    return float((o["x_next"] * R1).sum() + (o["u"] * R2).sum())


@pytest.mark.parametrize("kind,n", [("lite", 2), ("lite", 3), ("lite", 4), ("sk", 2), ("sk", 3), ("sk", 4)])
def test_backward_finite_differences(kind, n):
    T, C = 3, 8
    L = _rand_layer(T, n, C, kind=kind, seed=40 + n)
    R1, R2 = L["g"], L["du"]
    gr = O.layer_bwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6, R1, R2, kind=kind)
    names = dict(x="dx", y="dy", W="dW", b="db", alpha="dalpha", gain="dgain")
    h = 1e-5
    r = np.random.default_rng(9)
    for key, gname in names.items():
        base = np.asarray(L[key], dtype=float)
        an = np.asarray(gr[gname]).reshape(base.shape)
        idx = [tuple(r.integers(0, s) for s in base.shape) for _ in range(min(base.size, 25))]
        if base.size <= 25:
            idx = list(np.ndindex(base.shape))
        scale = np.abs(an).max() + 1e-30
        for ix in idx:
            pp = base.copy(); pp[ix] += h
            pm = base.copy(); pm[ix] -= h
            fd = (_loss(L, kind, R1, R2, **{key: pp}) - _loss(L, kind, R1, R2, **{key: pm})) / (2 * h)
            assert abs(fd - an[ix]) <= 2e-7 * scale + 1e-9, (key, ix, fd, an[ix])


def test_backward_identities():
    n, T, C = 4, 5, 8
    L = _rand_layer(T, n, C, seed=77)
    gr = O.layer_bwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6, L["g"], L["du"])
    # softmax gradient: the residual logit gradients of a token sum to zero
    assert np.abs(gr["dz"][:, :24].sum(axis=1)).max() < 1e-12
    # W = 0: the coefficients do not depend on x, so dx = H_res^T g + H_pre du exactly
    Z = 0 * L["W"]
    co = O.coeffs_fwd(L["x"], Z, L["b"], L["alpha"], L["gain"], 1e-6)
    g0 = O.layer_bwd(L["x"], L["y"], Z, L["b"], L["alpha"], L["gain"], 1e-6, L["g"], L["du"])
    ref = np.einsum("tij,tic->tjc", co["H_res"], L["g"]) + co["H_pre"][:, :, None] * L["du"][:, None, :]
    assert np.abs(g0["dx"] - ref).max() < 1e-13
    assert np.abs(g0["dx_coeffs"]).max() < 1e-13
    # RMSNorm is invariant to the scale of x when eps = 0: <x, dx_coeffs> = 0 per token
    g1 = O.layer_bwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 0.0, L["g"], L["du"])
    assert np.abs((g1["dx_coeffs"] * L["x"]).sum(axis=(1, 2))).max() < 1e-12


def test_round_bf16():
    # exact bf16 values are fixed points; ties go to even; matches a direct rounding
    v = np.array([1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -1.0 - 2 ** -8, 1.0 + 2 ** -8 + 2 ** -40,
                  1.0 + 2 ** -8 - 2 ** -40, 3.14159, 1e-30, 65504.0])
    out = O.round_bf16(v)
    assert out[0] == 1.0 and out[1] == 1.0 + 2 ** -7
    assert out[2] == 1.0                       # tie -> even (mantissa 0)
    assert out[3] == 1.0 + 2 ** -6             # tie -> even (mantissa 2)
    assert out[4] == -1.0
    assert out[5] == 1.0 + 2 ** -7 and out[6] == 1.0      # just above / below a tie (double rounding guarded)
    assert abs(out[7] - 3.14159) <= 2 ** -7 * 2
    for o in out:
        assert (np.float32(o).view(np.uint32) & 0xFFFF) == 0


# ------------------------------------------------------------------ Eq. (3): zero entries and the degenerate matrix
def test_relative_range_skips_zeros():
    # smallest POSITIVE entry over the largest: the zero of [[0,2],[4,8]] is skipped -> 2/8
    assert O.relative_range(np.array([[[0.0, 2.0], [4.0, 8.0]]]))[0] == 0.25
    # a negative entry is not "positive" either
    assert O.relative_range(np.array([[[-1.0, 2.0], [4.0, 8.0]]]))[0] == 0.25
    # no positive entry at all: nu = 0 (1/nu unbounded)
    assert O.relative_range(np.zeros((1, 3, 3)))[0] == 0.0
    # batch of two, mixed
    out = O.relative_range(np.array([[[1.0, 0.0], [0.0, 4.0]], [[0.0, 0.0], [0.0, 0.0]]]))
    assert out.tolist() == [0.25, 0.0]


# ------------------------------------------------------------------ stand-in sublayer and the layer stack (24-layer workload)
def test_standin_sublayer_hand_case_and_gradient():
    # y = u / sqrt(mean(u^2) + eps): u = (3, 4), eps = 0 -> mean square 12.5
    y = O.standin_sublayer_fwd(np.array([[3.0, 4.0]]), 0.0)
    assert np.abs(y[0] - np.array([3.0, 4.0]) / math.sqrt(12.5)).max() < 1e-16
    # eps enters under the root: u = (1,-1,1,-1), eps = 3 -> 1/sqrt(4)
    y = O.standin_sublayer_fwd(np.array([[1.0, -1.0, 1.0, -1.0]]), 3.0)
    assert np.abs(y[0] - np.array([0.5, -0.5, 0.5, -0.5])).max() < 1e-16
    # gradient by central finite differences of the forward
    r = np.random.default_rng(5)
    u = r.standard_normal((3, 6)); dy = r.standard_normal((3, 6)); eps = 1e-3
    an = O.standin_sublayer_bwd(u, dy, eps)
    h = 1e-6
    for ix in np.ndindex(u.shape):
        up = u.copy(); up[ix] += h
        um = u.copy(); um[ix] -= h
        fd = ((O.standin_sublayer_fwd(up, eps) - O.standin_sublayer_fwd(um, eps)) * dy).sum() / (2 * h)
        assert abs(fd - an[ix]) <= 2e-7 * np.abs(an).max(), (ix, fd, an[ix])
    # eps = 0: y does not depend on the scale of u, so <u, du> = 0 for every token
    du0 = O.standin_sublayer_bwd(u, dy, 0.0)
    assert np.abs((u * du0).sum(axis=1)).max() < 1e-13


def test_premix_row_rstd_hand_cases():
    # closed forms: u = (3, 4), eps = 0 -> mean square 12.5; u = (1,-1,1,-1), eps = 3 -> 1/sqrt(4); u = 0 -> eps^-1/2
    assert abs(O.premix_row_rstd(np.array([[3.0, 4.0]]), 0.0)[0] - 1.0 / math.sqrt(12.5)) < 1e-16
    assert abs(O.premix_row_rstd(np.array([[1.0, -1.0, 1.0, -1.0]]), 3.0)[0] - 0.5) < 1e-16
    assert abs(O.premix_row_rstd(np.zeros((1, 8)), 0.25)[0] - 2.0) < 1e-16
    # one value per token, each from its own row only; a row scaled by s has its statistic divided by s at eps = 0
    r = np.random.default_rng(11)
    u = r.standard_normal((5, 12))
    got = O.premix_row_rstd(u, 0.0)
    assert got.shape == (5,)
    u2 = u.copy(); u2[3] *= 4.0
    got2 = O.premix_row_rstd(u2, 0.0)
    assert np.abs(got2[[0, 1, 2, 4]] - got[[0, 1, 2, 4]]).max() == 0.0 and abs(got2[3] - got[3] / 4.0) < 1e-15
    # the normalised row has unit mean square
    assert np.abs(np.mean((u * got[:, None]) ** 2, axis=1) - 1.0).max() < 1e-14


def _stack_params(Ld, n, C, seed):
    r = np.random.default_rng(seed)
    N = math.factorial(n) + 2 * n
    return [(r.standard_normal((n * C, N)) * 0.3, r.standard_normal(N) * 0.5, np.array([0.7, 1.1, 0.9]),
             1.0 + 0.2 * r.standard_normal(n * C)) for _ in range(Ld)]


def _stack_loss(x0, params, R, eps):
    x = x0
    for (W, b, al, ga) in params:
        co = O.coeffs_fwd(x, W, b, al, ga, eps)
        y = O.standin_sublayer_fwd(O.premix_fwd(x, co["H_pre"]), eps)
        x = O.postres_fwd(x, y, co["H_res"], co["H_post"])
    return float((x * R).sum())


def test_stack_equals_hand_chained_layers_and_finite_differences():
    T, n, C, Ld, eps = 2, 3, 4, 3, 1e-3
    r = np.random.default_rng(21)
    params = _stack_params(Ld, n, C, 22)
    x0 = r.standard_normal((T, n, C)); R = r.standard_normal((T, n, C))
    st = O.stack_fwd_bwd(x0, params, R, eps, bf16_storage=False)
    # forward: layer by layer with the single-layer functions
    xs, us, ys = [x0], [], []
    for (W, b, al, ga) in params:
        co = O.coeffs_fwd(xs[-1], W, b, al, ga, eps)
        us.append(O.premix_fwd(xs[-1], co["H_pre"]))
        ys.append(O.standin_sublayer_fwd(us[-1], eps))
        fw = O.layer_fwd(xs[-1], ys[-1], W, b, al, ga, eps)
        assert np.abs(fw["u"] - us[-1]).max() == 0
        xs.append(fw["x_next"])
    for l in range(Ld + 1):
        assert np.abs(st["xs"][l] - xs[l]).max() < 1e-14
    # backward: layer l gets the gradient that layer l + 1 returned, and du = standin_bwd(u_l, dy_l)
    g = R
    for l in reversed(range(Ld)):
        W, b, al, ga = params[l]
        dy = O.postres_bwd(xs[l], ys[l], st["H_res"][l], O.coeffs_fwd(xs[l], W, b, al, ga, eps)["H_post"], g)["dy"]
        du = O.standin_sublayer_bwd(us[l], dy, eps)
        bw = O.layer_bwd(xs[l], ys[l], W, b, al, ga, eps, g, du)
        for k in ("dW", "db", "dalpha", "dgain"):
            assert np.abs(st["grads"][l][k] - bw[k]).max() < 1e-12, (l, k)
        g = bw["dx"]
    assert np.abs(st["dx0"] - g).max() < 1e-12
    # finite differences of the stacked forward: dx0, and one entry of dW, db, dalpha, dgain per layer
    h = 1e-6
    scale = np.abs(st["dx0"]).max()
    for ix in [(0, 0, 0), (1, 2, 3), (0, 1, 2), (1, 0, 1)]:
        xp = x0.copy(); xp[ix] += h
        xm = x0.copy(); xm[ix] -= h
        fd = (_stack_loss(xp, params, R, eps) - _stack_loss(xm, params, R, eps)) / (2 * h)
        assert abs(fd - st["dx0"][ix]) <= 2e-7 * scale + 1e-9, (ix, fd, st["dx0"][ix])
    names = ("dW", "db", "dalpha", "dgain")
    for l in range(Ld):
        for pi, ix in enumerate([(5, 2), (7,), (1,), (9,)]):
            def loss_with(delta):
                ps = [list(p) for p in params]
                arr = np.array(ps[l][pi], dtype=float, copy=True); arr[ix] += delta
                ps[l][pi] = arr
                return _stack_loss(x0, [tuple(p) for p in ps], R, eps)
            fd = (loss_with(h) - loss_with(-h)) / (2 * h)
            an = st["grads"][l][names[pi]][ix]
            assert abs(fd - an) <= 2e-7 * np.abs(st["grads"][l][names[pi]]).max() + 1e-9, (l, names[pi], fd, an)


def test_stack_bf16_storage_lies_on_the_bf16_grid():
    T, n, C, Ld, eps = 3, 4, 8, 2, 1e-6
    r = np.random.default_rng(23)
    params = _stack_params(Ld, n, C, 24)
    x0 = O.round_bf16(r.standard_normal((T, n, C))); R = O.round_bf16(r.standard_normal((T, n, C)))
    st = O.stack_fwd_bwd(x0, params, R, eps, bf16_storage=True)
    on_grid = lambda a: ((np.asarray(a, dtype=np.float32).view(np.uint32) & 0xFFFF) == 0).all() and \
        (np.asarray(a, dtype=np.float32).astype(np.float64) == a).all()
    for l in range(Ld + 1):
        assert on_grid(st["xs"][l]), l
    assert on_grid(st["dx0"])
    # and it stays within bf16 rounding of the unrounded stack
    ex = O.stack_fwd_bwd(x0, params, R, eps, bf16_storage=False)
    assert np.abs(st["xs"][Ld] - ex["xs"][Ld]).max() <= 2.0 ** -6 * np.abs(ex["xs"][Ld]).max()
    assert np.abs(st["xs"][Ld] - ex["xs"][Ld]).max() > 0


# ------------------------------------------------------------------ Section 5: a subset of the permutations
@pytest.mark.parametrize("n,K", [(3, 2), (4, 7), (5, 8), (5, 64), (6, 24)])
def test_any_subset_of_permutations_is_exactly_doubly_stochastic(n, K):
    r = np.random.default_rng(n * 100 + K)
    full = np.array(list(itertools.permutations(range(n))))
    tab = full[r.choice(len(full), K, replace=False)]
    T, C = 16, 4
    N = K + 2 * n
    x = r.standard_normal((T, n, C)); W = r.standard_normal((n * C, N)); b = r.standard_normal(N)
    co = O.coeffs_fwd(x, W, b, [2.0, 1.0, 1.0], np.ones(n * C), 1e-6, table=tab)
    H = co["H_res"]
    assert co["a"].shape == (T, K) and H.shape == (T, n, n)
    assert (H >= 0).all()
    assert np.abs(H.sum(axis=1) - 1).max() < 1e-14 and np.abs(H.sum(axis=2) - 1).max() < 1e-14
    # entries outside the support of the sampled permutations are exactly zero
    support = np.zeros((n, n), dtype=bool)
    for row in tab:
        support[np.arange(n), row] = True
    assert (H[:, ~support] == 0).all()
    # brute-force Eq. (5) over the subset for one token
    ref = np.zeros((n, n))
    for k, row in enumerate(tab):
        P = np.zeros((n, n)); P[np.arange(n), row] = 1
        ref += co["a"][0, k] * P
    assert np.abs(H[0] - ref).max() < 1e-15


@pytest.mark.parametrize("n", [3, 4])
def test_full_table_as_subset_reproduces_eq5(n):
    L = _rand_layer(5, n, 8, seed=60 + n)
    tab = O.perm_table(n)
    a = O.layer_fwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6)
    b = O.layer_fwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6, table=tab)
    for k in ("H_res", "H_pre", "H_post", "a", "u", "x_next"):
        assert np.abs(a[k] - b[k]).max() < 1e-15, k
    ga = O.layer_bwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6, L["g"], L["du"])
    gb = O.layer_bwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6, L["g"], L["du"], table=tab)
    for k in ("dx", "dW", "db", "dalpha", "dgain"):
        assert np.abs(ga[k] - gb[k]).max() < 1e-13, k
    # a permuted table permutes the residual columns: row order is the caller's
    perm = np.random.default_rng(3).permutation(len(tab))
    N = len(tab) + 2 * n
    cols = np.concatenate([perm, np.arange(len(tab), N)])
    c = O.coeffs_fwd(L["x"], L["W"][:, cols], L["b"][cols], L["alpha"], L["gain"], 1e-6, table=tab[perm])
    assert np.abs(c["H_res"] - a["H_res"]).max() < 1e-14


def test_subset_one_hot_and_rejections():
    n, C, T = 5, 4, 2
    tab = np.array([[0, 1, 2, 3, 4], [4, 3, 2, 1, 0], [1, 0, 3, 2, 4]])
    N = 3 + 2 * n
    x = np.random.default_rng(1).standard_normal((T, n, C))
    for k in range(3):
        b = np.zeros(N); b[:3] = -800.0; b[k] = 0.0
        co = O.coeffs_fwd(x, np.zeros((n * C, N)), b, [1, 1, 1], np.ones(n * C), 1e-6, table=tab)
        expect = np.zeros((n, n)); expect[np.arange(n), tab[k]] = 1.0
        assert (co["H_res"] == expect).all()
    with pytest.raises(ValueError):
        O.check_perm_rows([[0, 1, 1]], 3)                       # not a bijection
    with pytest.raises(ValueError):
        O.check_perm_rows([[0, 1, 2], [0, 1, 2]], 3)            # repeated row
    with pytest.raises(ValueError):
        O.check_perm_rows([[0, 1, 3]], 3)                       # out of range
    with pytest.raises(ValueError):
        O.check_perm_rows([[0, 1]], 3)                          # wrong width
    assert O.check_perm_rows([[2, 0, 1]], 3).tolist() == [[2, 0, 1]]


@pytest.mark.parametrize("n,K", [(4, 5), (5, 8), (6, 6)])
def test_subset_backward_finite_differences(n, K):
    T, C = 2, 4
    r = np.random.default_rng(70 + n)
    full = np.array(list(itertools.permutations(range(n))))
    tab = full[r.choice(len(full), K, replace=False)]
    N = K + 2 * n
    L = dict(x=r.standard_normal((T, n, C)), y=r.standard_normal((T, C)), W=r.standard_normal((n * C, N)) * 0.3,
             b=r.standard_normal(N) * 0.5, alpha=np.array([0.7, 1.1, 0.9]), gain=1.0 + 0.2 * r.standard_normal(n * C))
    R1, R2 = r.standard_normal((T, n, C)), r.standard_normal((T, C))

    def loss(**over):
        p = {**L, **over}
        o = O.layer_fwd(p["x"], p["y"], p["W"], p["b"], p["alpha"], p["gain"], 1e-6, table=tab)
        return float((o["x_next"] * R1).sum() + (o["u"] * R2).sum())

    gr = O.layer_bwd(L["x"], L["y"], L["W"], L["b"], L["alpha"], L["gain"], 1e-6, R1, R2, table=tab)
    assert np.abs(gr["dz"][:, :K].sum(axis=1)).max() < 1e-12
    h = 1e-5
    for key, gname in dict(x="dx", y="dy", W="dW", b="db", alpha="dalpha", gain="dgain").items():
        base = np.asarray(L[key], dtype=float)
        an = np.asarray(gr[gname]).reshape(base.shape)
        idx = list(np.ndindex(base.shape))
        if len(idx) > 20:
            idx = [idx[i] for i in r.choice(len(idx), 20, replace=False)]
        scale = np.abs(an).max() + 1e-30
        for ix in idx:
            pp = base.copy(); pp[ix] += h
            pm = base.copy(); pm[ix] -= h
            fd = (loss(**{key: pp}) - loss(**{key: pm})) / (2 * h)
            assert abs(fd - an[ix]) <= 2e-7 * scale + 1e-9, (key, ix, fd, an[ix])
