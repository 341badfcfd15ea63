"""Pins for the float64 oracle: closed forms, brute force, invariants, finite differences.

None of these re-type the oracle's own code path: brute force is written with
numpy broadcasting, closed forms come from the mathematics (Kac-Murdock-Szego
inverse, spectral form of the Newton-Schulz polynomial), and gradients are
checked against central differences of the oracle's *forward*.
"""
import os

import numpy as np
import pytest

import oracle
from oracle import Problem

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "hand_values.txt")) as fh:
    for line in fh:
        if line.startswith("#") or "|" not in line:
            continue
        name, val, _ = [t.strip() for t in line.split("|")]
        GOLD[name] = float(val)


def np_l1(A, Bm, lam):
    """Brute force with broadcasting: exp(-sum_c |a_ic - b_jc| / lam)."""
    return np.exp(-np.abs(A[:, None, :] - Bm[None, :, :]).sum(-1) / lam)


# --------------------------------------------------------------------------- kernel
def test_l1_hand_values():
    k = oracle.l1_kernel(np.zeros((1, 1, 4)), np.ones((1, 1, 4)), 4.0)
    assert k[0, 0, 0] == pytest.approx(GOLD["k_unit_offset"], rel=1e-15)
    k = oracle.l1_kernel(np.array([[[0.5, -1.0]]]), np.array([[[0.25, 1.0]]]), 2.0)
    assert k[0, 0, 0] == pytest.approx(GOLD["k_two_dim"], rel=1e-15)


def test_l1_bruteforce_and_properties():
    rng = np.random.default_rng(1)
    A = rng.standard_normal((3, 17, 5))
    Bm = rng.standard_normal((3, 9, 5))
    K, rs = oracle.l1_kernel(A, Bm, 2.5, want_rowsum=True)
    for b in range(3):
        np.testing.assert_allclose(K[b], np_l1(A[b], Bm[b], 2.5), rtol=1e-14)
    np.testing.assert_allclose(rs, K.sum(-1), rtol=1e-14)
    # product form over coordinates
    prod = np.prod(np.exp(-np.abs(A[0][:, None, :] - Bm[0][None, :, :]) / 2.5), axis=-1)
    np.testing.assert_allclose(K[0], prod, rtol=1e-13)
    # symmetry, unit diagonal, range
    S = oracle.l1_kernel(A, A, 2.5)
    np.testing.assert_array_equal(S, S.transpose(0, 2, 1))
    np.testing.assert_array_equal(np.diagonal(S, axis1=1, axis2=2), 1.0)
    assert (S > 0).all() and (S <= 1).all()
    # triangle inequality of the l1 distance: k(x,z) >= k(x,y) k(y,z)
    KB = oracle.l1_kernel(Bm, Bm, 2.5)
    lhs = K[0][:, None, :]                       # k(a_i, b_j) for every middle point b_k
    rhs = K[0][:, :, None] * KB[0][None, :, :]   # k(a_i, b_k) k(b_k, b_j)
    assert (lhs + 1e-15 >= rhs).all()


def test_l1_single_pair_gradient_norm():
    # App. A: ||grad_x k||_2 = sqrt(d)/lambda * k when no coordinate ties
    x = np.zeros((1, 1, 4)); y = np.ones((1, 1, 4))
    dA, dB = oracle.l1_kernel_bwd(x, y, 4.0, np.ones((1, 1, 1)))
    assert np.linalg.norm(dA) == pytest.approx(GOLD["grad_norm_unit_offset"], rel=1e-15)
    # x < y in every coordinate: d k / d x_c = -(1/lambda) sign(x-y) k = +k/lambda
    np.testing.assert_allclose(dA, +GOLD["k_unit_offset"] / 4.0)
    np.testing.assert_allclose(dB, -GOLD["k_unit_offset"] / 4.0)


def test_l1_gradient_tie_is_zero():
    x = np.array([[[1.0, 2.0]]]); y = np.array([[[1.0, 3.0]]])
    dA, dB = oracle.l1_kernel_bwd(x, y, 1.0, np.ones((1, 1, 1)))
    assert dA[0, 0, 0] == 0.0 and dB[0, 0, 0] == 0.0
    assert dA[0, 0, 1] == pytest.approx(np.exp(-1.0))


def test_l1_bwd_finite_differences():
    rng = np.random.default_rng(2)
    A = rng.standard_normal((2, 6, 4)); Bm = rng.standard_normal((2, 5, 4))
    dK = rng.standard_normal((2, 6, 5))
    dA, dB = oracle.l1_kernel_bwd(A, Bm, 1.7, dK)
    f = lambda a, b: float((oracle.l1_kernel(a, b, 1.7) * dK).sum())
    h = 1e-6
    for arr, grad, which in ((A, dA, 0), (Bm, dB, 1)):
        for idx in [(0, 0, 0), (1, 3, 2), (0, 4, 3), (1, 2, 1)]:
            p = arr.copy(); p[idx] += h
            q = arr.copy(); q[idx] -= h
            fd = (f(p, Bm) - f(q, Bm)) / (2 * h) if which == 0 else (f(A, p) - f(A, q)) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=1e-7, abs=1e-9)


# --------------------------------------------------------------------------- landmark kernel + Newton-Schulz
def kms(m, rho):
    idx = np.arange(m)
    return rho ** np.abs(idx[:, None] - idx[None, :])


def test_kms_closed_form_inverse():
    # d = 1, equally spaced points, lambda = 1/ln 2 -> W_ij = (1/2)^|i-j|
    pts = np.arange(4, dtype=np.float64).reshape(1, 4, 1)
    W = oracle.l1_kernel(pts, pts, 1.0 / np.log(2.0))
    np.testing.assert_allclose(W[0], kms(4, 0.5), rtol=1e-14)
    X, resid, alpha = oracle.ns_pinv(W, 60, eps=0.0)
    assert resid[0] < 1e-12
    assert X[0, 0, 0] == pytest.approx(GOLD["kms_inv_corner"], rel=1e-12)
    assert X[0, 3, 3] == pytest.approx(GOLD["kms_inv_corner"], rel=1e-12)
    assert X[0, 1, 1] == pytest.approx(GOLD["kms_inv_inner_diag"], rel=1e-12)
    assert X[0, 1, 2] == pytest.approx(GOLD["kms_inv_offdiag"], rel=1e-12)
    assert X[0, 2, 1] == pytest.approx(GOLD["kms_inv_offdiag"], rel=1e-12)
    assert abs(X[0, 0, 2]) < 1e-12 and abs(X[0, 0, 3]) < 1e-12
    # general m, rho: tridiagonal closed form
    m, rho = 9, 0.8
    Winv = np.zeros((m, m))
    for i in range(m):
        Winv[i, i] = (1 + rho * rho) if 0 < i < m - 1 else 1.0
        if i + 1 < m:
            Winv[i, i + 1] = Winv[i + 1, i] = -rho
    Winv /= (1 - rho * rho)
    X, resid, _ = oracle.ns_pinv(kms(m, rho)[None], 80)
    np.testing.assert_allclose(X[0], Winv, atol=1e-10)


def test_ns_alpha_rule_and_spectral_closed_form():
    # For symmetric W: I - W X_T = (I - alpha W^2)^(2^T), so in the eigenbasis of W
    # X_T = U diag((1 - (1 - alpha w_i^2)^(2^T)) / w_i) U^T  -- pins the UNCONVERGED iterate.
    rng = np.random.default_rng(3)
    pts = rng.standard_normal((1, 12, 6))
    W = oracle.l1_kernel(pts, pts, 6.0)[0]
    eps = 1e-3
    We = W + eps * np.eye(12)
    for T in (0, 1, 3, 6):
        X, resid, alpha = oracle.ns_pinv(W[None], T, eps=eps)
        a = 1.0 / (np.abs(We).sum(0).max() * np.abs(We).sum(1).max())
        assert alpha[0] == pytest.approx(a, rel=1e-14)
        w, U = np.linalg.eigh(We)
        xs = (1.0 - (1.0 - a * w * w) ** (2 ** T)) / w
        np.testing.assert_allclose(X[0], (U * xs) @ U.T, rtol=0, atol=1e-12 * np.abs(xs).max())
        assert resid[0] == pytest.approx(np.linalg.norm(np.eye(12) - We @ X[0]), rel=1e-10)


def test_ns_nonsymmetric_matches_definition():
    # Alg. 2 is stated for a general W (X_0 = alpha W^T): check against a direct numpy loop
    rng = np.random.default_rng(4)
    W = np.eye(5) + 0.2 * rng.standard_normal((5, 5))
    a = 1.0 / (np.abs(W).sum(0).max() * np.abs(W).sum(1).max())
    X = a * W.T
    hist = []
    for _ in range(5):
        hist.append(X)
        X = X @ (2 * np.eye(5) - W @ X)
    Xo, _, alpha, Xh = oracle.ns_pinv(W[None], 5, want_hist=True)
    np.testing.assert_allclose(Xo[0], X, rtol=1e-13)
    np.testing.assert_allclose(Xh[0], np.stack(hist), rtol=1e-13)
    Xc, resid, _ = oracle.ns_pinv(W[None], 50)
    np.testing.assert_allclose(Xc[0], np.linalg.inv(W), atol=1e-11)


def test_ns_converges_to_inverse_and_residual_monotone():
    rng = np.random.default_rng(5)
    pts = rng.standard_normal((2, 16, 8))
    W = oracle.l1_kernel(pts, pts, 8.0)
    # symmetric, unit diagonal, positive definite
    np.testing.assert_array_equal(W, W.transpose(0, 2, 1))
    for b in range(2):
        np.linalg.cholesky(W[b])
    prev = None
    for T in range(0, 45, 3):
        X, resid, _ = oracle.ns_pinv(W, T, eps=1e-9)
        if prev is not None:
            assert (resid <= prev * (1 + 1e-9) + 1e-13).all()
        prev = resid
    X, resid, _ = oracle.ns_pinv(W, 45, eps=0.0)
    for b in range(2):
        assert np.abs(X[b] @ W[b] - np.eye(16)).max() < 1e-10


def test_ns_degenerate_cases():
    X, resid, alpha = oracle.ns_pinv(np.eye(7)[None], 0)
    np.testing.assert_allclose(X[0], np.eye(7), rtol=1e-15)          # alpha = 1, X_0 = I
    X, resid, alpha = oracle.ns_pinv(np.array([[[4.0]]]), 0)          # m = 1: alpha = 1/16, X_0 = 1/4
    assert X[0, 0, 0] == pytest.approx(0.25)
    X, _, _ = oracle.ns_pinv(np.array([[[4.0]]]), 3, eps=1.0)         # exact at X_0 already: 1/(W+eps)
    assert X[0, 0, 0] == pytest.approx(0.2)


def test_ns_literal_alpha_diverges():
    # alpha = 2/||W||_2 as printed in Alg. 2 violates ||I - alpha W W^T|| < 1 for unit-diagonal W
    rng = np.random.default_rng(6)
    pts = rng.standard_normal((1, 16, 8))
    W = oracle.l1_kernel(pts, pts, 8.0)
    lit = 2.0 / np.linalg.norm(W[0], 2)
    with np.errstate(all="ignore"):
        X, resid, alpha = oracle.ns_pinv(W, 8, alpha=lit)
    assert alpha[0] == lit
    assert not np.isfinite(resid[0]) or resid[0] > 1e6


@pytest.mark.parametrize("kappa", [2.0, 10.0, 50.0])
def test_ns_condition_number_sweep(kappa):
    # Fig. 6 setting: SPD matrices of prescribed condition number, error ||X_k - W^-1||_F / ||W^-1||_F
    rng = np.random.default_rng(7)
    Qm, _ = np.linalg.qr(rng.standard_normal((24, 24)))
    w = np.geomspace(1.0, 1.0 / kappa, 24)
    W = (Qm * w) @ Qm.T
    W = 0.5 * (W + W.T)
    Winv = np.linalg.inv(W)
    errs = []
    for T in range(0, 30, 2):
        X, _, _ = oracle.ns_pinv(W[None], T)
        errs.append(np.linalg.norm(X[0] - Winv) / np.linalg.norm(Winv))
    assert all(e2 <= e1 * (1 + 1e-9) + 1e-14 for e1, e2 in zip(errs, errs[1:]))
    assert errs[-1] < 1e-10


def test_ns_bwd_finite_differences():
    rng = np.random.default_rng(8)
    pts = rng.standard_normal((1, 5, 3))
    W = oracle.l1_kernel(pts, pts, 3.0) + 0.01 * rng.standard_normal((1, 5, 5))  # general (non-symmetric)
    dX = rng.standard_normal((1, 5, 5))
    for alpha in (0.0, 0.03):
        dW = oracle.ns_pinv_bwd(W, 4, 1e-3, alpha, dX)
        f = lambda w: float((oracle.ns_pinv(w, 4, eps=1e-3, alpha=alpha)[0] * dX).sum())
        h = 1e-6
        for i in range(5):
            for j in range(5):
                p = W.copy(); p[0, i, j] += h
                q = W.copy(); q[0, i, j] -= h
                assert dW[0, i, j] == pytest.approx((f(p) - f(q)) / (2 * h), rel=2e-6, abs=1e-8)


def test_norm_gradient_at_tied_columns_goes_through_the_lowest_index():
    """alpha = 1/(||W||_1 ||W||_inf) (Alg. 2) is not differentiable where two columns attain the maximum, and two
    identical landmarks make two column sums equal exactly.  The reading: the gradient of a norm is taken through the
    lowest index whose sum lies within 2^-14 (relative) of the maximum, whatever the rounding of the sums says."""
    rng = np.random.default_rng(88)
    pts = rng.standard_normal((1, 7, 3)) * 2.0
    pts[0, 5] = pts[0, 2]                                    # landmark 5 is a copy of landmark 2
    W = oracle.l1_kernel(pts, pts, 3.0)
    eps, T = 1e-6, 3
    cs = np.abs(W[0] + eps * np.eye(7)).sum(0)
    assert np.argsort(-cs)[:2].tolist() in ([2, 5], [5, 2]) and abs(cs[2] - cs[5]) < 1e-12      # the tied pair is the maximum
    dX = rng.standard_normal((1, 7, 7))

    def alpha_term(Wm):
        # gradient with alpha derived from the norms minus the gradient with the same alpha given: what remains is
        # d(loss)/d(alpha) * d(alpha)/dW, which lives in column jstar and row istar only
        a = oracle.ns_pinv(Wm, T, eps=eps)[2][0]
        D = oracle.ns_pinv_bwd(Wm, T, eps, 0.0, dX) - oracle.ns_pinv_bwd(Wm, T, eps, a, dX)
        cols = sorted(set(np.nonzero(np.abs(D[0]).sum(0) > 1e-14 * np.abs(D).max())[0].tolist()))
        rows = sorted(set(np.nonzero(np.abs(D[0]).sum(1) > 1e-14 * np.abs(D).max())[0].tolist()))
        return D[0], cols, rows

    D, cols, rows = alpha_term(W)
    # column 2 and row 2 carry the two norm terms (every entry of W is positive: the whole column / row is touched);
    # nothing else is
    off = D.copy(); off[:, 2] = 0.0; off[2, :] = 0.0
    assert np.abs(off).max() == 0.0 and np.abs(D[:, 2]).min() > 0.0 and np.abs(D[2, :]).min() > 0.0
    # a perturbation far below the window that makes column 5 the strict maximum does not move the choice
    Wp = W.copy(); Wp[0, 0, 5] += 1e-7; Wp[0, 5, 0] += 1e-7
    Dp, _, _ = alpha_term(Wp)
    off = Dp.copy(); off[:, 2] = 0.0; off[2, :] = 0.0
    assert np.abs(off).max() == 0.0
    # well outside the window the larger column wins
    Wq = W.copy(); Wq[0, :, 5] *= 1.01; Wq[0, 5, :] *= 1.01
    Dq, _, _ = alpha_term(Wq)
    off = Dq.copy(); off[:, 5] = 0.0; off[5, :] = 0.0
    assert np.abs(off).max() == 0.0 and np.abs(Dq[:, 5]).min() > 0.0
    # and the norm itself is the true maximum in every case
    for Wm in (W, Wp, Wq):
        A = Wm[0] + eps * np.eye(7)
        assert oracle.ns_pinv(Wm, T, eps=eps)[2][0] == pytest.approx(1.0 / (np.abs(A).sum(0).max() * np.abs(A).sum(1).max()), rel=1e-14)


# --------------------------------------------------------------------------- pooling
def test_pool_divisible_and_adjoint():
    p = Problem(B=1, H=2, n=1 + 6 * 4, d=3, m=6, lam=3.0, ns_iters=2, prefix=1, gh=6, gw=4, mh=3, mw=2)
    rng = np.random.default_rng(9)
    K = rng.standard_normal((1, 2, p.n, 3))
    L = oracle.landmarks_pool(p, K)
    grid = K[:, :, 1:].reshape(1, 2, 6, 4, 3)
    hand = grid.reshape(1, 2, 3, 2, 2, 2, 3).mean(axis=(3, 5)).reshape(1, 2, 6, 3)   # 2x2 / stride-2 means
    np.testing.assert_allclose(L, hand, rtol=1e-14)
    U = rng.standard_normal(L.shape)
    dK = oracle.landmarks_pool_bwd(p, U)
    assert float((L * U).sum()) == pytest.approx(float((K * dK).sum()), rel=1e-12)
    assert np.abs(dK[:, :, 0]).max() == 0.0          # prefix token is never pooled


def test_pool_adaptive_bins_overlap_and_identity():
    # 14 -> 4 bins: floor(a*14/4) .. ceil((a+1)*14/4): [0,4) [3,7) [7,11) [10,14)
    p = Problem(B=1, H=1, n=14, d=1, m=4, lam=1.0, ns_iters=0, gh=1, gw=14, mh=1, mw=4)
    K = np.arange(14, dtype=np.float64).reshape(1, 1, 14, 1)
    L = oracle.landmarks_pool(p, K)[0, 0, :, 0]
    np.testing.assert_allclose(L, [1.5, 4.5, 8.5, 11.5])
    # each row of the pooling matrix sums to one: pooling a constant gives the constant
    L1 = oracle.landmarks_pool(p, np.ones((1, 1, 14, 1)))
    np.testing.assert_allclose(L1, 1.0)
    # bins == grid: landmarks are the keys themselves
    p2 = Problem(B=1, H=1, n=12, d=2, m=12, lam=1.0, ns_iters=0, gh=3, gw=4, mh=3, mw=4)
    K2 = np.random.default_rng(10).standard_normal((1, 1, 12, 2))
    np.testing.assert_array_equal(oracle.landmarks_pool(p2, K2), K2)


# --------------------------------------------------------------------------- the whole chain
def exact_attention(Q, K, V, lam, s=None, map_mode=1):
    """Eq. 4 + Eq. 7 without any approximation: Z_full V with Z_full built from G = k(Q, K)."""
    G = np_l1(Q, K, lam)
    n = K.shape[0]
    if map_mode == 0:
        return G @ V
    s = np.ones(n) if s is None else s
    Z = (G - G.mean(1, keepdims=True)) * s[None, :] + 1.0 / n
    return Z @ V


@pytest.mark.parametrize("map_mode", [0, 1])
def test_m_equals_n_reproduces_exact_attention(map_mode):
    rng = np.random.default_rng(11)
    n, d = 12, 4
    p = Problem(B=1, H=2, n=n, d=d, m=n, lam=float(d), ns_iters=60, ridge_eps=0.0, map_mode=map_mode,
                lm_mode=1, gh=3, gw=4, mh=3, mw=4)
    Q, K, V = (rng.standard_normal((1, 2, n, d)) for _ in range(3))
    s = rng.uniform(0.5, 2.0, (2, n))
    O = oracle.forward(p, Q, K, V, whiten=s)
    for h in range(2):
        ref = exact_attention(Q[0, h], K[0, h], V[0, h], float(d), s[h], map_mode)
        np.testing.assert_allclose(O[0, h], ref, atol=1e-9)


def test_intermediates_and_folded_form():
    rng = np.random.default_rng(12)
    n, d, m = 20, 4, 5
    p = Problem(B=2, H=2, n=n, d=d, m=m, lam=float(d), ns_iters=3, lm_mode=1, gh=4, gw=5, mh=1, mw=5)
    Q, K, V = (rng.standard_normal((2, 2, n, d)) for _ in range(3))
    s = rng.uniform(0.5, 2.0, (2, m))
    O, x = oracle.forward(p, Q, K, V, whiten=s, want=("L", "C", "R", "W", "X", "M", "Y", "Z"))
    for bh in range(4):
        q, k, v = Q.reshape(4, n, d)[bh], K.reshape(4, n, d)[bh], V.reshape(4, n, d)[bh]
        L = np.stack([k.reshape(4, 5, d)[:, b].mean(0) for b in range(5)])   # 4x5 grid -> 1x5 bins = column means
        np.testing.assert_allclose(x["L"][bh], L, rtol=1e-14)
        np.testing.assert_allclose(x["C"][bh], np_l1(q, L, d), rtol=1e-13)
        np.testing.assert_allclose(x["R"][bh], np_l1(L, k, d), rtol=1e-13)
        np.testing.assert_allclose(x["W"][bh], np_l1(L, L, d), rtol=1e-13)
        sh = s[bh % 2]
        # rows of Z sum to one when s = 1 (checked below); with s general the centred part is scaled
        Z = (x["C"][bh] - x["C"][bh].mean(1, keepdims=True)) * sh + 1.0 / m
        np.testing.assert_allclose(x["Z"][bh], Z, rtol=1e-13)
        Y = x["X"][bh] @ (x["R"][bh] @ v)
        np.testing.assert_allclose(x["Y"][bh], Y, rtol=1e-12)
        # folded form: O = C Ytilde + 1 ybar^T
        Yt = sh[:, None] * Y - (sh[:, None] * Y).mean(0, keepdims=True)
        ybar = Y.mean(0)
        np.testing.assert_allclose(O.reshape(4, n, d)[bh], x["C"][bh] @ Yt + ybar, rtol=1e-10, atol=1e-12)
    O1, x1 = oracle.forward(p, Q, K, V, whiten=None, want=("Z",))
    np.testing.assert_allclose(x1["Z"].sum(-1), GOLD["z_row_sum"], rtol=1e-13)


@pytest.mark.parametrize("lm_mode,map_mode,use_s", [(1, 1, True), (1, 0, False), (0, 1, True), (0, 1, False)])
def test_full_backward_finite_differences(lm_mode, map_mode, use_s):
    rng = np.random.default_rng(13 + lm_mode + 2 * map_mode)
    n, d, m, T = 24, 6, 6, 4
    p = Problem(B=1, H=2, n=n, d=d, m=m, lam=float(d), ns_iters=T, ridge_eps=1e-6, map_mode=map_mode,
                lm_mode=lm_mode, gh=4, gw=6, mh=2, mw=3)
    Q, K, V, dO = (rng.standard_normal((1, 2, n, d)) for _ in range(4))
    L = rng.standard_normal((1, 2, m, d)) if lm_mode == 0 else None
    s = rng.uniform(0.5, 2.0, (2, m)) if use_s else None
    dQ, dK, dV, dL = oracle.backward(p, Q, K, V, dO, L=L, whiten=s)
    loss = lambda q, k, v, l: float((oracle.forward(p, q, k, v, L=l, whiten=s) * dO).sum())
    h = 1e-6
    probes = [(0, 0, 0, 0), (0, 1, 7, 3), (0, 0, 23, 5), (0, 1, 11, 2), (0, 0, 5, 1)]
    for name, arr, grad in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        for idx in probes:
            a = {"Q": Q, "K": K, "V": V}
            plus = dict(a); minus = dict(a)
            plus[name] = arr.copy(); plus[name][idx] += h
            minus[name] = arr.copy(); minus[name][idx] -= h
            fd = (loss(plus["Q"], plus["K"], plus["V"], L) - loss(minus["Q"], minus["K"], minus["V"], L)) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=5e-6, abs=1e-8), (name, idx)
    if lm_mode == 0:
        for idx in [(0, 0, 0, 0), (0, 1, 5, 5), (0, 0, 3, 2)]:
            lp = L.copy(); lp[idx] += h
            lm_ = L.copy(); lm_[idx] -= h
            fd = (loss(Q, K, V, lp) - loss(Q, K, V, lm_)) / (2 * h)
            assert dL[idx] == pytest.approx(fd, rel=5e-6, abs=1e-8)
    else:
        assert dL is None


def test_whiten_stats_hand_values_and_invariants():
    """Eq. 5-6: population variance over the batch of query rows, scale 1/sqrt(sigma^2 + eps)."""
    C = np.array([[[1.0, 7.0], [2.0, 7.0], [3.0, 7.0], [4.0, 7.0]]])            # one head, four rows, two landmarks
    s = oracle.whiten_stats(C, 1, 0.35)
    assert abs(s[0, 0] - GOLD["whiten_scale_1234"]) < 1e-15
    assert abs(oracle.whiten_stats(C, 1, 0.25)[0, 1] - GOLD["whiten_scale_constant"]) < 1e-15
    rng = np.random.default_rng(5)
    B, H, n, m = 3, 2, 17, 5
    C = rng.uniform(0.2, 0.8, (B * H, n, m))
    s = oracle.whiten_stats(C, H, 1e-5)
    # against the library's population variance, on the rows of a head gathered over the batch
    for h in range(H):
        rows = np.concatenate([C[b * H + h] for b in range(B)], axis=0)
        assert np.allclose(s[h], 1.0 / np.sqrt(rows.var(axis=0) + 1e-5), rtol=1e-12)
    # the order of the batch elements and a shift of a column do not matter; a scale a multiplies sigma by |a|
    perm = np.concatenate([np.arange(H) + b * H for b in (2, 0, 1)])
    assert np.allclose(oracle.whiten_stats(C[perm], H, 1e-5), s, rtol=1e-12)
    assert np.allclose(oracle.whiten_stats(C + 3.0, H, 1e-5), s, rtol=1e-9)
    assert np.allclose(oracle.whiten_stats(-2.0 * C, H, 0.0), oracle.whiten_stats(C, H, 0.0) / 2.0, rtol=1e-12)
    # heads do not mix: changing head 1 leaves the scale of head 0 alone
    C2 = C.copy(); C2[1::H] *= 1.7
    assert np.array_equal(oracle.whiten_stats(C2, H, 1e-5)[0], s[0])


# --------------------------------------------------------------------------- pooling adjoint on overlapping bins
def test_pool_bwd_overlapping_bins_hand_values():
    # 14 -> 4 bins (Sec. 4.2 pooling, adaptive bins): [0,4) [3,7) [7,11) [10,14), four tokens each.
    # Token 3 lies in bins 0 and 1 and token 10 in bins 2 and 3; every other token lies in one bin.
    p = Problem(B=1, H=1, n=14, d=1, m=4, lam=1.0, ns_iters=0, gh=1, gw=14, mh=1, mw=4)
    dL = np.array([1.0, 10.0, 100.0, 1000.0]).reshape(1, 1, 4, 1)
    dK = oracle.landmarks_pool_bwd(p, dL)[0, 0, :, 0]
    hand = np.array([0.25, 0.25, 0.25, 0.25 + 2.5, 2.5, 2.5, 2.5, 25.0, 25.0, 25.0, 25.0 + 250.0, 250.0, 250.0, 250.0])
    np.testing.assert_allclose(dK, hand, rtol=1e-15)
    # two-dimensional overlap: 3 x 3 grid into 2 x 2 bins of 2 x 2 tokens; the centre token lies in all four bins
    p2 = Problem(B=1, H=1, n=9, d=1, m=4, lam=1.0, ns_iters=0, gh=3, gw=3, mh=2, mw=2)
    dL2 = np.array([4.0, 40.0, 400.0, 4000.0]).reshape(1, 1, 4, 1)
    dK2 = oracle.landmarks_pool_bwd(p2, dL2)[0, 0, :, 0].reshape(3, 3)
    hand2 = np.array([[1.0, 11.0, 10.0], [101.0, 1111.0, 1010.0], [100.0, 1100.0, 1000.0]])
    np.testing.assert_allclose(dK2, hand2, rtol=1e-15)


@pytest.mark.parametrize("gh,gw,mh,mw,prefix", [(14, 14, 4, 8, 0), (56, 56, 8, 16, 0), (14, 14, 4, 8, 2), (5, 7, 3, 3, 1)])
def test_pool_bwd_overlapping_bins_adjoint_identity(gh, gw, mh, mw, prefix):
    # <pool(K), U> = <K, pool^T(U)> on the non-divisible geometries of the workloads (14 -> 4 x 8, 56 -> 8 x 16)
    d = 3
    p = Problem(B=1, H=2, n=prefix + gh * gw, d=d, m=mh * mw, lam=1.0, ns_iters=0, prefix=prefix, gh=gh, gw=gw, mh=mh, mw=mw)
    rng = np.random.default_rng(31)
    K = rng.standard_normal((1, 2, p.n, d))
    U = rng.standard_normal((1, 2, p.m, d))
    L = oracle.landmarks_pool(p, K)
    dK = oracle.landmarks_pool_bwd(p, U)
    assert float((L * U).sum()) == pytest.approx(float((K * dK).sum()), rel=1e-12)
    assert np.abs(dK[:, :, :prefix]).max(initial=0.0) == 0.0
    # the pooling matrix applied to unit vectors: column sums of pool^T(e_l) are one (a bin's weights sum to one)
    for l in (0, p.m // 2, p.m - 1):
        e = np.zeros((1, 2, p.m, d)); e[:, :, l] = 1.0
        np.testing.assert_allclose(oracle.landmarks_pool_bwd(p, e).sum(axis=2), 1.0, rtol=1e-13)


def test_full_backward_finite_differences_overlapping_bins():
    # the whole backward with landmarks pooled over a grid the bins do not divide (5 x 7 -> 2 x 3, class token in front)
    rng = np.random.default_rng(41)
    d, T = 5, 3
    p = Problem(B=1, H=1, n=1 + 35, d=d, m=6, lam=float(d), ns_iters=T, ridge_eps=1e-6, map_mode=1, lm_mode=1,
                prefix=1, gh=5, gw=7, mh=2, mw=3)
    Q, K, V, dO = (rng.standard_normal((1, 1, p.n, d)) for _ in range(4))
    s = rng.uniform(0.5, 2.0, (1, p.m))
    dQ, dK, dV, _ = oracle.backward(p, Q, K, V, dO, whiten=s)
    loss = lambda k: float((oracle.forward(p, Q, k, V, whiten=s) * dO).sum())
    h = 1e-6
    # tokens 18 (row 2, col 3: shared by both bin rows) and 11 (row 1, col 3) lie in overlapping bins; 0 is the class token
    for idx in [(0, 0, 0, 0), (0, 0, 18, 2), (0, 0, 11, 4), (0, 0, 35, 1), (0, 0, 4, 0)]:
        kp = K.copy(); kp[idx] += h
        km = K.copy(); km[idx] -= h
        assert dK[idx] == pytest.approx((loss(kp) - loss(km)) / (2 * h), rel=5e-6, abs=1e-8), idx


# --------------------------------------------------------------------------- landmarks rounded to single precision
def _lm_case(seed):
    rng = np.random.default_rng(seed)
    p0 = Problem(B=1, H=2, n=1 + 8 * 6, d=8, m=12, lam=8.0, ns_iters=4, ridge_eps=1e-6, map_mode=1, lm_mode=1,
                 prefix=1, gh=8, gw=6, mh=4, mw=3)
    Q, K, V, dO = (rng.standard_normal((1, 2, p0.n, p0.d)) for _ in range(4))
    s = rng.uniform(0.5, 2.0, (2, p0.m))
    return p0, Q, K, V, dO, s


def test_lm_f32_is_the_given_landmark_path_on_rounded_means():
    # lm_f32 = 1 must be exactly: pool in float64, round each landmark coordinate to float32 (numpy's cast), and carry on
    # as if those landmarks had been given (lm_mode 0); the landmark gradient then returns to the keys through the
    # pooling adjoint
    from dataclasses import replace
    p0, Q, K, V, dO, s = _lm_case(51)
    p1 = replace(p0, lm_f32=1)
    L32 = oracle.landmarks_pool(p0, K).astype(np.float32).astype(np.float64)
    pg = replace(p0, lm_mode=0)
    O1 = oracle.forward(p1, Q, K, V, whiten=s)
    Og = oracle.forward(pg, Q, K, V, L=L32, whiten=s)
    np.testing.assert_array_equal(O1, Og)
    dQ1, dK1, dV1, _ = oracle.backward(p1, Q, K, V, dO, whiten=s)
    dQg, dKg, dVg, dLg = oracle.backward(pg, Q, K, V, dO, L=L32, whiten=s)
    np.testing.assert_array_equal(dQ1, dQg)
    np.testing.assert_array_equal(dV1, dVg)
    np.testing.assert_allclose(dK1, dKg + oracle.landmarks_pool_bwd(p0, dLg), rtol=1e-13, atol=1e-15)
    # and the flag does change the landmarks (otherwise the comparison above would be vacuous)
    assert np.abs(L32 - oracle.landmarks_pool(p0, K)).max() > 0.0


def test_lm_f32_moves_results_only_at_rounding_level_away_from_ties():
    from dataclasses import replace
    p0, Q, K, V, dO, s = _lm_case(52)
    p1 = replace(p0, lm_f32=1)
    L64 = oracle.landmarks_pool(p0, K)
    L32 = L64.astype(np.float32).astype(np.float64)
    # places where sign(token - landmark) differs between the two landmark precisions: only there can the flag move
    # a gradient by more than rounding (an exact tie with a mean that float32 holds exactly is a tie on both sides)
    near = 0
    for T_ in (Q, K):
        near += int((np.sign(T_[:, :, :, None, :] - L64[:, :, None, :, :]) != np.sign(T_[:, :, :, None, :] - L32[:, :, None, :, :])).sum())
    assert near == 0                                    # none on this seeded case
    O0, O1 = oracle.forward(p0, Q, K, V, whiten=s), oracle.forward(p1, Q, K, V, whiten=s)
    assert np.linalg.norm(O0 - O1) <= 1e-7 * np.linalg.norm(O0)
    g0 = oracle.backward(p0, Q, K, V, dO, whiten=s)[:3]
    g1 = oracle.backward(p1, Q, K, V, dO, whiten=s)[:3]
    for a, b in zip(g0, g1):
        assert np.linalg.norm(a - b) <= 1e-6 * np.linalg.norm(a)
    # a planted near-tie: one query coordinate placed between a landmark's exact mean and its float32 rounding
    l, c = 3, 2
    lo, hi = sorted((L64[0, 0, l, c], L32[0, 0, l, c]))
    assert hi > lo
    Qt = Q.copy(); Qt[0, 0, 5, c] = 0.5 * (lo + hi)
    d0 = oracle.backward(p0, Qt, K, V, dO, whiten=s)[0]
    d1 = oracle.backward(p1, Qt, K, V, dO, whiten=s)[0]
    diff = np.abs(d0 - d1)
    assert diff[0, 0, 5, c] > 1e3 * np.delete(diff[0, 0, 5], c).max()   # the sign of that one term flipped, nothing else moved


def test_exact_attention_definition_against_brute_force_and_m_equals_n():
    # oracle.exact_attention (the O(n^2) definition) against the broadcasting brute force of this file, and against the
    # Nystrom chain at m = n with converged Newton-Schulz
    rng = np.random.default_rng(61)
    n, d = 12, 3
    Q, K, V = (rng.standard_normal((1, 2, n, d)) for _ in range(3))
    for map_mode in (0, 1):
        O = oracle.exact_attention(Q, K, V, float(d), map_mode)
        for h in range(2):
            np.testing.assert_allclose(O[0, h], exact_attention(Q[0, h], K[0, h], V[0, h], float(d), None, map_mode), rtol=1e-13)
        p = Problem(B=1, H=2, n=n, d=d, m=n, lam=float(d), ns_iters=40, ridge_eps=0.0, map_mode=map_mode, lm_mode=1,
                    gh=3, gw=4, mh=3, mw=4)
        np.testing.assert_allclose(oracle.forward(p, Q, K, V), O, rtol=1e-8, atol=1e-10)


def test_landmarks_pooled_from_queries_variant():
    # lm_mode 2 (Sec. 4.2 "Landmark Selection" pools the query tensor): the same chain with L = pool(Q); pinned against
    # the given-landmark path fed with pool(Q), the landmark gradient returning to Q through the pooling adjoint, and
    # against central differences
    from dataclasses import replace
    rng = np.random.default_rng(71)
    p2 = Problem(B=1, H=2, n=2 + 5 * 6, d=4, m=6, lam=4.0, ns_iters=3, ridge_eps=1e-6, map_mode=1, lm_mode=2,
                 prefix=2, gh=5, gw=6, mh=2, mw=3)
    Q, K, V, dO = (rng.standard_normal((1, 2, p2.n, p2.d)) for _ in range(4))
    s = rng.uniform(0.5, 2.0, (2, p2.m))
    Lq = oracle.landmarks_pool(replace(p2, lm_mode=1), Q)
    pg = replace(p2, lm_mode=0)
    np.testing.assert_array_equal(oracle.forward(p2, Q, K, V, whiten=s), oracle.forward(pg, Q, K, V, L=Lq, whiten=s))
    dQ, dK, dV, dL = oracle.backward(p2, Q, K, V, dO, whiten=s)
    dQg, dKg, dVg, dLg = oracle.backward(pg, Q, K, V, dO, L=Lq, whiten=s)
    assert dL is None
    np.testing.assert_array_equal(dK, dKg)
    np.testing.assert_array_equal(dV, dVg)
    np.testing.assert_allclose(dQ, dQg + oracle.landmarks_pool_bwd(replace(p2, lm_mode=1), dLg), rtol=1e-13, atol=1e-15)
    loss = lambda q: float((oracle.forward(p2, q, K, V, whiten=s) * dO).sum())
    h = 1e-6
    for idx in [(0, 0, 0, 0), (0, 1, 9, 2), (0, 0, 31, 3)]:
        qp, qm = Q.copy(), Q.copy(); qp[idx] += h; qm[idx] -= h
        assert dQ[idx] == pytest.approx((loss(qp) - loss(qm)) / (2 * h), rel=5e-6, abs=1e-8)


# --------------------------------------------------------------------------- whitening with batch statistics
@pytest.mark.parametrize("lm_mode", [1, 0])
def test_batch_whitening_backward_finite_differences(lm_mode):
    # Eq. 5-6 in training mode: s comes from the batch's own kernel block; the batch elements of a head are coupled
    rng = np.random.default_rng(81)
    d, T, eps_w = 4, 3, 1e-3
    p = Problem(B=3, H=2, n=12, d=d, m=4, lam=float(d), ns_iters=T, ridge_eps=1e-6, map_mode=1, lm_mode=lm_mode,
                gh=3, gw=4, mh=2, mw=2)
    Q, K, V, dO = (rng.standard_normal((3, 2, p.n, d)) for _ in range(4))
    L = rng.standard_normal((3, 2, p.m, d)) if lm_mode == 0 else None
    O, s = oracle.forward_batch_whiten(p, Q, K, V, eps_w, L=L)
    # the forward is the constant-scale path fed with the statistic of the already pinned whiten_stats
    np.testing.assert_array_equal(O, oracle.forward(p, Q, K, V, L=L, whiten=s))
    dQ, dK, dV, dL, s2 = oracle.backward_batch_whiten(p, Q, K, V, dO, eps_w, L=L)
    np.testing.assert_array_equal(s, s2)
    loss = lambda q, k, v, l: float((oracle.forward_batch_whiten(p, q, k, v, eps_w, L=l)[0] * dO).sum())
    h = 1e-6
    for name, arr, grad in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        for idx in [(0, 0, 0, 1), (2, 1, 7, 2), (1, 0, 11, 3)]:
            a = {"Q": Q, "K": K, "V": V}
            plus, minus = dict(a), dict(a)
            plus[name] = arr.copy(); plus[name][idx] += h
            minus[name] = arr.copy(); minus[name][idx] -= h
            fd = (loss(plus["Q"], plus["K"], plus["V"], L) - loss(minus["Q"], minus["K"], minus["V"], L)) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=2e-5, abs=1e-8), (name, idx)
    if lm_mode == 0:
        for idx in [(0, 1, 1, 0), (2, 0, 3, 3)]:
            lp, lm_ = L.copy(), L.copy(); lp[idx] += h; lm_[idx] -= h
            assert dL[idx] == pytest.approx((loss(Q, K, V, lp) - loss(Q, K, V, lm_)) / (2 * h), rel=2e-5, abs=1e-8)
    # the variance path matters: with s held constant the query gradient is a different one
    dQc = oracle.backward(p, Q, K, V, dO, L=L, whiten=s)[0]
    assert np.linalg.norm(dQc - dQ) > 1e-3 * np.linalg.norm(dQ)


def test_two_landmark_sets_variant_of_alg1():
    # lm_mode 3 (Alg. 1 as printed): Lq = pool(Q), Lk = pool(K), C = k(Q, Lk), W = k(Lq, Lk), R = k(Lq, K)
    from dataclasses import replace
    rng = np.random.default_rng(91)
    p3 = Problem(B=1, H=2, n=1 + 4 * 6, d=4, m=6, lam=4.0, ns_iters=3, ridge_eps=1e-6, map_mode=1, lm_mode=3,
                 prefix=1, gh=4, gw=6, mh=2, mw=3)
    Q, K, V, dO = (rng.standard_normal((1, 2, p3.n, p3.d)) for _ in range(4))
    s = rng.uniform(0.5, 2.0, (2, p3.m))
    # the blocks are what the algorithm says: checked against the stand-alone kernel and the direct Newton-Schulz loop
    O, x = oracle.forward(p3, Q, K, V, whiten=s, want=("C", "R", "W", "X", "M", "Y", "Z"))
    p1 = replace(p3, lm_mode=1)
    Lk, Lq = oracle.landmarks_pool(p1, K), oracle.landmarks_pool(p1, Q)
    for h in range(2):
        np.testing.assert_allclose(x["C"][h], np_l1(Q[0, h], Lk[0, h], 4.0), rtol=1e-13)
        np.testing.assert_allclose(x["W"][h], np_l1(Lq[0, h], Lk[0, h], 4.0), rtol=1e-13)
        np.testing.assert_allclose(x["R"][h], np_l1(Lq[0, h], K[0, h], 4.0), rtol=1e-13)
        W = x["W"][h] + 1e-6 * np.eye(6)
        assert np.abs(W - W.T).max() > 1e-3                         # a genuinely non-symmetric W
        X = W.T / (np.abs(W).sum(0).max() * np.abs(W).sum(1).max())
        for _ in range(3):
            X = X @ (2 * np.eye(6) - W @ X)
        np.testing.assert_allclose(x["X"][h], X, rtol=1e-11)
        np.testing.assert_allclose(O[0, h], x["Z"][h] @ (X @ (x["R"][h] @ V[0, h])), rtol=1e-10)
    # with Q == K the two sets coincide and the variant is the one-set path
    np.testing.assert_allclose(oracle.forward(p3, K, K, V, whiten=s), oracle.forward(p1, K, K, V, whiten=s), rtol=1e-13)
    # backward by central differences
    dQ, dK, dV, dL = oracle.backward(p3, Q, K, V, dO, whiten=s)
    assert dL is None
    loss = lambda q, k, v: float((oracle.forward(p3, q, k, v, whiten=s) * dO).sum())
    h_ = 1e-6
    for name, arr, grad in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        for idx in [(0, 0, 0, 1), (0, 1, 7, 2), (0, 0, 24, 3)]:
            a = {"Q": Q, "K": K, "V": V}
            plus, minus = dict(a), dict(a)
            plus[name] = arr.copy(); plus[name][idx] += h_
            minus[name] = arr.copy(); minus[name][idx] -= h_
            fd = (loss(plus["Q"], plus["K"], plus["V"]) - loss(minus["Q"], minus["K"], minus["V"])) / (2 * h_)
            assert grad[idx] == pytest.approx(fd, rel=5e-6, abs=1e-8), (name, idx)
