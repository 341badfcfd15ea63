"""Pins of the oracle's conjugate-gradient solver (the other solver of Sec. 5.3 / Table 4) against what the mathematics
fixes: the one-step closed form, the Krylov-subspace optimality of every iterate (computed here by a dense projected
solve, not by a recurrence), termination in m steps, the library's dense solve, and finite differences of the whole
path once the solver has converged.  CPU only."""
import numpy as np
import pytest

import oracle
from oracle import Problem


def spd(rng, m, kappa):
    """Symmetric positive definite matrix with eigenvalues spread geometrically over [1, kappa]."""
    Qm, _ = np.linalg.qr(rng.standard_normal((m, m)))
    ev = np.geomspace(1.0, kappa, m)
    return (Qm * ev) @ Qm.T


def krylov_minimiser(W, b, k):
    """argmin over x in span{b, W b, ..., W^(k-1) b} of the energy norm of the error: the k-th CG iterate by definition."""
    cols = [b]
    for _ in range(k - 1):
        cols.append(W @ cols[-1])
    Kb, _ = np.linalg.qr(np.stack(cols, axis=1))            # orthonormal basis: the projected system stays well conditioned
    y = np.linalg.solve(Kb.T @ W @ Kb, Kb.T @ b)
    return Kb @ y


def test_one_step_closed_form_and_zero_steps():
    rng = np.random.default_rng(3)
    m, d = 7, 3
    W = spd(rng, m, 10.0)[None]
    Bm = rng.standard_normal((1, m, d))
    X0 = oracle.cg_solve(W, Bm, 0)
    assert np.abs(X0).max() == 0.0                           # x_0 = 0
    X1 = oracle.cg_solve(W, Bm, 1)
    for c in range(d):
        b = Bm[0, :, c]
        np.testing.assert_allclose(X1[0, :, c], (b @ b) / (b @ W[0] @ b) * b, rtol=1e-13)   # steepest descent from zero


@pytest.mark.parametrize("kappa", [2.0, 50.0])
def test_every_iterate_is_the_krylov_minimiser(kappa):
    rng = np.random.default_rng(int(kappa))
    m, d = 12, 2
    W = spd(rng, m, kappa)
    Bm = rng.standard_normal((1, m, d))
    for k in (1, 2, 3, 5):
        Xk = oracle.cg_solve(W[None], Bm, k)
        for c in range(d):
            np.testing.assert_allclose(Xk[0, :, c], krylov_minimiser(W, Bm[0, :, c], k), rtol=2e-8, atol=1e-10)


def test_terminates_in_m_steps_and_error_decreases():
    rng = np.random.default_rng(11)
    m, d = 10, 4
    W = spd(rng, m, 20.0)
    Bm = rng.standard_normal((2, m, d))
    Ws = np.stack([W, spd(rng, m, 5.0)])
    exact = np.linalg.solve(Ws, Bm)
    Xm = oracle.cg_solve(Ws, Bm, m)
    np.testing.assert_allclose(Xm, exact, rtol=1e-8, atol=1e-10)
    # the energy norm of the error never grows from one step to the next
    prev = None
    for k in range(0, m + 1):
        E = oracle.cg_solve(Ws, Bm, k) - exact
        en = np.einsum("bic,bij,bjc->bc", E, Ws, E)
        if prev is not None:
            assert (en <= prev * (1 + 1e-12) + 1e-22).all()
        prev = en
    # more steps than unknowns change nothing once the residual is at rounding level
    np.testing.assert_allclose(oracle.cg_solve(Ws, Bm, m + 5), exact, rtol=1e-8, atol=1e-10)


def test_ridge_identity_and_independent_columns():
    rng = np.random.default_rng(5)
    m, d = 6, 3
    Bm = rng.standard_normal((1, m, d))
    # W = I: one step is exact; the ridge enters as W + eps I
    X = oracle.cg_solve(np.eye(m)[None], Bm, 1, eps=0.25)
    np.testing.assert_allclose(X, Bm / 1.25, rtol=1e-14)
    # a column does not see the others
    W = spd(rng, m, 8.0)[None]
    Xa = oracle.cg_solve(W, Bm, 3)
    Xb = oracle.cg_solve(W, Bm[:, :, 1:2].copy(), 3)
    np.testing.assert_array_equal(Xa[:, :, 1:2], Xb)
    # a zero right-hand side stays zero (no division by its zero residual)
    Z = Bm.copy(); Z[:, :, 0] = 0.0
    assert np.abs(oracle.cg_solve(W, Z, 4)[:, :, 0]).max() == 0.0


def test_path_with_cg_equals_a_dense_solve_when_converged():
    # m steps on a small, well-conditioned landmark matrix: Y must be (W + eps I)^-1 M, and O follows from it
    rng = np.random.default_rng(21)
    n, d, m = 24, 6, 6
    p = Problem(B=1, H=2, n=n, d=d, m=m, lam=float(d), ns_iters=3 * m, ridge_eps=1e-3, map_mode=1, lm_mode=1,
                gh=4, gw=6, mh=2, mw=3, solver=1)
    Q, K, V = (rng.standard_normal((1, 2, n, d)) for _ in range(3))
    s = rng.uniform(0.5, 2.0, (2, m))
    O, x = oracle.forward(p, Q, K, V, whiten=s, want=("W", "M", "Y", "Z"))
    for bh in range(2):
        Y = np.linalg.solve(x["W"][bh] + 1e-3 * np.eye(m), x["M"][bh])
        np.testing.assert_allclose(x["Y"][bh], Y, rtol=1e-8, atol=1e-11)
        np.testing.assert_allclose(O.reshape(2, n, d)[bh], x["Z"][bh] @ Y, rtol=1e-8, atol=1e-11)


@pytest.mark.parametrize("lm_mode", [0, 1])
def test_backward_with_cg_matches_finite_differences_when_converged(lm_mode):
    # the backward rule differentiates the linear system the solver approximates; with the solver converged the rule is
    # the derivative of what the forward pass computes, and central differences must agree
    rng = np.random.default_rng(31 + lm_mode)
    n, d, m = 24, 5, 6
    p = Problem(B=1, H=2, n=n, d=d, m=m, lam=float(d), ns_iters=4 * m, ridge_eps=1e-2, map_mode=1, lm_mode=lm_mode,
                gh=4, gw=6, mh=2, mw=3, solver=1)
    Q, K, V, dO = (rng.standard_normal((1, 2, n, d)) for _ in range(4))
    L = rng.standard_normal((1, 2, m, d)) if lm_mode == 0 else None
    s = rng.uniform(0.5, 2.0, (2, m))
    dQ, dK, dV, dL = oracle.backward(p, Q, K, V, dO, L=L, whiten=s)
    loss = lambda q, k, v, l: float((oracle.forward(p, q, k, v, L=l, whiten=s) * dO).sum())
    h = 1e-6
    for name, arr, grad in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        for idx in [(0, 0, 0, 0), (0, 1, 7, 3), (0, 0, 23, 4), (0, 1, 11, 2)]:
            a = {"Q": Q, "K": K, "V": V}
            plus = dict(a); minus = dict(a)
            plus[name] = arr.copy(); plus[name][idx] += h
            minus[name] = arr.copy(); minus[name][idx] -= h
            fd = (loss(plus["Q"], plus["K"], plus["V"], L) - loss(minus["Q"], minus["K"], minus["V"], L)) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=2e-5, abs=1e-8), (name, idx)
    if lm_mode == 0:
        for idx in [(0, 0, 0, 0), (0, 1, 5, 4), (0, 0, 3, 2)]:
            lp = L.copy(); lp[idx] += h
            lm_ = L.copy(); lm_[idx] -= h
            assert dL[idx] == pytest.approx((loss(Q, K, V, lp) - loss(Q, K, V, lm_)) / (2 * h), rel=2e-5, abs=1e-8)


def test_backward_rule_at_few_steps_is_the_stated_one():
    # at few steps the rule is not the derivative of the truncated iteration; it is what it says: dM from the same
    # T-step solve on dY, dW = -dM Y^T.  Checked on a problem whose only trainable input is V (M = R V is linear in V,
    # W does not depend on V): dV = R^T CG_T(W, dY).
    rng = np.random.default_rng(41)
    n, d, m, T = 24, 4, 6, 2
    p = Problem(B=1, H=1, n=n, d=d, m=m, lam=float(d), ns_iters=T, ridge_eps=1e-3, map_mode=0, lm_mode=1,
                gh=4, gw=6, mh=2, mw=3, solver=1)
    Q, K, V, dO = (rng.standard_normal((1, 1, n, d)) for _ in range(4))
    _, x = oracle.forward(p, Q, K, V, want=("W", "R", "Z"))
    dV = oracle.backward(p, Q, K, V, dO)[2]
    dY = x["Z"][0].T @ dO[0, 0]
    dM = oracle.cg_solve(x["W"], dY[None], T, eps=1e-3)[0]
    np.testing.assert_allclose(dV[0, 0], x["R"][0].T @ dM, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("kappa", [2.0, 10.0, 50.0])
def test_energy_norm_error_bound_over_condition_numbers(kappa):
    # the textbook bound ||x_k - x*||_W <= 2 ((sqrt(kappa) - 1) / (sqrt(kappa) + 1))^k ||x*||_W, the behaviour the paper's
    # convergence figure (Sec. 5.3) describes: fast at kappa = 2, slower as the condition number grows
    rng = np.random.default_rng(100 + int(kappa))
    m, d = 24, 3
    W = spd(rng, m, kappa)
    Bm = rng.standard_normal((1, m, d))
    exact = np.linalg.solve(W, Bm[0])
    e0 = np.sqrt(np.einsum("ic,ij,jc->c", exact, W, exact))
    rho = (np.sqrt(kappa) - 1) / (np.sqrt(kappa) + 1)
    errs = []
    for k in (1, 2, 4, 8):
        E = oracle.cg_solve(W[None], Bm, k)[0] - exact
        en = np.sqrt(np.einsum("ic,ij,jc->c", E, W, E))
        assert (en <= 2 * rho ** k * e0 * (1 + 1e-10)).all(), (kappa, k)
        errs.append(en.max() / e0.max())
    if kappa == 2.0:
        assert errs[-1] < 1e-5          # eight steps at kappa = 2: converged
    if kappa == 50.0:
        assert errs[-1] > 1e-5          # and not yet at kappa = 50
