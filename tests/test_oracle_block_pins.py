"""Pins for the oracle's attention-block steps either side of the path: rotary position embedding (Sec. 5.1) and
Attention = Z V + DWC(V) (Eq. 7).  Closed forms, library routines (scipy's 2-D correlation), invariants and central
finite differences; nothing here re-types the oracle's loops."""
import numpy as np
import pytest
from scipy.signal import correlate2d

import oracle
from oracle import Problem


# --------------------------------------------------------------------------- rotary embedding
def test_rope_hand_values_and_identity_positions():
    X = np.zeros((1, 1, 4, 4))
    X[0, 0, :, 0] = 1.0                      # pair 0 = (1, 0), pair 1 = (0, 0) ... then pair 1 = (0, 2)
    X[0, 0, :, 3] = 2.0
    out = oracle.rope(X, prefix=1, base=100.0)
    np.testing.assert_array_equal(out[0, 0, 0], X[0, 0, 0])              # the prefix token is not rotated
    np.testing.assert_allclose(out[0, 0, 1], X[0, 0, 1], atol=1e-16)     # grid position 0: angle 0
    # grid position p = 2 (token 3): pair 0 rotates by p * 100^0 = 2, pair 1 by p * 100^(-2/4) = 0.2
    np.testing.assert_allclose(out[0, 0, 3], [np.cos(2.0), np.sin(2.0), -2 * np.sin(0.2), 2 * np.cos(0.2)], rtol=1e-14)


def test_rope_is_orthogonal_and_relative():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((2, 3, 10, 8))
    Y = oracle.rope(X, prefix=2, base=10000.0)
    pairs = lambda A: (A.reshape(2, 3, 10, 4, 2) ** 2).sum(-1)
    np.testing.assert_allclose(pairs(Y), pairs(X), rtol=1e-13)           # each channel pair keeps its norm
    np.testing.assert_allclose(oracle.rope(Y, prefix=2, base=10000.0, inverse=True), X, rtol=1e-12, atol=1e-14)
    # adjoint = inverse: <rope(X), U> = <X, rope^T(U)>
    U = rng.standard_normal(X.shape)
    assert float((Y * U).sum()) == pytest.approx(float((X * oracle.rope(U, 2, 10000.0, inverse=True)).sum()), rel=1e-12)
    # the defining property of the rotation: the inner product of two rotated vectors depends on the position
    # difference only
    q, k = rng.standard_normal(8), rng.standard_normal(8)
    def dot_at(pq, pk):
        T = np.zeros((1, 1, 12, 8)); T[0, 0, pq] = q
        S = np.zeros((1, 1, 12, 8)); S[0, 0, pk] = k
        return float(oracle.rope(T, 0, 50.0)[0, 0, pq] @ oracle.rope(S, 0, 50.0)[0, 0, pk])
    assert dot_at(7, 3) == pytest.approx(dot_at(5, 1), rel=1e-12)
    assert dot_at(7, 3) == pytest.approx(dot_at(11, 7), rel=1e-12)
    assert abs(dot_at(7, 3) - dot_at(7, 4)) > 1e-3


def test_round_bf16_matches_the_definition():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.3, 1e-3, 3.0e38 * 0 + 123456.789])
    r = oracle.round_bf16(x)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: ties go to the even mantissa (1); 1 + 3 * 2^-8 is a tie that goes up
    np.testing.assert_array_equal(r[:4], [1.0, 1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -6])
    assert np.all(np.abs(r - x) <= np.abs(x) * 2.0 ** -8)
    assert np.all(np.frexp(r)[0] * 256 == np.round(np.frexp(r)[0] * 256))     # 8 significant bits


# --------------------------------------------------------------------------- depth-wise convolution
def test_dwc_matches_scipy_correlation_and_special_filters():
    rng = np.random.default_rng(2)
    B, H, d, gh, gw, prefix, ks = 2, 2, 3, 5, 4, 1, 3
    n = prefix + gh * gw
    V = rng.standard_normal((B, H, n, d))
    Wd = rng.standard_normal((H, d, ks, ks))
    out = oracle.dwc(V, Wd, prefix, gh, gw)
    assert np.abs(out[:, :, :prefix]).max() == 0.0
    for b in range(B):
        for h in range(H):
            for c in range(d):
                img = V[b, h, prefix:, c].reshape(gh, gw)
                ref = correlate2d(img, Wd[h, c], mode="same", boundary="fill", fillvalue=0.0)
                np.testing.assert_allclose(out[b, h, prefix:, c].reshape(gh, gw), ref, rtol=1e-13, atol=1e-14)
    # a centred delta filter is the identity on the grid; a delta one step to the right shifts the image left
    delta = np.zeros((H, d, ks, ks)); delta[:, :, 1, 1] = 1.0
    np.testing.assert_array_equal(oracle.dwc(V, delta, prefix, gh, gw)[:, :, prefix:], V[:, :, prefix:])
    right = np.zeros((H, d, ks, ks)); right[:, :, 1, 2] = 1.0
    sh = oracle.dwc(V, right, prefix, gh, gw)[0, 0, prefix:, 0].reshape(gh, gw)
    img = V[0, 0, prefix:, 0].reshape(gh, gw)
    np.testing.assert_array_equal(sh[:, :-1], img[:, 1:])
    assert np.abs(sh[:, -1]).max() == 0.0                                 # zero padding
    # 5 x 5 filters
    W5 = rng.standard_normal((H, d, 5, 5))
    o5 = oracle.dwc(V, W5, prefix, gh, gw)
    ref = correlate2d(V[1, 1, prefix:, 2].reshape(gh, gw), W5[1, 2], mode="same")
    np.testing.assert_allclose(o5[1, 1, prefix:, 2].reshape(gh, gw), ref, rtol=1e-13, atol=1e-14)


def test_dwc_bwd_adjoint_and_finite_differences():
    rng = np.random.default_rng(3)
    B, H, d, gh, gw, prefix, ks = 2, 2, 2, 4, 3, 2, 3
    n = prefix + gh * gw
    V, U = rng.standard_normal((B, H, n, d)), rng.standard_normal((B, H, n, d))
    Wd = rng.standard_normal((H, d, ks, ks))
    dV, dWd = oracle.dwc_bwd(V, Wd, U, prefix, gh, gw)
    # linear in V: <DWC(V), U> = <V, DWC^T(U)>; linear in Wd: <DWC_Wd(V), U> = <Wd, dWd>
    lhs = float((oracle.dwc(V, Wd, prefix, gh, gw) * U).sum())
    assert lhs == pytest.approx(float((V * dV).sum()), rel=1e-12)
    assert lhs == pytest.approx(float((Wd * dWd).sum()), rel=1e-12)
    assert np.abs(dV[:, :, :prefix]).max() == 0.0
    h = 1e-6
    for idx in [(0, 1, 0, 2), (1, 0, 2, 1)]:
        wp, wm = Wd.copy(), Wd.copy(); wp[idx] += h; wm[idx] -= h
        fd = ((oracle.dwc(V, wp, prefix, gh, gw) - oracle.dwc(V, wm, prefix, gh, gw)) * U).sum() / (2 * h)
        assert dWd[idx] == pytest.approx(fd, rel=1e-7)


# --------------------------------------------------------------------------- the block
@pytest.mark.parametrize("rope_base,use_dwc", [(100.0, True), (0.0, True), (100.0, False)])
def test_block_backward_finite_differences(rope_base, use_dwc):
    rng = np.random.default_rng(5)
    d, T = 4, 3
    p = Problem(B=2, H=1, n=1 + 12, d=d, m=4, lam=float(d), ns_iters=T, ridge_eps=1e-6, map_mode=1, lm_mode=1,
                prefix=1, gh=3, gw=4, mh=2, mw=2)
    Q, K, V, dO = (rng.standard_normal((2, 1, p.n, d)) for _ in range(4))
    Wd = rng.standard_normal((1, d, 3, 3)) if use_dwc else None
    s = rng.uniform(0.5, 2.0, (1, p.m))
    dQ, dK, dV, dWd = oracle.block_backward(p, Q, K, V, dO, Wd=Wd, rope_base=rope_base, whiten=s)
    loss = lambda q, k, v, w: float((oracle.block_forward(p, q, k, v, Wd=w, rope_base=rope_base, whiten=s) * dO).sum())
    h = 1e-6
    for name, arr, grad in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        for idx in [(0, 0, 0, 1), (1, 0, 7, 2), (0, 0, 12, 3)]:
            a = {"Q": Q, "K": K, "V": V}
            plus, minus = dict(a), dict(a)
            plus[name] = arr.copy(); plus[name][idx] += h
            minus[name] = arr.copy(); minus[name][idx] -= h
            fd = (loss(plus["Q"], plus["K"], plus["V"], Wd) - loss(minus["Q"], minus["K"], minus["V"], Wd)) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=5e-6, abs=1e-8), (name, idx)
    if use_dwc:
        for idx in [(0, 0, 1, 1), (0, 3, 0, 2)]:
            wp, wm = Wd.copy(), Wd.copy(); wp[idx] += h; wm[idx] -= h
            assert dWd[idx] == pytest.approx((loss(Q, K, V, wp) - loss(Q, K, V, wm)) / (2 * h), rel=5e-6, abs=1e-8)
    else:
        assert dWd is None
    # without rotation and convolution the block is the path itself
    np.testing.assert_array_equal(oracle.block_forward(p, Q, K, V, whiten=s), oracle.forward(p, Q, K, V, whiten=s))


def test_rotated_tokens_enter_the_path_in_storage_precision():
    # The rotated Q and K are rounded once to the storage type before the path sees them (what a device that stores them
    # does): sign(token - landmark) in the kernel gradient is then decided on the stored numbers.  With fp32 storage a
    # token coordinate lies within one rounding of a landmark coordinate about once per few hundred thousand (token,
    # landmark, dim) triples; decided on the unrounded double it falls on the other side in half of those cases and one
    # gradient entry changes by 2 g / lambda.
    from dataclasses import replace
    rng = np.random.default_rng(9)
    d = 4
    p = Problem(B=1, H=1, n=6, d=d, m=6, lam=float(d), ns_iters=3, ridge_eps=1e-3, map_mode=1, lm_mode=1, gh=2, gw=3, mh=2, mw=3, lm_f32=1)
    Q, K, V, dO = (rng.standard_normal((1, 1, p.n, d)) for _ in range(4))
    for flags in (dict(store_f32=True), dict(store_bf16=True)):
        rnd = (lambda x: oracle.round_bf16(x)) if "store_bf16" in flags else (lambda x: x.astype(np.float32).astype(np.float64))
        Qr, Kr = rnd(oracle.rope(Q, 0, 100.0)), rnd(oracle.rope(K, 0, 100.0))
        # bins of one token: a landmark is its key, bit for bit, also after the landmarks' own cast to single precision
        np.testing.assert_array_equal(oracle.landmarks_pool(replace(p, lm_f32=0), Kr), Kr)
        assert (Kr.astype(np.float32).astype(np.float64) == Kr).all()
        # the block entry points do exactly this: rotate, round, run the path; the gradient returns through the inverse rotation
        np.testing.assert_array_equal(oracle.block_forward(p, Q, K, V, rope_base=100.0, **flags), oracle.forward(p, Qr, Kr, V))
        dQr, dKr, dV, _ = oracle.backward(p, Qr, Kr, V, dO)
        dQ, dK, dV2, _ = oracle.block_backward(p, Q, K, V, dO, rope_base=100.0, **flags)
        np.testing.assert_array_equal(dQ, oracle.rope(dQr, 0, 100.0, inverse=True))
        np.testing.assert_array_equal(dK, oracle.rope(dKr, 0, 100.0, inverse=True))
        np.testing.assert_array_equal(dV, dV2)
    # without a flag nothing is rounded
    np.testing.assert_array_equal(oracle.block_forward(p, Q, K, V, rope_base=100.0),
                                  oracle.forward(p, oracle.rope(Q, 0, 100.0), oracle.rope(K, 0, 100.0), V))
