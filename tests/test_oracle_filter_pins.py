"""Pins of the oracle's depth-wise-convolution landmark selection (Sec. 4.2, the alternative to average pooling):
one r x r filter per head and channel, stride r, over the regions average pooling would average.  Pinned against the
library's grouped strided convolution, against average pooling (constant filter), the adjoint identity and finite
differences of the whole path including the filter's own gradient."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from oracle import Problem


def _case(seed, lm_mode=1, B=2, H=2, gh=6, gw=8, mh=3, mw=2, d=6, prefix=1, T=3):
    rng = np.random.default_rng(seed)
    n, m = prefix + gh * gw, mh * mw
    taps = (gh // mh) * (gw // mw)
    F = rng.standard_normal((H, taps, d)) / taps
    p = Problem(B=B, H=H, n=n, d=d, m=m, lam=float(d), ns_iters=T, ridge_eps=1e-6, map_mode=1, lm_mode=lm_mode,
                prefix=prefix, gh=gh, gw=gw, mh=mh, mw=mw, lm_filter=F)
    Q, K, V, dO = (rng.standard_normal((B, H, n, d)) for _ in range(4))
    s = rng.uniform(0.5, 2.0, (H, m))
    return p, Q, K, V, dO, s


def test_filter_selection_is_a_grouped_strided_convolution():
    # the library routine: conv2d with one group per (head, channel), kernel (rh, rw), stride (rh, rw), no bias
    p, _, K, _, _, _ = _case(3, gh=6, gw=8, mh=3, mw=2)          # regions of 2 x 4: rh != rw, class token in front
    rh, rw = p.gh // p.mh, p.gw // p.mw
    L = oracle.landmarks_pool(p, K)
    grid = K[:, :, p.prefix:, :].reshape(p.B, p.H, p.gh, p.gw, p.d)
    x = torch.from_numpy(np.ascontiguousarray(grid.transpose(0, 1, 4, 2, 3))).reshape(p.B, p.H * p.d, p.gh, p.gw)
    w = torch.from_numpy(np.ascontiguousarray(p.lm_filter.transpose(0, 2, 1))).reshape(p.H * p.d, 1, rh, rw)
    y = torch.nn.functional.conv2d(x, w, stride=(rh, rw), groups=p.H * p.d)       # [B, H d, mh, mw]
    ref = y.reshape(p.B, p.H, p.d, p.mh * p.mw).permute(0, 1, 3, 2).numpy()
    assert np.abs(L - ref).max() < 1e-13
    # a hand value: landmark (0, 0) of head 1, channel 2 is the dot product of its eight taps with its eight tokens
    toks = [p.prefix + u * p.gw + v for u in range(rh) for v in range(rw)]
    hand = sum(p.lm_filter[1, t, 2] * K[0, 1, tok, 2] for t, tok in enumerate(toks))
    assert L[0, 1, 0, 2] == pytest.approx(hand, rel=1e-14)


@pytest.mark.parametrize("lm_mode", [1, 2])
def test_constant_filter_is_average_pooling(lm_mode):
    p, Q, K, V, dO, s = _case(5, lm_mode=lm_mode)
    taps = p.lm_filter.shape[1]
    pf = replace(p, lm_filter=np.full_like(p.lm_filter, 1.0 / taps))
    pa = replace(p, lm_filter=None)
    assert np.abs(oracle.forward(pf, Q, K, V, whiten=s) - oracle.forward(pa, Q, K, V, whiten=s)).max() < 1e-12
    gf = oracle.backward(pf, Q, K, V, dO, whiten=s)
    ga = oracle.backward(pa, Q, K, V, dO, whiten=s)
    for a, b in zip(gf[:3], ga[:3]):
        assert np.abs(a - b).max() < 1e-10 * max(1.0, np.abs(b).max())
    assert ga[3] is None and gf[3].shape == p.lm_filter.shape


def test_filter_selection_adjoint_identity():
    p, _, K, _, _, _ = _case(7, gh=8, gw=6, mh=2, mw=3, prefix=2)
    rng = np.random.default_rng(70)
    U = rng.standard_normal((p.B, p.H, p.m, p.d))
    lhs = float((oracle.landmarks_pool(p, K) * U).sum())
    back = oracle.landmarks_pool_bwd(p, U)
    assert lhs == pytest.approx(float((K * back).sum()), rel=1e-12)
    assert np.abs(back[:, :, :p.prefix, :]).max() == 0.0            # class tokens are not selected from


@pytest.mark.parametrize("lm_mode", [1, 2])
def test_filter_backward_finite_differences(lm_mode):
    p, Q, K, V, dO, s = _case(11 + lm_mode, lm_mode=lm_mode, B=2, H=2, gh=4, gw=6, mh=2, mw=3, d=5, prefix=1, T=4)
    dQ, dK, dV, dF = oracle.backward(p, Q, K, V, dO, whiten=s)
    h = 1e-6

    def loss(q, k, v, f):
        return float((oracle.forward(replace(p, lm_filter=f), q, k, v, whiten=s) * dO).sum())

    F = p.lm_filter
    for name, arr, grad in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        for idx in [(0, 0, 0, 0), (1, 1, 7, 3), (0, 1, 24, 4), (1, 0, 13, 2)]:
            a = {"Q": Q, "K": K, "V": V}
            plus, minus = dict(a), dict(a)
            plus[name] = arr.copy(); plus[name][idx] += h
            minus[name] = arr.copy(); minus[name][idx] -= h
            fd = (loss(plus["Q"], plus["K"], plus["V"], F) - loss(minus["Q"], minus["K"], minus["V"], F)) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=5e-6, abs=1e-8), (name, idx)
    # the filter's own gradient: it is shared by the batch elements of a head, so both contribute
    for idx in [(0, 0, 0), (1, 3, 4), (0, 2, 1), (1, 0, 2)]:
        fp = F.copy(); fp[idx] += h
        fm = F.copy(); fm[idx] -= h
        fd = (loss(Q, K, V, fp) - loss(Q, K, V, fm)) / (2 * h)
        assert dF[idx] == pytest.approx(fd, rel=5e-6, abs=1e-8), idx
