"""The no-allocation entry point, ns_pinv_static, against the ordinary ns_pinv.

ns_pinv_static is for callers that cannot call cudaMalloc (a serving loop with a fully committed
memory pool, a plug-in that only gets input/output pointers): its scratch is a fixed array inside
the library.  This file is collected last on purpose, so that a run that stops at the first
failure has already been through every other test.  It has to pass on its own in a fresh process
and after all the others, and on two calls in a row, because every call reuses the same scratch
with the previous call's contents still in it.
"""
import numpy as np
import pytest
import torch

import paper_2604_20368_b200 as ln
from paper_2604_20368_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _matrices(batch, m, seed):
    # symmetric, unit diagonal, positive definite: Laplacian kernel of random points, built on the host
    pts = np.random.default_rng(seed).standard_normal((batch, m, 16))
    dist = np.abs(pts[:, :, None, :] - pts[:, None, :, :]).sum(-1)
    return torch.from_numpy(np.exp(-dist / 16.0).astype(np.float32)).to(DEV)


def _rel(a, b):
    return float((a - b).norm() / b.norm())


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    calls = [(_matrices(6, 49, 1), 6, 1e-6), (_matrices(3, 64, 2), 8, 1e-6)]
    for W, T, eps in calls:                      # second call finds the first call's leftovers in the scratch
        ref, _, ref_resid = ln.ns_pinv(W, T, ridge_eps=eps, want_resid=True)
        X = torch.full_like(W, float("nan"))     # outputs are the caller's, allocated up front
        resid = torch.full((W.shape[0],), float("nan"), device=DEV)
        ln.ns_pinv_static(W, T, X, ridge_eps=eps, resid=resid)
        torch.cuda.synchronize()
        assert torch.isfinite(X).all()
        assert _rel(X, ref) < 2e-5               # same tolerance as the ns_pinv parity test
        assert torch.allclose(resid, ref_resid, rtol=1e-3, atol=1e-4)
    # and once more on the first problem, now with the second call's contents lying around
    W, T, eps = calls[0]
    X = torch.empty_like(W)
    ln.ns_pinv_static(W, T, X, ridge_eps=eps)
    assert _rel(X, ln.ns_pinv(W, T, ridge_eps=eps)[0]) < 2e-5


def test_static_scratch_limit_is_reported_and_nothing_runs():
    lib = binding.lib()
    limit = lib.ns_pinv_static_scratch_bytes()
    assert limit == 8 << 20
    batch, m, T = 64, 128, 8                     # needs far more than the fixed scratch
    assert lib.ns_pinv_workspace_bytes(batch, m, T) > limit
    W = torch.zeros(batch, m, m, device=DEV)
    X = torch.zeros(batch, m, m, device=DEV)
    with pytest.raises(ln.LnError) as e:
        ln.ns_pinv_static(W, T, X)
    assert e.value.status == -5 and "static scratch" in str(e.value)
    torch.cuda.synchronize()
    assert float(X.abs().max()) == 0.0           # rejected on the host: the output was not touched
    assert lib.ln_status_string(-5).startswith(b"problem exceeds the static scratch")
