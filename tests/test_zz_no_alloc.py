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

import oracle
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
        assert torch.equal(X, ref)               # in fact the same kernel on other scratch: the same bits
        assert torch.equal(resid, ref_resid)
        # and against the float64 oracle's Alg. 2 iterate, at the bar the ns_pinv parity test uses
        Xo = oracle.ns_pinv(W.cpu().double().numpy(), T, eps=float(np.float32(eps)))[0]
        assert float(np.linalg.norm(X.cpu().double().numpy() - Xo) / np.linalg.norm(Xo)) < 2e-5
    # and once more on the first problem, now with the second call's contents lying around
    W, T, eps = calls[0]
    X = torch.empty_like(W)
    ln.ns_pinv_static(W, T, X, ridge_eps=eps)
    assert torch.equal(X, ln.ns_pinv(W, T, ridge_eps=eps)[0])


def test_static_scratch_call_allocates_nothing():
    """Free device memory as the driver reports it, and what torch's allocator holds, are the same before and
    after a call: the entry point takes its scratch from the library image, not from an allocator."""
    W = _matrices(4, 49, 3)
    X = torch.empty_like(W)
    ln.ns_pinv_static(W, 6, X)                   # first call on the device: looks up the scratch address
    torch.cuda.synchronize()
    free0, reserved0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved(), torch.cuda.memory_allocated()
    for _ in range(3):
        ln.ns_pinv_static(W, 6, X)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_reserved() == reserved0 and torch.cuda.memory_allocated() == alloc0


def test_static_scratch_largest_documented_case_and_first_one_beyond():
    lib = binding.lib()
    limit = lib.ns_pinv_static_scratch_bytes()
    batch, m, T = 2, 256, 8                      # the largest case the header names: just under the limit
    assert lib.ns_pinv_workspace_bytes(batch, m, T) <= limit < lib.ns_pinv_workspace_bytes(batch, m, T + 2)
    W = _matrices(batch, m, 4)
    X = torch.empty_like(W)
    ln.ns_pinv_static(W, T, X)
    assert torch.equal(X, ln.ns_pinv(W, T)[0])
    with pytest.raises(ln.LnError) as e:         # two more iterates no longer fit
        ln.ns_pinv_static(W, T + 2, X)
    assert e.value.status == -5


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
