"""GPU parity: the CUDA library, called through its C ABI, against the float64 oracle on the same
seeded inputs, element by element.  Tolerances are norm-wise relative errors: 1e-4 for fp32
storage, 2e-2 for bf16 storage (outputs and gradients alike)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_20368_b200 as ln
from paper_2604_20368_b200 import synth
from parity import (TOL, TOL_INTERMEDIATE, assert_parity, compare, compare_intermediates, f64, oracle_problem, rel_err,
                    run_gpu, run_oracle_heads)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _rand(shape, seed, dtype):
    x = torch.from_numpy(np.random.default_rng(seed).standard_normal(shape, dtype=np.float32))
    return x.to(dtype)


# ------------------------------------------------------------------------------------------ l1_kernel
@pytest.mark.parametrize("batch,na,nb,d", [(3, 197, 49, 64), (1, 1, 1, 1), (2, 130, 131, 7), (1, 300, 70, 128),
                                           (2, 64, 256, 32), (1, 129, 65, 40)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_l1_kernel(batch, na, nb, d, dtype):
    A, Bm = _rand((batch, na, d), 1, dtype), _rand((batch, nb, d), 2, dtype)
    lam = float(max(d, 2))
    K, rs = ln.l1_kernel(A.to(DEV), Bm.to(DEV), lam, want_rowsum=True)
    Ko, rso = oracle.l1_kernel(f64(A), f64(Bm), lam, want_rowsum=True)
    assert rel_err(f64(K), Ko) < 2e-6
    assert np.abs(f64(K) - Ko).max() < 4e-6
    assert rel_err(f64(rs), rso) < 2e-6


@pytest.mark.parametrize("batch,na,nb,d", [(1, 300, 1000, 64), (2, 64, 2049, 32), (1, 1025, 513, 128), (1, 8, 4100, 40)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_l1_kernel_few_large_blocks_split_their_columns(batch, na, nb, d, dtype):
    """Few, large blocks without row sums (the setting of the paper's kernel micro-benchmark, Sec. 4.3): the launch
    splits the column range over the grid's third dimension; ragged last tiles in both directions."""
    A, Bm = _rand((batch, na, d), 11, dtype), _rand((batch, nb, d), 12, dtype)
    lam = float(max(d, 2))
    K = ln.l1_kernel(A.to(DEV), Bm.to(DEV), lam)
    Ko = oracle.l1_kernel(f64(A), f64(Bm), lam)
    assert rel_err(f64(K), Ko) < 2e-6
    assert np.abs(f64(K) - Ko).max() < 4e-6
    # and the same values as the unsplit launch that also returns row sums
    K2, _ = ln.l1_kernel(A.to(DEV), Bm.to(DEV), lam, want_rowsum=True)
    assert torch.equal(K, K2)


@pytest.mark.parametrize("batch,na,nb,d", [(1, 300, 777, 64), (2, 130, 1000, 32), (1, 70, 2049, 128)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_l1_kernel_bwd_few_large_blocks(batch, na, nb, d, dtype):
    """Gradient of few, large kernel blocks: the pass over the rows splits the columns into partial sums; the upstream
    factor dK o K / lambda is formed inside the two sign kernels."""
    A, Bm = _rand((batch, na, d), 14, dtype), _rand((batch, nb, d), 15, dtype)
    A[0, 3] = Bm[0, 700]                                   # exact ties in the last column range: sign(0) = 0
    A[0, 4, : d // 2] = Bm[0, 2, : d // 2]
    dK = _rand((batch, na, nb), 16, torch.float32)
    lam = float(d)
    for Kmat in (None, ln.l1_kernel(A.to(DEV), Bm.to(DEV), lam)):
        dA, dB = ln.l1_kernel_bwd(A.to(DEV), Bm.to(DEV), lam, dK.to(DEV), Kmat=Kmat)
        dAo, dBo = oracle.l1_kernel_bwd(f64(A), f64(Bm), lam, f64(dK))
        tol = 1e-5 if dtype == torch.float32 else 5e-3    # bf16: only the output rounding
        assert rel_err(f64(dA), dAo) < tol
        assert rel_err(f64(dB), dBo) < tol


def test_l1_kernel_exact_properties():
    A = _rand((2, 90, 64), 3, torch.float32).to(DEV)
    K = ln.l1_kernel(A, A, 64.0)
    assert torch.equal(K, K.transpose(1, 2))                      # |a-b| = |b-a| in the same order
    assert torch.equal(torch.diagonal(K, dim1=1, dim2=2), torch.ones(2, 90, device=DEV))


@pytest.mark.parametrize("batch,na,nb,d", [(2, 197, 49, 64), (1, 70, 130, 32), (1, 33, 5, 128), (3, 1, 1, 32)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("recompute", [False, True])
def test_l1_kernel_bwd(batch, na, nb, d, dtype, recompute):
    A, Bm = _rand((batch, na, d), 4, dtype), _rand((batch, nb, d), 5, dtype)
    if na > 4 and nb > 2:                 # exact ties: sign(0) = 0 on both sides
        A[0, 3] = Bm[0, 1]
        A[0, 4, : d // 2] = Bm[0, 2, : d // 2]
    dK = _rand((batch, na, nb), 6, torch.float32)
    lam = float(d)
    Kmat = None if recompute else ln.l1_kernel(A.to(DEV), Bm.to(DEV), lam)
    dA, dB = ln.l1_kernel_bwd(A.to(DEV), Bm.to(DEV), lam, dK.to(DEV), Kmat=Kmat)
    dAo, dBo = oracle.l1_kernel_bwd(f64(A), f64(Bm), lam, f64(dK))
    tol = 1e-5 if dtype == torch.float32 else 5e-3    # bf16: only the output rounding
    assert rel_err(f64(dA), dAo) < tol
    assert rel_err(f64(dB), dBo) < tol


# ------------------------------------------------------------------------------------------ ns_pinv
def _kernel_matrices(batch, m, d, seed):
    pts = np.random.default_rng(seed).standard_normal((batch, m, d))
    return oracle.l1_kernel(pts, pts, float(d)).astype(np.float32)


@pytest.mark.parametrize("m,T", [(1, 0), (1, 3), (5, 4), (49, 6), (64, 8), (130, 8), (256, 12), (32, 0)])
def test_ns_pinv(m, T):
    W = _kernel_matrices(3, m, 16, 7)
    X, hist, resid = ln.ns_pinv(torch.from_numpy(W).to(DEV), T, ridge_eps=1e-6, want_hist=True, want_resid=True)
    Xo, resido, alphao, histo = oracle.ns_pinv(W, T, eps=float(np.float32(1e-6)), want_hist=True)
    assert rel_err(f64(X), Xo) < 2e-5
    if T > 0:
        assert rel_err(f64(hist)[:, :T], histo) < 2e-5
    assert rel_err(f64(hist)[:, T], Xo) < 2e-5
    assert np.allclose(f64(resid), resido, rtol=1e-3, atol=1e-4)


def test_ns_pinv_converges_and_given_alpha():
    W = _kernel_matrices(2, 24, 8, 8)
    X, _, resid = ln.ns_pinv(torch.from_numpy(W).to(DEV), 40, ridge_eps=0.0, want_resid=True)
    eye = np.eye(24)
    for b in range(2):
        assert np.abs(f64(X)[b] @ W[b].astype(np.float64) - eye).max() < 5e-3   # fp32 limit at cond ~ 1e2
    Xa, _, _ = ln.ns_pinv(torch.from_numpy(W).to(DEV), 3, alpha=0.01)
    Xo, _, _ = oracle.ns_pinv(W, 3, alpha=float(np.float32(0.01)))
    assert rel_err(f64(Xa), Xo) < 2e-5


@pytest.mark.parametrize("m,T", [(1, 2), (5, 4), (49, 6), (64, 8), (130, 4), (256, 4), (16, 0)])
@pytest.mark.parametrize("given_hist", [False, True])
def test_ns_pinv_bwd(m, T, given_hist):
    W = _kernel_matrices(2, m, 16, 9)
    dX = np.random.default_rng(10).standard_normal((2, m, m)).astype(np.float32)
    Wd = torch.from_numpy(W).to(DEV)
    hist = ln.ns_pinv(Wd, T, ridge_eps=1e-6, want_hist=True)[1] if given_hist else None
    dW = ln.ns_pinv_bwd(Wd, T, 1e-6, 0.0, torch.from_numpy(dX).to(DEV), X_hist=hist)
    dWo = oracle.ns_pinv_bwd(W, T, float(np.float32(1e-6)), 0.0, dX)
    assert rel_err(f64(dW), dWo) < 1e-4
    a = float(np.float32(0.9 / (m * m)))          # a given alpha inside the convergence region
    dWa = ln.ns_pinv_bwd(Wd, T, 1e-6, a, torch.from_numpy(dX).to(DEV))
    dWao = oracle.ns_pinv_bwd(W, T, float(np.float32(1e-6)), a, dX)
    assert rel_err(f64(dWa), dWao) < 1e-4


# ------------------------------------------------------------------------------------------ pooling
@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg4a"])
def test_landmarks_pool_fwd_bwd(name):
    cfg = synth.shrink(synth.CONFIGS[name], B=1, H=2)
    inp = synth.make_inputs(cfg)
    p = ln.problem_from_config(cfg)
    op = oracle.Problem(B=1, H=2, n=cfg.n, d=cfg.d, m=cfg.m, lam=cfg.lam, ns_iters=0, prefix=cfg.prefix,
                        gh=cfg.gh, gw=cfg.gw, mh=cfg.mh, mw=cfg.mw)
    L = ln.landmarks_pool(p, inp["K"].to(DEV))
    Lo = oracle.landmarks_pool(op, f64(inp["K"]))
    assert rel_err(f64(L), Lo) < 1e-6
    dL = torch.from_numpy(np.random.default_rng(11).standard_normal((1, 2, cfg.m, cfg.d), dtype=np.float32))
    dK = ln.landmarks_pool_bwd(p, dL.to(DEV))
    dKo = oracle.landmarks_pool_bwd(op, f64(dL))
    assert rel_err(f64(dK), dKo) < (1e-6 if cfg.dtype == "f32" else 4e-3)


# ------------------------------------------------------------------------------------------ whole path
def _run_case(cfg, use_whiten=True, map_mode=1, backward=True, heads=None, tol=None, intermediates=False):
    inp = synth.make_inputs(cfg)
    heads = list(range(cfg.B * cfg.H)) if heads is None else heads
    g = run_gpu(cfg, inp, use_whiten=use_whiten, map_mode=map_mode, backward=backward)
    assert int(g["status"].abs().max()) == 0
    if backward:
        assert int(g["status_bwd"].abs().max()) == 0
    o = run_oracle_heads(cfg, inp, heads, use_whiten=use_whiten, map_mode=map_mode, backward=backward)
    errs = compare(cfg, g, o, heads)
    print(cfg.name, {k: {a: f"{b:.1e}" for a, b in e.items()} for k, e in errs.items()})
    assert_parity(cfg, errs, tol)
    if intermediates and backward:
        ierr = compare_intermediates(cfg, g, inp, heads, use_whiten=use_whiten, map_mode=map_mode)
        print(cfg.name, "intermediates", {k: f"{v:.1e}" for k, v in ierr.items()})
        for k, e in ierr.items():
            assert e < TOL_INTERMEDIATE[cfg.dtype], (cfg.name, k, ierr)
    return errs


def test_cfg1_tiny_fp32_forward():
    _run_case(synth.CONFIGS["cfg1"], backward=False)


def test_cfg1_fp32_forward_and_backward():
    from dataclasses import replace
    _run_case(replace(synth.CONFIGS["cfg1"], backward=True))


@pytest.mark.parametrize("use_whiten,map_mode", [(True, 1), (False, 1), (False, 0)])
def test_cfg2_shape_small_batch(use_whiten, map_mode):
    _run_case(synth.shrink(synth.CONFIGS["cfg2"], B=2), use_whiten=use_whiten, map_mode=map_mode, intermediates=True)


def test_cfg2_shape_fp32_storage():
    from dataclasses import replace
    _run_case(replace(synth.shrink(synth.CONFIGS["cfg2"], B=1), dtype="f32"), intermediates=True)


def test_cfg3_shape_small_batch():
    _run_case(synth.shrink(synth.CONFIGS["cfg3"], B=2), intermediates=True)


def test_cfg4a_shape_small_batch():
    _run_case(synth.shrink(synth.CONFIGS["cfg4a"], B=1), intermediates=True)


@pytest.mark.parametrize("name", ["cfg5_m64_T4", "cfg5_m128_T8", "cfg5_m256_T12"])
def test_cfg5_shape_small_batch(name):
    _run_case(synth.shrink(synth.CONFIGS[name], B=1, H=2), intermediates=True)


# The high-resolution sweep at its full token counts (one head each: up to 16 token chunks per head, the largest
# offsets into the saved kernel blocks, the pooling adjoint over 112 x 112 and 224 x 224 grids).
@pytest.mark.parametrize("name", ["cfg4b", "cfg4c"])
def test_cfg4_full_token_count_one_head(name):
    _run_case(synth.shrink(synth.CONFIGS[name], B=1, H=1))


# The solver-stress configurations at their full batch (128 heads in flight, every head with its own duplicated
# landmark bins), eight sampled heads against the oracle.
@pytest.mark.parametrize("name", ["cfg5_m64_T4", "cfg5_m128_T8", "cfg5_m256_T12"])
def test_cfg5_full_size_sampled_heads(name):
    _run_case(synth.CONFIGS[name], heads=[0, 1, 17, 42, 63, 64, 100, 127])


def test_bins_equal_grid_every_key_ties_with_its_landmark_bf16():
    """bins == grid: every landmark IS a key, so sign(key - landmark) is an exact tie in all d dims for n pairs, the
    case the folded saturating step (one multiply-add for subtraction and sign) has to get exactly right."""
    cfg = synth.Config("ties", B=1, H=2, d=64, m=81, T=6, gh=9, gw=9, mh=9, mw=9, prefix=2, dtype="bf16", seed=9)
    inp = synth.make_inputs(cfg)
    inp["Q"][0, 0, 5] = inp["K"][0, 0, 2 + 7]          # a query that coincides with a landmark as well
    inp["Q"][0, 1, 11, :32] = inp["K"][0, 1, 2 + 40, :32]
    heads = [0, 1]
    g = run_gpu(cfg, inp)
    o = run_oracle_heads(cfg, inp, heads)
    errs = compare(cfg, g, o, heads)
    print(cfg.name, {k: {a: f"{b:.1e}" for a, b in e.items()} for k, e in errs.items()})
    assert_parity(cfg, errs)


def test_cfg2_full_size_sampled_heads():
    cfg = synth.CONFIGS["cfg2"]
    heads = [0, 1, 5, 6, 100, 191, 192, 300, 382, 383]
    _run_case(cfg, heads=heads)


def test_cfg3_full_size_sampled_heads():
    cfg = synth.CONFIGS["cfg3"]
    _run_case(cfg, heads=[0, 13, 31])



# Ragged shapes for the fused sign pass (token tiles of 8 * TG tokens, rounds of 8 landmarks, several token
# chunks per head, two 64-dim slabs) and for the per-head kernels (m <= 64, 64 < m <= 128, clustered m > 128).
@pytest.mark.parametrize("gh,gw,mh,mw,prefix,d,dtype", [
    (5, 7, 3, 3, 2, 64, "bf16"),        # n = 37 (one short tile), m = 9 (second round nearly empty)
    (23, 31, 5, 10, 1, 128, "bf16"),    # n = 714, m = 50: ragged last tile and last round, two slabs
    (40, 40, 9, 9, 0, 64, "bf16"),      # n = 1600, m = 81: tensor-core path for 64 < m <= 128, overlapping bins
    (36, 36, 12, 12, 3, 128, "bf16"),   # n = 1299, m = 144: clustered per-head kernels, m not a multiple of 8 * 128
    (9, 9, 3, 3, 0, 64, "f32"),         # fp32 storage through the fused pass
])
def test_ragged_shapes(gh, gw, mh, mw, prefix, d, dtype):
    cfg = synth.Config("ragged", B=2, H=2, d=d, m=mh * mw, T=5, gh=gh, gw=gw, mh=mh, mw=mw, prefix=prefix,
                       dtype=dtype, seed=77)
    _run_case(cfg)


# Every size class of the tcgen05 Newton-Schulz engines (M = 64 accumulators, M = 128, 2 x 2 blocks shared by a
# cluster) at its edges: m just above a class boundary, m one short of the padded size, and zero, one and several steps.
@pytest.mark.parametrize("mh,mw", [(1, 1), (7, 9), (8, 8), (5, 13), (8, 16), (10, 13), (15, 17), (16, 16)])
@pytest.mark.parametrize("T", [0, 1, 3])
def test_newton_schulz_engines_at_their_edges(mh, mw, T):
    cfg = synth.Config("ns_edges", B=1, H=2, d=64, m=mh * mw, T=T, gh=20, gw=20, mh=mh, mw=mw, prefix=1,
                       dtype="bf16", seed=123 + mh * mw + T)
    _run_case(cfg)


def test_many_heads_several_chunks():
    """Few heads and many tokens: the landmark gradient is summed over several token chunks per head."""
    cfg = synth.Config("chunks", B=1, H=1, d=64, m=32, T=4, gh=96, gw=96, mh=4, mw=8, dtype="bf16", seed=5)
    _run_case(cfg)

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_given_landmarks_and_their_gradient(dtype):
    # lm_mode 0: caller-provided landmarks, dL returned
    rng = np.random.default_rng(21)
    B, H, n, d, m, T = 1, 2, 150, 32, 20, 5
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    Q, K, V, dO = (torch.from_numpy(rng.standard_normal((B, H, n, d), dtype=np.float32)).to(td) for _ in range(4))
    L = torch.from_numpy(rng.standard_normal((B, H, m, d), dtype=np.float32)).to(td)
    wh = torch.from_numpy(rng.uniform(0.5, 2.0, (H, m)).astype(np.float32))
    p = ln.Problem(B=B, H=H, n=n, d=d, m=m, lam=float(d), ns_iters=T, dtype=ln.LN_F32 if dtype == "f32" else ln.LN_BF16,
                   whiten=wh.to(DEV), lm_mode=0)
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=DEV)
    args = [t.to(DEV) for t in (Q, K, V)]
    O = ln.laplace_nystrom_fwd(p, *args, L=L.to(DEV), saved=saved)
    dQ, dK, dV, dL = ln.laplace_nystrom_bwd(p, *args, dO.to(DEV), saved, L=L.to(DEV))
    op = oracle.Problem(B=B, H=H, n=n, d=d, m=m, lam=float(d), ns_iters=T, ridge_eps=float(np.float32(1e-6)), lm_mode=0)
    Oo = oracle.forward(op, f64(Q), f64(K), f64(V), L=f64(L), whiten=f64(wh))
    dQo, dKo, dVo, dLo = oracle.backward(op, f64(Q), f64(K), f64(V), f64(dO), L=f64(L), whiten=f64(wh))
    for name, got, ref in (("O", O, Oo), ("dQ", dQ, dQo), ("dK", dK, dKo), ("dV", dV, dVo), ("dL", dL, dLo)):
        assert rel_err(f64(got), ref) < TOL[dtype], name


@pytest.mark.parametrize("lm_mode,name,B,H,fused", [
    (2, "cfg2", 2, 2, True), (2, "cfg1", 1, 2, True), (2, "cfg5_m128_T8", 1, 1, True), (2, "cfg4a", 1, 1, True),
    (3, "cfg2", 2, 2, True), (3, "cfg2", 1, 2, False), (3, "cfg1", 1, 2, True), (3, "cfg3", 1, 2, True),
    (3, "cfg5_m128_T8", 1, 1, True), (3, "cfg4a", 1, 1, True), (3, "cfg5_m256_T4", 1, 1, True)])
def test_landmarks_pooled_from_queries(lm_mode, name, B, H, fused):
    """lm_mode 2 (Sec. 4.2 pools the query tensor): L = pool(Q); the landmark gradient returns to dQ.
    lm_mode 3 (Alg. 1 as printed): two landmark sets, C = k(Q, pool K), W = k(pool Q, pool K), R = k(pool Q, K); W is
    not symmetric, and both landmark gradients return to their tensors through the pooling adjoint."""
    from dataclasses import replace
    cfg = replace(synth.shrink(synth.CONFIGS[name], B=B, H=H), backward=True)
    inp = synth.make_inputs(cfg)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    p = ln.problem_from_config(cfg, whiten=inp["whiten"].to(DEV))
    p.lm_mode = lm_mode
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=DEV)
    status = torch.full((cfg.B * cfg.H,), -1, dtype=torch.int32, device=DEV)
    was = ln.set_fused_sign(fused)
    try:
        O = ln.laplace_nystrom_fwd(p, Q, K, V, saved=saved, dev_status=status)
        dQ, dK, dV, dL = ln.laplace_nystrom_bwd(p, Q, K, V, dO, saved)
    finally:
        ln.set_fused_sign(was)
    assert dL is None
    assert int(status.abs().max()) == 0
    op = oracle_problem(cfg, lm_mode=lm_mode)
    wh = f64(inp["whiten"])
    Oo = oracle.forward(op, f64(inp["Q"]), f64(inp["K"]), f64(inp["V"]), whiten=wh)
    dQo, dKo, dVo, _ = oracle.backward(op, f64(inp["Q"]), f64(inp["K"]), f64(inp["V"]), f64(inp["dO"]), whiten=wh)
    from parity import metrics
    BH = cfg.B * cfg.H
    errs = {k: metrics(f64(g).reshape(BH, cfg.n, cfg.d), r.reshape(BH, cfg.n, cfg.d), cfg.dtype == "bf16")
            for k, g, r in (("O", O, Oo), ("dQ", dQ, dQo), ("dK", dK, dKo), ("dV", dV, dVo))}
    print(cfg.name, "lm_mode", lm_mode, {k: {a: f"{b:.1e}" for a, b in e.items()} for k, e in errs.items()})
    assert_parity(cfg, errs)


@pytest.mark.parametrize("lm_mode,name,B,H,dtype", [(1, "cfg2", 3, 2, "bf16"), (2, "cfg2", 2, 2, "bf16"), (1, "cfg2", 2, 2, "f32"),
                                                    (1, "cfg3", 2, 1, "bf16"), (1, "cfg5_m128_T8", 2, 2, "bf16"),
                                                    (2, "cfg5_m256_T4", 1, 2, "bf16"), (1, "cfg5_m64_T4", 2, 1, "f32")])
def test_landmarks_selected_by_a_depthwise_filter(lm_mode, name, B, H, dtype):
    """Sec. 4.2's alternative landmark selection: one r x r filter per head and channel, stride r, in place of the
    average over a region; the backward pass also returns the filter's gradient, summed over the batch."""
    from dataclasses import replace
    from parity import metrics
    cfg = replace(synth.shrink(synth.CONFIGS[name], B=B, H=H), backward=True, dtype=dtype)
    inp = synth.make_inputs(cfg)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    taps = (cfg.gh // cfg.mh) * (cfg.gw // cfg.mw)
    rng = np.random.default_rng(cfg.seed + 77)
    F = torch.from_numpy((rng.standard_normal((cfg.H, taps, cfg.d)) / taps + 1.0 / taps).astype(np.float32))
    p = ln.problem_from_config(cfg, whiten=inp["whiten"].to(DEV))
    p.lm_mode = lm_mode
    p.lm_filter = F.to(DEV)
    p.lm_filter_grad = torch.full_like(p.lm_filter, float("nan"))
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=DEV)
    O = ln.laplace_nystrom_fwd(p, Q, K, V, saved=saved)
    dQ, dK, dV, _ = ln.laplace_nystrom_bwd(p, Q, K, V, dO, saved)
    op = replace(oracle_problem(cfg, lm_mode=lm_mode), lm_filter=np.ascontiguousarray(F.numpy().astype(np.float64)))
    wh = f64(inp["whiten"])
    q, k, v, g = (f64(inp[x]) for x in ("Q", "K", "V", "dO"))
    Oo = oracle.forward(op, q, k, v, whiten=wh)
    dQo, dKo, dVo, dFo = oracle.backward(op, q, k, v, g, whiten=wh)
    BH = cfg.B * cfg.H
    errs = {kk: metrics(f64(a).reshape(BH, cfg.n, cfg.d), r.reshape(BH, cfg.n, cfg.d), cfg.dtype == "bf16")
            for kk, a, r in (("O", O, Oo), ("dQ", dQ, dQo), ("dK", dK, dKo), ("dV", dV, dVo))}
    print(cfg.name, "filter selection, lm_mode", lm_mode, {kk: {a: f"{b:.1e}" for a, b in e.items()} for kk, e in errs.items()})
    assert_parity(cfg, errs)
    # the filter's gradient is fp32 whatever the storage type: held to the fp32 bar of the gradients it is summed from
    # (for bf16 storage the upstream dL carries the rounding of the bf16 inputs only, not of an output)
    e = rel_err(f64(p.lm_filter_grad), dFo)
    print("   filter gradient", f"{e:.1e}")
    assert e < (1e-4 if dtype == "f32" else 1e-3)


@pytest.mark.parametrize("name,B,H,dtype,T,lm_mode,ridge", [
    ("cfg1", 2, 2, "f32", 6, 1, 1e-6), ("cfg2", 2, 2, "bf16", 6, 1, 1e-6), ("cfg2", 1, 2, "f32", 0, 1, 1e-6),
    ("cfg2", 1, 2, "bf16", 1, 2, 1e-6), ("cfg3", 1, 2, "bf16", 4, 1, 1e-6), ("cfg4a", 1, 1, "bf16", 4, 1, 1e-6),
    ("cfg5_m128_T8", 1, 2, "bf16", 4, 1, 1e-6), ("cfg5_m256_T4", 1, 1, "bf16", 4, 1, 1e-6),
    ("cfg5_m64_T4", 1, 2, "f32", 12, 1, 1e-2)])
def test_conjugate_gradient_solver(name, B, H, dtype, T, lm_mode, ridge):
    """solver = 1 (Sec. 5.3, Table 4): Y from T steps of conjugate gradients on (W + eps I) Y = M; the backward pass
    solves the adjoint system by the same T steps.  Forward and backward against the oracle's plain CG.

    The step counts are the ones at which the T-step iterate is a stable function of its inputs.  Measured with the
    oracle alone (a relative perturbation of 1e-7 of the right-hand side, change of the iterate): 1e-5 at T = 4 on
    every shape here (the columns of M = R V lie almost along one eigenvector, and the other components decide the
    iterate), but 2.5e-4 on cfg3 at T = 6, 2.5e-2 on cfg4a at T = 6, 1e-2 on cfg5 m = 256 at T = 6 and 4e-2 on the
    adjoint solve of cfg5 m = 128 at T = 8, the same for a perturbation of 1e-5: the iterate jumps where a step reaches
    the small end of the spectrum (cfg5 duplicates landmarks: W is singular up to the ridge).  No two precisions agree
    there, whatever the implementation; the device runs the recurrence in double precision and differs from the
    oracle through the rounding of M, dY and W only."""
    from dataclasses import replace
    from parity import metrics
    cfg = replace(synth.shrink(synth.CONFIGS[name], B=B, H=H), backward=True, dtype=dtype, T=T, ridge_eps=ridge)
    inp = synth.make_inputs(cfg)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    p = ln.problem_from_config(cfg, whiten=inp["whiten"].to(DEV))
    p.lm_mode = lm_mode
    p.solver = 1
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=DEV)
    status = torch.full((cfg.B * cfg.H,), -1, dtype=torch.int32, device=DEV)
    O = ln.laplace_nystrom_fwd(p, Q, K, V, saved=saved, dev_status=status)
    dQ, dK, dV, _ = ln.laplace_nystrom_bwd(p, Q, K, V, dO, saved)
    assert int(status.abs().max()) == 0
    op = replace(oracle_problem(cfg, lm_mode=lm_mode), solver=1)
    wh = f64(inp["whiten"])
    q, k, v, g = (f64(inp[x]) for x in ("Q", "K", "V", "dO"))
    Oo = oracle.forward(op, q, k, v, whiten=wh)
    dQo, dKo, dVo, _ = oracle.backward(op, q, k, v, g, whiten=wh)
    # the two solvers do differ on this input (otherwise the comparison would not show which one ran)
    if T > 0:
        O_ns = oracle.forward(replace(op, solver=0), q, k, v, whiten=wh)
        assert rel_err(O_ns, Oo) > 1e-3
    BH = cfg.B * cfg.H
    errs = {kk: metrics(f64(a).reshape(BH, cfg.n, cfg.d), r.reshape(BH, cfg.n, cfg.d), cfg.dtype == "bf16")
            for kk, a, r in (("O", O, Oo), ("dQ", dQ, dQo), ("dK", dK, dKo), ("dV", dV, dVo))}
    print(cfg.name, "conjugate gradients, T", T, {kk: {a: f"{b:.1e}" for a, b in e.items()} for kk, e in errs.items()})
    assert_parity(cfg, errs)


@pytest.mark.parametrize("name,B,H,dtype", [("cfg2", 3, 2, "bf16"), ("cfg2", 2, 1, "f32"), ("cfg4a", 2, 1, "bf16"),
                                            ("cfg5_m64_T4", 2, 1, "bf16"), ("cfg1", 2, 2, "f32")])
def test_batch_statistic_whitening_training_mode(name, B, H, dtype):
    """whiten_mode 1 (Eq. 5-6 in training mode): the scale is estimated inside the kernel that forms C = k(Q, L), over
    the query rows of every batch element of a head, and the backward pass differentiates through the variance."""
    from dataclasses import replace
    from parity import metrics
    cfg = replace(synth.shrink(synth.CONFIGS[name], B=B, H=H), backward=True, dtype=dtype)
    inp = synth.make_inputs(cfg)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    eps_w = 1e-5
    p = ln.problem_from_config(cfg, whiten=None)
    p.whiten_mode, p.whiten_eps = 1, eps_w
    p.whiten_batch = torch.full((cfg.H, cfg.m), float("nan"), device=DEV)
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=DEV)
    O = ln.laplace_nystrom_fwd(p, Q, K, V, saved=saved)
    dQ, dK, dV, _ = ln.laplace_nystrom_bwd(p, Q, K, V, dO, saved)
    op = oracle_problem(cfg)
    q, k, v, g = (f64(inp[x]) for x in ("Q", "K", "V", "dO"))
    Oo, so = oracle.forward_batch_whiten(op, q, k, v, eps_w)
    dQo, dKo, dVo, _, _ = oracle.backward_batch_whiten(op, q, k, v, g, eps_w)
    assert rel_err(f64(p.whiten_batch), so) < 1e-4
    BH = cfg.B * cfg.H
    errs = {kk: metrics(f64(a).reshape(BH, cfg.n, cfg.d), r.reshape(BH, cfg.n, cfg.d), dtype == "bf16")
            for kk, a, r in (("O", O, Oo), ("dQ", dQ, dQo), ("dK", dK, dKo), ("dV", dV, dVo))}
    print(cfg.name, "batch whitening", {kk: {a: f"{b:.1e}" for a, b in e.items()} for kk, e in errs.items()})
    assert_parity(cfg, errs)
    # the variance path is really there: against the constant-scale gradient the query gradient differs visibly
    dQc = oracle.backward(op, q, k, v, g, whiten=so)[0]
    assert rel_err(f64(dQ), dQc) > 5 * rel_err(f64(dQ), dQo)


def test_inference_without_saved_matches_training_forward():
    cfg = synth.shrink(synth.CONFIGS["cfg2"], B=1)
    inp = synth.make_inputs(cfg)
    a = run_gpu(cfg, inp, backward=False)["O"]
    b = run_gpu(cfg, inp, backward=True)["O"]
    assert torch.equal(a, b)


def test_m_equals_n_reproduces_exact_attention_on_gpu():
    # landmarks = keys (bins == grid), many Newton-Schulz steps: Nystrom is exact (oracle pin, here on GPU)
    cfg = synth.Config("mn", B=1, H=2, d=32, m=48, T=40, gh=6, gw=8, mh=6, mw=8, dtype="f32", seed=5,
                       ridge_eps=0.0)
    inp = synth.make_inputs(cfg)
    g = run_gpu(cfg, inp, backward=False)
    Q, K, V = (f64(inp[k])[0] for k in ("Q", "K", "V"))
    s = f64(inp["whiten"])
    for h in range(2):
        G = np.exp(-np.abs(Q[h][:, None, :] - K[h][None, :, :]).sum(-1) / cfg.lam)
        Z = (G - G.mean(1, keepdims=True)) * s[h][None, :] + 1.0 / cfg.n
        assert rel_err(f64(g["O"])[0, h], Z @ V[h]) < 2e-3      # fp32 inverse of a cond ~ 1e2 matrix


def test_runs_twice_bit_identical():
    cfg = synth.shrink(synth.CONFIGS["cfg3"], B=1)
    inp = synth.make_inputs(cfg)
    a, b = run_gpu(cfg, inp), run_gpu(cfg, inp)
    for k in ("O", "dQ", "dK", "dV"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("name,B", [("cfg2", 8), ("cfg3", 2), ("cfg4a", 1), ("cfg5_m128_T8", 1), ("cfg5_m256_T4", 1)])
def test_overlap_on_the_side_stream_changes_no_bit(name, B):
    """With the per-head kernels on the library's second stream (the default) the results are the bits of
    the single-stream order, call after call: the fork and join events order every producer before its consumers."""
    cfg = synth.shrink(synth.CONFIGS[name], B=B)
    inp = synth.make_inputs(cfg)
    before = ln.set_overlap(False)
    try:
        ref = run_gpu(cfg, inp)
        ln.set_overlap(True)
        for _ in range(3):
            got = run_gpu(cfg, inp)
            for k in ("O", "dQ", "dK", "dV"):
                assert torch.equal(ref[k], got[k]), (name, k)
            assert int(got["status"].abs().max()) == 0
    finally:
        ln.set_overlap(before)


def test_singular_landmarks_are_flagged_finite():
    # all keys identical -> K_LL is all ones; the ridge keeps Newton-Schulz finite
    cfg = synth.shrink(synth.CONFIGS["cfg1"], H=1)
    inp = synth.make_inputs(cfg)
    inp["K"][:] = inp["K"][0, 0, 0]
    g = run_gpu(cfg, inp, backward=False)
    assert int(g["status"].abs().max()) == 0
    assert torch.isfinite(g["O"]).all()
    o = run_oracle_heads(cfg, inp, [0], backward=False)
    assert rel_err(f64(g["O"])[0, 0], o["O"][0]) < 1e-4


@pytest.mark.parametrize("name,B,H", [("cfg2", 1, 2), ("cfg4a", 1, 1), ("cfg5_m256_T4", 1, 1), ("cfg1", 1, 1)])
def test_diverged_iteration_sets_status_bit(name, B, H):
    """The step size printed in Alg. 2 (2 / ||W||_2, far above 1 / (||W||_1 ||W||_inf) for a unit-diagonal W) makes
    the iteration blow up; every Newton-Schulz engine (m <= 64, tcgen05, clustered, fp32) must report it in bit 0
    of dev_status instead of trapping, and a sane step size must leave the flags at zero."""
    cfg = synth.shrink(synth.CONFIGS[name], B=B, H=H)
    inp = synth.make_inputs(cfg)
    Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
    for alpha, want in ((1.9, 1), (0.0, 0)):
        p = ln.problem_from_config(cfg, whiten=inp["whiten"].to(DEV))
        p.ns_alpha = alpha
        p.ns_iters = max(cfg.T, 8)
        status = torch.full((cfg.B * cfg.H,), -1, dtype=torch.int32, device=DEV)
        ln.laplace_nystrom_fwd(p, Q, K, V, dev_status=status)
        torch.cuda.synchronize()
        assert all(int(v) & 1 == want for v in status.cpu()), (name, alpha, status)
        assert all(int(v) & 2 == 0 for v in status.cpu())


def test_bounded_wait_times_out_into_status_bit_1():
    """A wait that nothing satisfies runs out after its probe limit, sets bit 1 of the status word and the kernel
    returns; the context stays usable and the next real call reports clean flags."""
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    ln.selftest_wait_timeout(status, probes=2000)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [2, 0, 0, 0]
    cfg = synth.shrink(synth.CONFIGS["cfg2"], B=1)
    g = run_gpu(cfg, synth.make_inputs(cfg))
    assert int(g["status"].abs().max()) == 0 and int(g["status_bwd"].abs().max()) == 0
    assert torch.isfinite(g["dQ"].float()).all()


def test_host_buffer_step_matches_device_path():
    """laplace_nystrom_fwd_bwd_host (copies + forward + backward on one stream) returns the same bits as the device
    entry points called on device copies of the same tensors."""
    cfg = synth.shrink(synth.CONFIGS["cfg2"], B=2)
    inp = synth.make_inputs(cfg)
    g = run_gpu(cfg, inp)
    wh = inp["whiten"].to(DEV)
    p = ln.problem_from_config(cfg, whiten=wh)
    bufs = ln.HostStep(p, DEV)
    hin = {k: inp[k].pin_memory() for k in ("Q", "K", "V", "dO")}
    hout = {k: torch.empty_like(inp["Q"]).pin_memory() for k in ("O", "dQ", "dK", "dV")}
    status = torch.full((cfg.B * cfg.H,), -1, dtype=torch.int32, device=DEV)
    for _ in range(2):
        ln.laplace_nystrom_fwd_bwd_host(p, bufs, hin["Q"], hin["K"], hin["V"], hin["dO"], hout["O"], hout["dQ"],
                                        hout["dK"], hout["dV"], dev_status=status)
        torch.cuda.synchronize()
        assert int(status.abs().max()) == 0
        for k in ("O", "dQ", "dK", "dV"):
            assert torch.equal(hout[k], g[k].cpu()), k


@pytest.mark.parametrize("overlap", [True, False])
def test_host_buffer_steps_back_to_back_on_one_stream(overlap):
    """Two host-buffer steps with DIFFERENT inputs enqueued on one stream, one behind the other, without a host
    synchronisation in between and sharing their device buffers: the second step's copies in must not overtake the first
    step's kernels and copies out (the copies ride on the library's copy streams, ordered by events), and each step must
    return the bits of the device path on its own inputs.  With ln_set_overlap(0) everything is on the caller's stream."""
    from dataclasses import replace
    cfg = synth.shrink(synth.CONFIGS["cfg3"], B=2)
    inps = [synth.make_inputs(cfg), synth.make_inputs(replace(cfg, seed=cfg.seed + 1))]
    refs = [run_gpu(cfg, inp) for inp in inps]
    p = ln.problem_from_config(cfg, whiten=inps[0]["whiten"].to(DEV))        # the whitening scale of the two seeds
    # the second reference with the first problem's whitening scale (one problem struct serves both steps)
    inp1 = dict(inps[1]); inp1["whiten"] = inps[0]["whiten"]
    refs[1] = run_gpu(cfg, inp1)
    bufs = ln.HostStep(p, DEV)
    hin = [{k: inp[k].pin_memory() for k in ("Q", "K", "V", "dO")} for inp in inps]
    hout = [{k: torch.empty_like(inps[0]["Q"]).pin_memory() for k in ("O", "dQ", "dK", "dV")} for _ in range(2)]
    st = torch.cuda.Stream(device=DEV)
    was = ln.set_overlap(overlap)
    try:
        for rep in range(3):
            for i in (0, 1):
                ln.laplace_nystrom_fwd_bwd_host(p, bufs, hin[i]["Q"], hin[i]["K"], hin[i]["V"], hin[i]["dO"], hout[i]["O"],
                                                hout[i]["dQ"], hout[i]["dK"], hout[i]["dV"], stream=st)
            st.synchronize()
            for i in (0, 1):
                for k in ("O", "dQ", "dK", "dV"):
                    assert torch.equal(hout[i][k], refs[i][k].cpu()), (rep, i, k)
                    hout[i][k].zero_()
    finally:
        ln.set_overlap(was)


@pytest.mark.parametrize("name,B", [("cfg1", 1), ("cfg2", 5), ("cfg3", 2), ("cfg4a", 1), ("cfg5_m256_T4", 1)])
def test_whiten_stats_match_the_oracle(name, B):
    """Eq. 5-6 on the device (from the kernel block the forward pass saved) against the float64 oracle applied to the
    oracle's own kernel block; fp32-path bar (the statistic is accumulated in double on both sides)."""
    cfg = synth.shrink(synth.CONFIGS[name], B=B)
    inp = synth.make_inputs(cfg)
    Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
    p = ln.problem_from_config(cfg, whiten=None)
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=DEV)
    ln.laplace_nystrom_fwd(p, Q, K, V, saved=saved)
    eps_w = 1e-5
    got = ln.laplace_nystrom_whiten_stats(p, saved, eps_w)
    again = ln.laplace_nystrom_whiten_stats(p, saved, eps_w)
    torch.cuda.synchronize()
    assert torch.equal(got, again)                                   # fixed summation order
    BH = cfg.B * cfg.H
    op = oracle_problem(cfg)
    _, extra = oracle.forward(op, f64(inp["Q"]), f64(inp["K"]), f64(inp["V"]), want=("C",))
    ref = oracle.whiten_stats(extra["C"].reshape(BH, cfg.n, cfg.m), cfg.H, eps_w)
    assert rel_err(f64(got), ref) < TOL["f32"], (name, rel_err(f64(got), ref))
    # the estimated scale is accepted as the `whiten` input of the path
    p2 = ln.problem_from_config(cfg, whiten=got)
    O = ln.laplace_nystrom_fwd(p2, Q, K, V, saved=saved)
    o = run_oracle_heads(cfg, {**inp, "whiten": torch.from_numpy(ref).float()}, [0], backward=False)
    assert rel_err(f64(O).reshape(BH, cfg.n, cfg.d)[[0]], o["O"]) < TOL[cfg.dtype]


def _random_cases(count, seed):
    """Seeded draw of small problems over everything the entry points branch on: grid and landmark-grid shape (bins that
    divide the grid or overlap), class tokens, head dim, iteration count, storage type, landmark mode, map mode,
    duplicated bins."""
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < count:
        gh, gw = int(rng.integers(3, 21)), int(rng.integers(3, 21))
        mh, mw = int(rng.integers(1, min(gh, 16) + 1)), int(rng.integers(1, min(gw, 16) + 1))
        if mh * mw > 256 or mh * mw < 2:
            continue
        even = gh % mh == 0 and gw % mw == 0          # bins of one size: only then can a bin's keys be copies of another's
        cases.append(dict(gh=gh, gw=gw, mh=mh, mw=mw, prefix=int(rng.integers(0, 3)), d=int(rng.choice([32, 64, 128])),
                          T=int(rng.integers(0, 9)), dtype=str(rng.choice(["bf16", "f32"])), lm_mode=int(rng.choice([1, 2, 3])),
                          map_mode=int(rng.choice([0, 1])), dup=float(rng.choice([0.0, 0.2])) * even, B=int(rng.integers(1, 3)),
                          H=int(rng.integers(1, 4)), seed=int(rng.integers(1, 1 << 20))))
    return cases


def _random_cases_many_landmarks(count, seed):
    """The same draw restricted to 100 ... 256 landmarks and bf16 storage: the per-head engines above 64 and above 128
    landmarks at their ragged sizes (odd m, m not a multiple of 4, blocks of the 2 x 2 cut that are almost empty)."""
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < count:
        gh, gw = int(rng.integers(10, 25)), int(rng.integers(10, 25))
        mh, mw = int(rng.integers(4, min(gh, 16) + 1)), int(rng.integers(4, min(gw, 16) + 1))
        if not 100 <= mh * mw <= 256:
            continue
        even = gh % mh == 0 and gw % mw == 0
        cases.append(dict(gh=gh, gw=gw, mh=mh, mw=mw, prefix=int(rng.integers(0, 3)), d=int(rng.choice([32, 64, 128])),
                          T=int(rng.integers(0, 9)), dtype="bf16", lm_mode=int(rng.choice([1, 1, 2, 3])),
                          map_mode=int(rng.choice([0, 1])), dup=float(rng.choice([0.0, 0.2])) * even, B=int(rng.integers(1, 3)),
                          H=int(rng.integers(1, 4)), seed=int(rng.integers(1, 1 << 20))))
    return cases


def _cases_two_block_rows():
    """129 ... 256 landmarks at every head width: the 2 x 2 block cut of the per-head kernels with a second block row of
    one, a few, and all 128 landmarks; odd counts and counts that are no multiple of 4 (the backward products
    dX = dY M^T and dM = X_T^T dY read M, dY and X_T in 128-bit pieces where the row length allows)."""
    cases = []
    for (mh, mw, gh, gw), d, T, lm_mode, map_mode in (((3, 43, 6, 43), 64, 3, 1, 1), ((10, 13, 20, 13), 64, 5, 2, 0),
                                                       ((11, 13, 11, 26), 128, 4, 1, 1), ((11, 17, 22, 17), 64, 6, 1, 0),
                                                       ((15, 17, 15, 17), 128, 3, 2, 1), ((16, 16, 16, 32), 64, 8, 1, 1),
                                                       ((13, 17, 13, 34), 32, 7, 3, 0), ((7, 19, 14, 19), 128, 0, 1, 1)):
        cases.append(dict(gh=gh, gw=gw, mh=mh, mw=mw, prefix=len(cases) % 3, d=d, T=T, dtype="bf16", lm_mode=lm_mode,
                          map_mode=map_mode, dup=0.0, B=1 + len(cases) % 2, H=1 + len(cases) % 3, seed=4100 + len(cases)))
    return cases


@pytest.mark.parametrize("case", _random_cases(32, 20260) + _random_cases_many_landmarks(16, 31) + _cases_two_block_rows(),
                         ids=lambda c: "g{gh}x{gw}_m{mh}x{mw}_p{prefix}_d{d}_T{T}_{dtype}_lm{lm_mode}_map{map_mode}".format(**c))
def test_random_shapes_and_modes(case):
    from parity import metrics
    cfg = synth.Config("random", B=case["B"], H=case["H"], d=case["d"], m=case["mh"] * case["mw"], T=case["T"], gh=case["gh"],
                       gw=case["gw"], mh=case["mh"], mw=case["mw"], prefix=case["prefix"], dtype=case["dtype"],
                       dup_frac=case["dup"], seed=case["seed"])
    inp = synth.make_inputs(cfg)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    p = ln.problem_from_config(cfg, whiten=inp["whiten"].to(DEV), map_mode=case["map_mode"])
    p.lm_mode = case["lm_mode"]
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=DEV)
    status = torch.full((cfg.B * cfg.H,), -1, dtype=torch.int32, device=DEV)
    O = ln.laplace_nystrom_fwd(p, Q, K, V, saved=saved, dev_status=status)
    dQ, dK, dV, _ = ln.laplace_nystrom_bwd(p, Q, K, V, dO, saved)
    assert int(status.abs().max()) == 0
    op = oracle_problem(cfg, map_mode=case["map_mode"], lm_mode=case["lm_mode"])
    wh = f64(inp["whiten"])
    q, k, v, g = (f64(inp[x]) for x in ("Q", "K", "V", "dO"))
    Oo = oracle.forward(op, q, k, v, whiten=wh)
    dQo, dKo, dVo, _ = oracle.backward(op, q, k, v, g, whiten=wh)
    BH = cfg.B * cfg.H
    errs = {kk: metrics(f64(a).reshape(BH, cfg.n, cfg.d), r.reshape(BH, cfg.n, cfg.d), cfg.dtype == "bf16")
            for kk, a, r in (("O", O, Oo), ("dQ", dQ, dQo), ("dK", dK, dKo), ("dV", dV, dVo))}
    print(case, {kk: {a: f"{b:.1e}" for a, b in e.items()} for kk, e in errs.items()})
    assert_parity(cfg, errs)
