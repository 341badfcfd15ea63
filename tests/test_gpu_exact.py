"""The exact (m = n) Laplacian attention kernel against the oracle's plain definition (Eq. 4 + Eq. 7), and the
Nystrom path against it as the number of landmarks grows."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_20368_b200 as ln
from paper_2604_20368_b200 import synth
from parity import f64, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("n,d", [(197, 64), (64, 32), (130, 128), (1, 32), (321, 64)])
@pytest.mark.parametrize("dtype,tol", [(torch.float32, 2e-5), (torch.bfloat16, 4e-3)])
@pytest.mark.parametrize("map_mode", [0, 1])
def test_exact_kernel_matches_definition(n, d, dtype, tol, map_mode):
    rng = np.random.default_rng(n + d)
    Q, K, V = (torch.from_numpy(rng.standard_normal((2, 2, n, d), dtype=np.float32)).to(dtype) for _ in range(3))
    O = ln.laplace_exact_fwd(Q.to(DEV), K.to(DEV), V.to(DEV), float(d), map_mode)
    ref = oracle.exact_attention(f64(Q), f64(K), f64(V), float(d), map_mode)
    assert rel_err(f64(O), ref) < tol


def test_nystrom_reaches_exact_attention_at_m_equals_n_and_improves_with_m():
    # fp32 storage, unit whitening: bins == grid and many Newton-Schulz steps reproduce the exact kernel's output
    errs = {}
    for mh, mw in ((2, 2), (4, 4), (8, 8)):
        cfg = synth.Config("acc", B=1, H=2, d=32, m=mh * mw, T=30, gh=8, gw=8, mh=mh, mw=mw, dtype="f32", seed=3, ridge_eps=1e-7)
        inp = synth.make_inputs(cfg)
        Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
        p = ln.problem_from_config(cfg, whiten=None)
        O = ln.laplace_nystrom_fwd(p, Q, K, V)
        E = ln.laplace_exact_fwd(Q, K, V, cfg.lam, 1)
        errs[mh * mw] = rel_err(f64(O), f64(E))
    print("Nystrom against exact attention by m:", errs)
    assert errs[64] < 5e-3                      # m = n: the approximation is exact up to the fp32 inverse
    assert errs[64] < errs[16] and errs[64] < errs[4]
