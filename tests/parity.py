"""Helpers shared by the GPU parity tests: run the oracle and the CUDA path on the same seeded
inputs and compare with the norm-wise relative error the tolerances are stated in."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2604_20368_b200 as ln
from paper_2604_20368_b200 import synth

# relative Frobenius error, outputs and gradients alike: fp32 storage / bf16 storage
TOL = {"f32": 1e-4, "bf16": 2e-2}


def rel_err(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    return float(np.linalg.norm((got - ref).ravel()) / (den if den > 0 else 1.0))


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_problem(cfg: synth.Config, H=None, map_mode=1, lm_mode=1) -> oracle.Problem:
    return oracle.Problem(B=cfg.B if H is None else 1, H=cfg.H if H is None else H, n=cfg.n, d=cfg.d, m=cfg.m,
                          lam=cfg.lam, ns_iters=cfg.T, ridge_eps=cfg.ridge_eps, map_mode=map_mode, lm_mode=lm_mode,
                          prefix=cfg.prefix, gh=cfg.gh, gw=cfg.gw, mh=cfg.mh, mw=cfg.mw, lm_f32=1)


def run_gpu(cfg: synth.Config, inp, use_whiten=True, map_mode=1, backward=True):
    dev = torch.device("cuda:0")
    Q, K, V, dO = (inp[k].to(dev) for k in ("Q", "K", "V", "dO"))
    wh = inp["whiten"].to(dev) if use_whiten else None
    p = ln.problem_from_config(cfg, whiten=wh, map_mode=map_mode)
    saved = torch.empty(ln.laplace_nystrom_saved_bytes(p), dtype=torch.uint8, device=dev) if backward else None
    status = torch.full((cfg.B * cfg.H,), -1, dtype=torch.int32, device=dev)
    O = ln.laplace_nystrom_fwd(p, Q, K, V, saved=saved, dev_status=status)
    out = {"O": O, "status": status}
    if backward:
        dQ, dK, dV, _ = ln.laplace_nystrom_bwd(p, Q, K, V, dO, saved)
        out.update(dQ=dQ, dK=dK, dV=dV)
    torch.cuda.synchronize()
    return out


def run_oracle_heads(cfg: synth.Config, inp, heads, use_whiten=True, map_mode=1, backward=True):
    """Oracle on the listed flat head indices (b*H + h) of the full problem."""
    BH = cfg.B * cfg.H
    sel = lambda t: f64(t).reshape(BH, cfg.n, cfg.d)[heads][None]
    Q, K, V, dO = (sel(inp[k]) for k in ("Q", "K", "V", "dO"))
    wh = f64(inp["whiten"])[[h % cfg.H for h in heads]] if use_whiten else None
    op = oracle_problem(cfg, H=len(heads), map_mode=map_mode)
    out = {"O": oracle.forward(op, Q, K, V, whiten=wh)[0]}
    if backward:
        dQ, dK, dV, _ = oracle.backward(op, Q, K, V, dO, whiten=wh)
        out.update(dQ=dQ[0], dK=dK[0], dV=dV[0])
    return out


def compare(cfg: synth.Config, gpu_out, ora_out, heads):
    BH = cfg.B * cfg.H
    errs = {}
    for k, ref in ora_out.items():
        got = f64(gpu_out[k]).reshape(BH, cfg.n, cfg.d)[heads]
        errs[k] = rel_err(got, ref)
    return errs
