"""Helpers shared by the GPU parity tests: run the oracle and the CUDA path on the same seeded
inputs and compare them.

Four figures per tensor (outputs and gradients alike):
  fro      ||gpu - ref||_F / ||ref||_F over the whole tensor: the figure the tolerances are stated in
           (1e-4 fp32 storage, 2e-2 bf16 storage);
  row      max over token rows i of ||gpu_i - ref_i||_2 / max(||ref_i||_2, rms row norm): one wrong row cannot
           hide in a large tensor;
  maxabs   max |gpu - ref| / max |ref|;
  internal (bf16 storage only) the error left once the rounding of the bf16 output itself is taken out:
           || max(0, |gpu - ref| - ulp(gpu)/2) ||_F / ||ref||_F.  The device rounds an fp32 value v to gpu, so
           |v - ref| >= |gpu - ref| - ulp(gpu)/2: this is a lower bound on the error of the fp32 value the kernels
           computed, which the 2^-9 output rounding would otherwise bury.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2604_20368_b200 as ln
from paper_2604_20368_b200 import synth

# relative Frobenius error, outputs and gradients alike: fp32 storage / bf16 storage
TOL = {"f32": 1e-4, "bf16": 2e-2}
# per-row and max-abs figures: same bars (a row is held to what the whole tensor is held to)
TOL_ROW = {"f32": 2e-4, "bf16": 2e-2}
TOL_MAXABS = {"f32": 1e-4, "bf16": 2e-2}
# error of the fp32 values behind bf16 outputs (split-bf16 tensor-core operands carry about 16 mantissa bits)
TOL_INTERNAL = 1e-3
# fp32 intermediates the forward pass leaves in its context, against the oracle's
TOL_INTERMEDIATE = {"f32": 1e-4, "bf16": 5e-4}


def rel_err(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    return float(np.linalg.norm((got - ref).ravel()) / (den if den > 0 else 1.0))


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bf16 numbers at |x| (8 significant bits), for normal values."""
    ax = np.abs(np.asarray(x, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(ax, 2.0 ** -126)))
    return np.exp2(e - 7)


def metrics(got, ref, bf16: bool) -> dict:
    """got, ref: [heads, rows, cols] float64."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    diff = got - ref
    den = np.linalg.norm(ref.ravel()) or 1.0
    rown = np.linalg.norm(ref, axis=-1)
    rms = float(np.sqrt((rown ** 2).mean())) or 1.0
    out = {"fro": float(np.linalg.norm(diff.ravel()) / den),
           "row": float((np.linalg.norm(diff, axis=-1) / np.maximum(rown, rms)).max()),
           "maxabs": float(np.abs(diff).max() / (np.abs(ref).max() or 1.0))}
    if bf16:
        out["internal"] = float(np.linalg.norm(np.maximum(0.0, np.abs(diff) - 0.5 * bf16_ulp(got)).ravel()) / den)
    return out


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
    out = {"O": O, "status": status, "saved": saved, "problem": p}
    if backward:
        status_b = torch.full((cfg.B * cfg.H,), -1, dtype=torch.int32, device=dev)
        dQ, dK, dV, _ = ln.laplace_nystrom_bwd(p, Q, K, V, dO, saved, dev_status=status_b)
        out.update(dQ=dQ, dK=dK, dV=dV, status_bwd=status_b)
    torch.cuda.synchronize()
    return out


def run_oracle_heads(cfg: synth.Config, inp, heads, use_whiten=True, map_mode=1, backward=True, want=()):
    """Oracle on the listed flat head indices (b*H + h) of the full problem."""
    BH = cfg.B * cfg.H
    sel = lambda t: f64(t).reshape(BH, cfg.n, cfg.d)[heads][None]
    Q, K, V, dO = (sel(inp[k]) for k in ("Q", "K", "V", "dO"))
    wh = f64(inp["whiten"])[[h % cfg.H for h in heads]] if use_whiten else None
    op = oracle_problem(cfg, H=len(heads), map_mode=map_mode)
    if want:
        O, extra = oracle.forward(op, Q, K, V, whiten=wh, want=want)
        out = {"O": O[0], "extra": extra}
    else:
        out = {"O": oracle.forward(op, Q, K, V, whiten=wh)[0]}
    if backward:
        dQ, dK, dV, _ = oracle.backward(op, Q, K, V, dO, whiten=wh)
        out.update(dQ=dQ[0], dK=dK[0], dV=dV[0])
    return out


def compare(cfg: synth.Config, gpu_out, ora_out, heads):
    """Per tensor the four figures above, on the sampled heads."""
    BH = cfg.B * cfg.H
    errs = {}
    for k in ("O", "dQ", "dK", "dV"):
        if k not in ora_out:
            continue
        got = f64(gpu_out[k]).reshape(BH, cfg.n, cfg.d)[heads]
        errs[k] = metrics(got, ora_out[k], cfg.dtype == "bf16")
    return errs


def assert_parity(cfg: synth.Config, errs, tol=None):
    dt = cfg.dtype
    for k, e in errs.items():
        assert e["fro"] < (TOL[dt] if tol is None else tol), (cfg.name, k, e)
        assert e["row"] < (TOL_ROW[dt] if tol is None else 2 * tol), (cfg.name, k, e)
        assert e["maxabs"] < (TOL_MAXABS[dt] if tol is None else tol), (cfg.name, k, e)
        if "internal" in e:
            assert e["internal"] < TOL_INTERNAL, (cfg.name, k, e)


def compare_intermediates(cfg: synth.Config, gpu_out, inp, heads, use_whiten=True, map_mode=1):
    """The fp32 intermediates the forward pass left in its context against the oracle's: landmarks, the three kernel
    blocks, the Newton-Schulz iterate X_T, M = R V, the folded Y and the row means."""
    p, saved = gpu_out["problem"], gpu_out["saved"]
    o = run_oracle_heads(cfg, inp, heads, use_whiten=use_whiten, map_mode=map_mode, backward=False,
                         want=("L", "C", "R", "W", "X", "M", "Y"))["extra"]
    got = {k: f64(ln.saved_array(p, saved, k)[heads]) for k in ("L", "C", "Rt", "W", "X", "M", "Yt", "mu", "ybar")}
    s = f64(inp["whiten"])[[h % cfg.H for h in heads]] if use_whiten else np.ones((len(heads), cfg.m))
    Y = o["Y"]
    if map_mode == 1:       # Prop. 3 folded into the small factor: Ytilde_l = s_l Y_l - mean_l'(s_l' Y_l'), ybar = mean_l Y_l
        sY = s[:, :, None] * Y
        Yt, ybar = sY - sY.mean(axis=1, keepdims=True), Y.mean(axis=1, keepdims=True)
    else:
        Yt, ybar = Y, np.zeros_like(Y[:, :1])
    ref = {"L": o["L"], "C": o["C"], "Rt": np.swapaxes(o["R"], 1, 2), "W": o["W"], "X": o["X"], "M": o["M"], "Yt": Yt,
           "ybar": ybar}
    if map_mode == 1:
        ref["mu"] = o["C"].mean(axis=2)[:, None, :]
    return {k: rel_err(got[k], v) for k, v in ref.items()}
