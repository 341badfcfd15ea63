"""Seeded synthetic inputs with the shapes of the paper's workloads.

The paper measures on ImageNet-1K images passed through DeiT / PVT style backbones; neither the
data nor trained weights are available, so these tensors take those models' token grids (14x14,
56x56, 112x112, 224x224), head dims and pooled landmark grids and stand in for them.  This module
holds no arithmetic of the method: it only draws numbers, rounds them to the storage type and
copies keys around to create duplicated landmark bins.  It serves the oracle and the CUDA path
alike (both receive exactly the same rounded values) and imports neither.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Config:
    name: str
    B: int
    H: int
    d: int
    m: int
    T: int
    gh: int
    gw: int
    mh: int
    mw: int
    prefix: int = 0
    dtype: str = "bf16"         # storage type of Q, K, V, dO
    sigma: float = 1.0          # Q, K, V, dO ~ N(0, sigma^2)
    v_uniform: bool = False     # V ~ U(-1, 1) instead
    dup_frac: float = 0.0       # fraction of landmark bins whose keys are copies of another bin's
    seed: int = 0
    backward: bool = True
    ridge_eps: float = 1e-6

    @property
    def n(self) -> int:
        return self.prefix + self.gh * self.gw

    @property
    def lam(self) -> float:
        return float(self.d)


def _cfg5(m, mh, mw, T, i_m, i_T):
    return Config(f"cfg5_m{m}_T{T}", B=16, H=8, d=128, m=m, T=T, gh=64, gw=64, mh=mh, mw=mw,
                  v_uniform=True, dup_frac=0.1, seed=500 + 10 * i_m + i_T)


CONFIGS: Dict[str, Config] = {c.name: c for c in [
    # tiny correctness case: fp32, forward only
    Config("cfg1", B=1, H=3, d=64, m=32, T=6, gh=14, gw=14, mh=4, mw=8, dtype="f32", seed=0, backward=False),
    # DeiT-Small shaped: class token + 14x14 patches, 7x7 landmarks
    Config("cfg2", B=64, H=6, d=64, m=49, T=6, gh=14, gw=14, mh=7, mw=7, prefix=1, seed=2),
    # PVT stage-1 shaped: 56x56 tokens, 8x8 landmarks
    Config("cfg3", B=32, H=1, d=64, m=64, T=8, gh=56, gw=56, mh=8, mw=8, seed=3),
    # high-resolution sweep
    Config("cfg4a", B=8, H=2, d=64, m=128, T=8, gh=56, gw=56, mh=8, mw=16, sigma=0.5, seed=40),
    Config("cfg4b", B=8, H=2, d=64, m=128, T=8, gh=112, gw=112, mh=8, mw=16, sigma=0.5, seed=41),
    Config("cfg4c", B=8, H=2, d=64, m=128, T=8, gh=224, gw=224, mh=8, mw=16, sigma=0.5, seed=42),
] + [
    # landmark / solver stress with duplicated keys (near-singular landmark kernel)
    _cfg5(m, mh, mw, T, i_m, i_T)
    for i_m, (m, mh, mw) in enumerate([(64, 8, 8), (128, 8, 16), (256, 16, 16)])
    for i_T, T in enumerate([4, 8, 12])
]}


def shrink(cfg: Config, B: Optional[int] = None, H: Optional[int] = None) -> Config:
    """Same shapes per head, fewer heads (for parity runs the oracle can finish)."""
    return replace(cfg, B=B if B is not None else cfg.B, H=H if H is not None else cfg.H)


def _round(x: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x))
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _bin_tokens(cfg: Config, l: int) -> np.ndarray:
    a, b = divmod(l, cfg.mw)
    r0, r1 = (a * cfg.gh) // cfg.mh, -((-(a + 1) * cfg.gh) // cfg.mh)
    c0, c1 = (b * cfg.gw) // cfg.mw, -((-(b + 1) * cfg.gw) // cfg.mw)
    rr, cc = np.meshgrid(np.arange(r0, r1), np.arange(c0, c1), indexing="ij")
    return (cfg.prefix + rr * cfg.gw + cc).reshape(-1)


def make_inputs(cfg: Config) -> Dict[str, torch.Tensor]:
    """CPU tensors in the storage dtype: Q, K, V, dO [B,H,n,d]; whiten fp32 [H,m].

    Drawn with numpy.random.default_rng(seed).standard_normal(float32) in the order Q, K, V, dO,
    then (per head, in order) the duplicated-bin permutations, then the whitening scale.
    """
    rng = np.random.default_rng(cfg.seed)
    shape = (cfg.B, cfg.H, cfg.n, cfg.d)
    Q = rng.standard_normal(shape, dtype=np.float32) * np.float32(cfg.sigma)
    K = rng.standard_normal(shape, dtype=np.float32) * np.float32(cfg.sigma)
    if cfg.v_uniform:
        V = rng.random(shape, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
    else:
        V = rng.standard_normal(shape, dtype=np.float32) * np.float32(cfg.sigma)
    dO = rng.standard_normal(shape, dtype=np.float32) * np.float32(cfg.sigma)
    if cfg.dup_frac > 0:
        ndup = int(math.ceil(cfg.dup_frac * cfg.m))
        bins = [_bin_tokens(cfg, l) for l in range(cfg.m)]
        for b in range(cfg.B):
            for h in range(cfg.H):
                perm = rng.permutation(cfg.m)
                for dst, src in zip(perm[:ndup], perm[ndup:2 * ndup]):
                    K[b, h, bins[dst]] = K[b, h, bins[src]]
    # whitening scale of Eq. 6, s = 1/sqrt(var + eps): a constant input of the path ("estimated
    # offline").  Kernel values against pooled landmarks spread by a few hundredths, so the
    # variances are drawn around that.
    var = rng.uniform(1.0e-3, 4.0e-3, size=(cfg.H, cfg.m)).astype(np.float32)
    whiten = (1.0 / np.sqrt(var + np.float32(1e-5))).astype(np.float32)
    return {"Q": _round(Q, cfg.dtype), "K": _round(K, cfg.dtype), "V": _round(V, cfg.dtype),
            "dO": _round(dO, cfg.dtype), "whiten": torch.from_numpy(whiten)}
