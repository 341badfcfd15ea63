"""Float64 CPU oracle (test infrastructure, not the product).

ctypes front end of ``laplace_oracle.c``.  Arrays go in and come out as
C-contiguous float64 numpy arrays.  Nothing here imports or is imported by the
CUDA package; only tests, the smoke check and the benchmark's CPU-baseline leg
may use it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "laplace_oracle.c")
_LIB = os.path.join(_HERE, "liblaplace_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over heads) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Problem(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("n", ctypes.c_int32),
        ("d", ctypes.c_int32), ("m", ctypes.c_int32),
        ("lambda_", ctypes.c_double),
        ("ns_iters", ctypes.c_int32),
        ("ridge_eps", ctypes.c_double),
        ("ns_alpha", ctypes.c_double),
        ("map_mode", ctypes.c_int32),
        ("lm_mode", ctypes.c_int32),
        ("prefix", ctypes.c_int32), ("gh", ctypes.c_int32), ("gw", ctypes.c_int32),
        ("mh", ctypes.c_int32), ("mw", ctypes.c_int32),
        ("lm_f32", ctypes.c_int32),
        ("lm_filter", ctypes.c_void_p),
        ("solver", ctypes.c_int32),
    ]


@dataclass
class Problem:
    """Arguments of the path in the paper's notation (B, heads, n tokens, head dim d, m landmarks)."""
    B: int
    H: int
    n: int
    d: int
    m: int
    lam: float
    ns_iters: int
    ridge_eps: float = 1e-6
    ns_alpha: float = 0.0
    map_mode: int = 1
    lm_mode: int = 1
    prefix: int = 0
    gh: int = 0
    gw: int = 0
    mh: int = 0
    mw: int = 0
    lm_f32: int = 0   # 1: pooled landmarks rounded to single precision (what the device stores)
    # depth-wise-convolution landmark selection (Sec. 4.2): float64 [H, taps, d], taps = (gh/mh)*(gw/mw), or None
    lm_filter: Optional[np.ndarray] = field(default=None, repr=False)
    solver: int = 0   # 0: Newton-Schulz (Alg. 2); 1: conjugate gradients, ns_iters steps (Sec. 5.3, Table 4)

    def c(self) -> _Problem:
        f = None
        if self.lm_filter is not None:
            assert self.lm_mode in (1, 2) and self.gh % self.mh == 0 and self.gw % self.mw == 0
            f = self.lm_filter
            assert f.dtype == np.float64 and f.flags["C_CONTIGUOUS"]
            assert f.shape == (self.H, (self.gh // self.mh) * (self.gw // self.mw), self.d)
            f = f.ctypes.data
        assert self.solver in (0, 1) and not (self.solver == 1 and self.lm_mode == 3), "conjugate gradients need the symmetric W of one landmark set"
        return _Problem(self.B, self.H, self.n, self.d, self.m, float(self.lam), self.ns_iters,
                        float(self.ridge_eps), float(self.ns_alpha), self.map_mode, self.lm_mode,
                        self.prefix, self.gh, self.gw, self.mh, self.mw, self.lm_f32, f, self.solver)


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    if a is None:
        return None
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def l1_kernel(A, Bm, lam, want_rowsum=False):
    """K[b,i,j] = exp(-||A[b,i]-Bm[b,j]||_1 / lam).  A [batch,na,d], Bm [batch,nb,d]."""
    A, Bm = _f64(A), _f64(Bm)
    batch, na, d = A.shape
    nb = Bm.shape[1]
    K = np.empty((batch, na, nb))
    rs = np.empty((batch, na)) if want_rowsum else None
    _load().oracle_l1_kernel(batch, na, nb, d, _p(A), _p(Bm), ctypes.c_double(lam), _p(K), _p(rs))
    return (K, rs) if want_rowsum else K


def l1_kernel_bwd(A, Bm, lam, dK):
    A, Bm, dK = _f64(A), _f64(Bm), _f64(dK)
    batch, na, d = A.shape
    nb = Bm.shape[1]
    dA, dB = np.empty_like(A), np.empty_like(Bm)
    _load().oracle_l1_kernel_bwd(batch, na, nb, d, _p(A), _p(Bm), ctypes.c_double(lam), _p(dK), _p(dA), _p(dB))
    return dA, dB


def cg_solve(W, Bm, iters, eps=0.0):
    """T-step conjugate-gradient iterates of (W + eps I) X = B (Sec. 5.3).  W [batch,m,m], B [batch,m,d]."""
    W, Bm = _f64(W), _f64(Bm)
    batch, m, d = Bm.shape
    X = np.empty_like(Bm)
    _load().oracle_cg_solve(batch, m, d, _p(W), ctypes.c_double(eps), iters, _p(Bm), _p(X))
    return X


def ns_pinv(W, iters, eps=0.0, alpha=0.0, want_hist=False):
    """Newton-Schulz T-step iterate of (W + eps I)^-1.  W [batch,m,m].  Returns X, resid, alpha(, X_hist)."""
    W = _f64(W)
    batch, m, _ = W.shape
    X = np.empty_like(W)
    hist = np.empty((batch, max(iters, 1), m, m)) if want_hist else None
    resid = np.empty(batch)
    aout = np.empty(batch)
    _load().oracle_ns_pinv(batch, m, _p(W), iters, ctypes.c_double(eps), ctypes.c_double(alpha),
                           _p(X), _p(hist), _p(resid), _p(aout))
    if want_hist:
        return X, resid, aout, hist[:, :iters]
    return X, resid, aout


def ns_pinv_bwd(W, iters, eps, alpha, dX):
    W, dX = _f64(W), _f64(dX)
    batch, m, _ = W.shape
    dW = np.empty_like(W)
    _load().oracle_ns_pinv_bwd(batch, m, _p(W), iters, ctypes.c_double(eps), ctypes.c_double(alpha), _p(dX), _p(dW))
    return dW


def landmarks_pool(p: Problem, K):
    K = _f64(K)
    L = np.empty((p.B, p.H, p.m, p.d))
    cp = p.c()
    _load().oracle_landmarks_pool(ctypes.byref(cp), _p(K), _p(L))
    return L


def landmarks_pool_bwd(p: Problem, dL):
    dL = _f64(dL)
    dK = np.empty((p.B, p.H, p.n, p.d))
    cp = p.c()
    _load().oracle_landmarks_pool_bwd(ctypes.byref(cp), _p(dL), _p(dK))
    return dK


def forward(p: Problem, Q, K, V, L=None, whiten=None, want=()):
    """O [B,H,n,d]; ``want`` names intermediates to return as well (L C R W X M Y Z)."""
    Q, K, V, L, whiten = _f64(Q), _f64(K), _f64(V), _f64(L), _f64(whiten)
    BH = p.B * p.H
    shapes = {"L": (BH, p.m, p.d), "C": (BH, p.n, p.m), "R": (BH, p.m, p.n), "W": (BH, p.m, p.m),
              "X": (BH, p.m, p.m), "M": (BH, p.m, p.d), "Y": (BH, p.m, p.d), "Z": (BH, p.n, p.m)}
    extra = {k: (np.empty(shapes[k]) if k in want else None) for k in shapes}
    O = np.empty((p.B, p.H, p.n, p.d))
    cp = p.c()
    _load().oracle_fwd(ctypes.byref(cp), _p(Q), _p(K), _p(V), _p(L), _p(whiten), _p(O),
                       *[_p(extra[k]) for k in ("L", "C", "R", "W", "X", "M", "Y", "Z")])
    if want:
        return O, {k: extra[k] for k in want}
    return O


def backward(p: Problem, Q, K, V, dO, L=None, whiten=None):
    """Returns dQ, dK, dV, dL (dL is None when the landmarks are pooled from K).  With a landmark-selection filter
    (p.lm_filter) the fourth result is the filter's gradient [H, taps, d] instead (summed over the batch)."""
    Q, K, V, L, whiten, dO = _f64(Q), _f64(K), _f64(V), _f64(L), _f64(whiten), _f64(dO)
    dQ, dK, dV = np.empty_like(Q), np.empty_like(Q), np.empty_like(Q)
    dL = np.empty((p.B, p.H, p.m, p.d)) if p.lm_mode == 0 else None      # pooled landmarks (modes 1, 2): folded into dK / dQ
    dF = np.empty((p.B, p.H) + p.lm_filter.shape[1:]) if p.lm_filter is not None else None
    cp = p.c()
    _load().oracle_bwd(ctypes.byref(cp), _p(Q), _p(K), _p(V), _p(L), _p(whiten), _p(dO),
                       _p(dQ), _p(dK), _p(dV), _p(dL), _p(dF))
    if dF is not None:
        return dQ, dK, dV, dF.sum(axis=0)
    return dQ, dK, dV, dL


def whiten_stats(C, H, eps_w):
    """Diagonal whitening scale of Eq. 5-6 from the query-landmark kernel block.

    C: [B*H, n, m] (heads of one batch element contiguous, flat index b*H + h).  For head h and landmark l the
    "batch of vectors" of Eq. 5 is every query row of every batch element: mu_l = mean over (b, i) of C_il,
    sigma_l^2 = mean over (b, i) of (C_il - mu_l)^2 (the 1/B form of Eq. 5, no Bessel correction), and
    s_l = 1 / sqrt(sigma_l^2 + eps_w) (the diagonal of D^{-1/2}, Eq. 6).  Returns s [H, m].  Two passes, float64."""
    C = np.asarray(C, dtype=np.float64)
    BH, n, m = C.shape
    B = BH // H
    s = np.empty((H, m))
    for h in range(H):
        rows = np.concatenate([C[b * H + h] for b in range(B)], axis=0)      # [B*n, m]
        cnt = rows.shape[0]
        mu = np.zeros(m)
        for i in range(cnt):
            mu += rows[i]
        mu /= cnt
        var = np.zeros(m)
        for i in range(cnt):
            t = rows[i] - mu
            var += t * t
        var /= cnt
        s[h] = 1.0 / np.sqrt(var + eps_w)
    return s


# ---------------------------------------------------------------------------------------------------------------
# The steps either side of the path inside the attention block: rotary position embedding on Q and K (Sec. 5.1) and
# Attention = Z V + DWC(V) (Eq. 7)
def rope(X, prefix=0, base=10000.0, inverse=False):
    """Rotary position embedding of X [B,H,n,d] (d even): channel pairs (2i, 2i+1) of the token at grid position p
    are rotated by p * base^(-2i/d); the `prefix` leading tokens are left alone.  inverse=True applies the transpose."""
    X = _f64(X)
    B, H, n, d = X.shape
    out = np.empty_like(X)
    _load().oracle_rope(B * H, n, d, prefix, ctypes.c_double(base), int(inverse), _p(X), _p(out))
    return out


def dwc(V, Wd, prefix, gh, gw):
    """Depth-wise ks x ks cross-correlation of V [B,H,n,d] over the gh x gw token grid, zero padded, one filter per
    head and channel: Wd [H,d,ks,ks].  Prefix tokens receive 0."""
    V, Wd = _f64(V), _f64(Wd)
    B, H, n, d = V.shape
    ks = Wd.shape[-1]
    assert Wd.shape == (H, d, ks, ks) and ks % 2 == 1 and n == prefix + gh * gw
    out = np.empty_like(V)
    _load().oracle_dwc(B, H, n, d, prefix, gh, gw, ks, _p(V), _p(Wd), _p(out))
    return out


def dwc_bwd(V, Wd, dO, prefix, gh, gw):
    """Adjoint of dwc: returns dV [B,H,n,d] and dWd [H,d,ks,ks] (summed over the batch)."""
    V, Wd, dO = _f64(V), _f64(Wd), _f64(dO)
    B, H, n, d = V.shape
    ks = Wd.shape[-1]
    dV, dWd = np.empty_like(V), np.empty_like(Wd)
    _load().oracle_dwc_bwd(B, H, n, d, prefix, gh, gw, ks, _p(V), _p(Wd), _p(dO), _p(dV), _p(dWd))
    return dV, dWd


def round_bf16(x):
    """Nearest bf16 value (8 significant bits, ties to even) of every element, rounded once from float64 and returned
    as float64: the storage rounding a tensor takes when the device keeps it in bf16 (normal range only)."""
    x = np.asarray(x, dtype=np.float64)
    mant, expo = np.frexp(x)                       # x = mant * 2^expo, 0.5 <= |mant| < 1
    return np.ldexp(np.rint(mant * 256.0) / 256.0, expo)      # rint rounds halves to even


def _round_storage(x, store_bf16, store_f32):
    if store_bf16:
        return round_bf16(x)
    if store_f32:
        return x.astype(np.float32).astype(np.float64)       # numpy rounds to nearest, ties to even
    return x


def block_forward(p: Problem, Q, K, V, Wd=None, rope_base=0.0, whiten=None, store_bf16=False, store_f32=False):
    """The attention block around the path: rotary embedding on Q and K (rope_base > 0), the Nystrom Laplacian
    attention, plus DWC(V) (Wd given).  store_bf16 / store_f32: the rotated Q and K are rounded once to the type a
    device keeps them in (the kernel gradient's sign(token - landmark) must be decided on the same numbers: a landmark
    pooled from a single token equals that token only if both went through the same rounding)."""
    Qr, Kr = _f64(Q), _f64(K)
    if rope_base > 0:
        Qr, Kr = rope(Qr, p.prefix, rope_base), rope(Kr, p.prefix, rope_base)
        Qr, Kr = _round_storage(Qr, store_bf16, store_f32), _round_storage(Kr, store_bf16, store_f32)
    O = forward(p, Qr, Kr, V, whiten=whiten)
    if Wd is not None:
        O = O + dwc(V, Wd, p.prefix, p.gh, p.gw)
    return O


def block_backward(p: Problem, Q, K, V, dO, Wd=None, rope_base=0.0, whiten=None, store_bf16=False, store_f32=False):
    """Adjoint of block_forward: dQ, dK, dV, dWd (None without the convolution).  The rounding of the rotated
    tensors, where asked for, is treated as the identity (straight-through), as storage rounding is everywhere."""
    Qr, Kr = _f64(Q), _f64(K)
    if rope_base > 0:
        Qr, Kr = rope(Qr, p.prefix, rope_base), rope(Kr, p.prefix, rope_base)
        Qr, Kr = _round_storage(Qr, store_bf16, store_f32), _round_storage(Kr, store_bf16, store_f32)
    dQr, dKr, dV, _ = backward(p, Qr, Kr, V, dO, whiten=whiten)
    dWd = None
    if Wd is not None:
        dV2, dWd = dwc_bwd(V, Wd, dO, p.prefix, p.gh, p.gw)
        dV = dV + dV2
    if rope_base > 0:
        dQr, dKr = rope(dQr, p.prefix, rope_base, inverse=True), rope(dKr, p.prefix, rope_base, inverse=True)
    return dQr, dKr, dV, dWd


def exact_attention(Q, K, V, lam, map_mode=1):
    """Exact Laplacian-kernel attention (Eq. 4 + Eq. 7, no Nystrom approximation, unit whitening), the plain
    definition: G = k(Q, K) [n x n], Z = G - rowmean(G) + 1/n, O = Z V (map_mode 0: O = G V).  [B,H,n,d] arrays."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    B, H, n, d = Q.shape
    O = np.empty_like(Q)
    for b in range(B):
        for h in range(H):
            G = l1_kernel(Q[b, h][None], K[b, h][None], lam)[0]
            Z = G if map_mode == 0 else G - G.mean(axis=1, keepdims=True) + 1.0 / n
            O[b, h] = Z @ V[b, h]
    return O


# ---------------------------------------------------------------------------------------------------------------
# Whitening with batch statistics (Eq. 5-6 in training mode): the diagonal scale s is estimated from the kernel block
# C = k(Q, L) of the very batch it is applied to, and the gradient flows through the variance.
def forward_batch_whiten(p: Problem, Q, K, V, eps_w, L=None):
    """O and s [H, m]: s_l = 1 / sqrt(Var_{b,i}(C_il) + eps_w) over the query rows of every batch element of head h
    (Eq. 5-6), then the path with that s (Prop. 3)."""
    _, extra = forward(p, Q, K, V, L=L, want=("C",))
    s = whiten_stats(extra["C"], p.H, eps_w)
    return forward(p, Q, K, V, L=L, whiten=s), s


def backward_batch_whiten(p: Problem, Q, K, V, dO, eps_w, L=None):
    """Adjoint of forward_batch_whiten.  With N = B n rows per head, c_l the column mean of C over them,
    Z_il = s_l (C_il - mu_i) + 1/m and dZ = dO Y^T:
        ds_l = sum_{b,i} dZ_il (C_il - mu_i),   dsigma2_l = -1/2 s_l^3 ds_l,   dC_il += dsigma2_l (2/N) (C_il - c_l),
    on top of the gradient with s held constant; the extra dC goes back through C = k(Q, L) (App. A) and, for pooled
    landmarks, through the pooling adjoint."""
    Q, K, V, dO = _f64(Q), _f64(K), _f64(V), _f64(dO)
    B, H, n, d, m = p.B, p.H, p.n, p.d, p.m
    _, x = forward(p, Q, K, V, L=L, want=("C", "L"))
    s = whiten_stats(x["C"], H, eps_w)
    _, x2 = forward(p, Q, K, V, L=L, whiten=s, want=("Y",))
    dQ, dK, dV, dL = backward(p, Q, K, V, dO, L=L, whiten=s)
    C = x["C"].reshape(B, H, n, m)
    Y = x2["Y"].reshape(B, H, m, d)
    Lm = x["L"].reshape(B, H, m, d)
    N = B * n
    for h in range(H):
        ds = np.zeros(m)
        for b in range(B):
            dZ = dO[b, h] @ Y[b, h].T                                   # [n, m]
            ds += (dZ * (C[b, h] - C[b, h].mean(axis=1, keepdims=True))).sum(axis=0)
        cbar = C[:, h].reshape(N, m).mean(axis=0)
        dsig2 = -0.5 * s[h] ** 3 * ds
        for b in range(B):
            dC = dsig2[None, :] * (2.0 / N) * (C[b, h] - cbar[None, :])
            dq, dl = l1_kernel_bwd(Q[b, h][None], Lm[b, h][None], p.lam, dC[None])
            dQ[b, h] += dq[0]
            if p.lm_mode == 0:
                dL[b, h] += dl[0]
            else:
                one = Problem(B=1, H=1, n=n, d=d, m=m, lam=p.lam, ns_iters=0, prefix=p.prefix, gh=p.gh, gw=p.gw, mh=p.mh, mw=p.mw)
                back = landmarks_pool_bwd(one, dl[None])[0, 0]
                if p.lm_mode == 1:
                    dK[b, h] += back
                else:
                    dQ[b, h] += back
    return dQ, dK, dV, dL, s
