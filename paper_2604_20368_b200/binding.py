"""Thin ctypes binding of ``include/laplace_nystrom.h``.

Argument marshalling only: every step of the path runs in the CUDA library.  torch is used
for device memory and streams.  There is no CPU fallback: if the shared library cannot be
loaded, or a tensor is not on a CUDA device, the call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import Optional

import torch

from . import build as _build

LN_F32, LN_BF16 = 0, 1
_STATUS = {0: "ok", -1: "invalid argument", -2: "outside the supported envelope",
           -3: "workspace too small", -4: "CUDA launch failed",
           -5: "problem exceeds the static scratch of the no-allocation entry point"}

EXPORTS = [
    "ln_status_string", "laplace_nystrom_saved_bytes", "laplace_nystrom_workspace_bytes",
    "laplace_nystrom_fwd", "laplace_nystrom_bwd", "ns_pinv_workspace_bytes", "ns_pinv", "ns_pinv_bwd",
    "l1_kernel", "l1_kernel_bwd_workspace_bytes", "l1_kernel_bwd", "landmarks_pool", "landmarks_pool_bwd",
    "ln_trace_begin", "ln_trace_end", "ns_pinv_static_scratch_bytes", "ns_pinv_static",
    "laplace_nystrom_host_staging_bytes", "laplace_nystrom_fwd_bwd_host", "ln_set_overlap", "ln_launch_count",
    "laplace_nystrom_whiten_stats_workspace_bytes", "laplace_nystrom_whiten_stats",
    "laplace_nystrom_saved_array", "ln_set_fused_sign", "laplace_attention_block_saved_bytes",
    "laplace_attention_block_workspace_bytes", "laplace_attention_block_fwd", "laplace_attention_block_bwd", "laplace_exact_fwd", "ln_selftest_wait_timeout", "ln_fp32_add_probe", "ln_fp32_add_probe_lane_ops",
]


class LnError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where}: status {status} ({_STATUS.get(status, 'unknown')})")
        self.status = status


class _CProblem(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("n", ctypes.c_int32), ("d", ctypes.c_int32),
        ("m", ctypes.c_int32), ("lambda_", ctypes.c_float), ("ns_iters", ctypes.c_int32),
        ("ridge_eps", ctypes.c_float), ("ns_alpha", ctypes.c_float), ("dtype", ctypes.c_int32),
        ("map_mode", ctypes.c_int32), ("whiten", ctypes.c_void_p), ("lm_mode", ctypes.c_int32),
        ("prefix", ctypes.c_int32), ("gh", ctypes.c_int32), ("gw", ctypes.c_int32),
        ("mh", ctypes.c_int32), ("mw", ctypes.c_int32),
        ("whiten_mode", ctypes.c_int32), ("whiten_eps", ctypes.c_float), ("whiten_batch", ctypes.c_void_p),
        ("lm_filter", ctypes.c_void_p), ("lm_filter_grad", ctypes.c_void_p),
        ("solver", ctypes.c_int32),
    ]


class _CBlock(ctypes.Structure):
    _fields_ = [("dwc_w", ctypes.c_void_p), ("dwc_ks", ctypes.c_int32), ("rope_base", ctypes.c_float)]


@dataclass
class Problem:
    """The problem statement in the paper's notation (B, heads, n tokens, head dim d, m landmarks,
    decay lambda, Newton-Schulz iteration count)."""
    B: int
    H: int
    n: int
    d: int
    m: int
    lam: float
    ns_iters: int
    ridge_eps: float = 1e-6
    ns_alpha: float = 0.0
    dtype: int = LN_BF16
    map_mode: int = 1
    whiten: Optional[torch.Tensor] = field(default=None, repr=False)   # device fp32 [H, m] or None
    lm_mode: int = 1
    prefix: int = 0
    gh: int = 0
    gw: int = 0
    mh: int = 0
    mw: int = 0
    whiten_mode: int = 0          # 1: s from this batch's kernel block (Eq. 5-6), gradient through the variance
    whiten_eps: float = 1e-5
    whiten_batch: Optional[torch.Tensor] = field(default=None, repr=False)   # device fp32 [H, m], written by the forward pass
    # depth-wise-convolution landmark selection (Sec. 4.2): device fp32 [H, (gh/mh)*(gw/mw), d] each; the gradient is
    # overwritten by the backward pass
    lm_filter: Optional[torch.Tensor] = field(default=None, repr=False)
    lm_filter_grad: Optional[torch.Tensor] = field(default=None, repr=False)
    solver: int = 0   # 0: Newton-Schulz (Alg. 2); 1: conjugate gradients, ns_iters steps (Sec. 5.3, Table 4)

    def c(self) -> _CProblem:
        w = None
        if self.whiten is not None:
            assert self.whiten.is_cuda and self.whiten.dtype == torch.float32 and self.whiten.is_contiguous()
            assert tuple(self.whiten.shape) == (self.H, self.m)
            w = self.whiten.data_ptr()
        return _CProblem(self.B, self.H, self.n, self.d, self.m, float(self.lam), self.ns_iters,
                         float(self.ridge_eps), float(self.ns_alpha), self.dtype, self.map_mode, w,
                         self.lm_mode, self.prefix, self.gh, self.gw, self.mh, self.mw, self.whiten_mode,
                         float(self.whiten_eps), None if self.whiten_batch is None else self.whiten_batch.data_ptr(),
                         self._filter_ptr(self.lm_filter), self._filter_ptr(self.lm_filter_grad), self.solver)

    def _filter_ptr(self, t):
        if t is None:
            return None
        assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
        assert tuple(t.shape) == (self.H, (self.gh // self.mh) * (self.gw // self.mw), self.d)
        return t.data_ptr()

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == LN_F32 else torch.bfloat16


_lib = None


def lib():
    """Load (building first if the sources are newer) the CUDA shared library; raises if impossible."""
    global _lib
    if _lib is None:
        path = _build.LIB
        try:
            path = _build.build()
        except Exception as e:   # no nvcc on this machine: use the library that travelled with the tree
            if not os.path.exists(path):
                raise RuntimeError(f"CUDA library {path} is missing and could not be built: {e}") from e
        L = ctypes.CDLL(path)
        vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float, ctypes.c_size_t
        pp = ctypes.POINTER(_CProblem)
        L.ln_status_string.restype = ctypes.c_char_p
        L.ln_status_string.argtypes = [ctypes.c_int]
        L.laplace_nystrom_saved_bytes.restype = sz
        L.laplace_nystrom_saved_bytes.argtypes = [pp]
        L.laplace_nystrom_workspace_bytes.restype = sz
        L.laplace_nystrom_workspace_bytes.argtypes = [pp, i32]
        L.laplace_nystrom_fwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.laplace_nystrom_bwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.laplace_nystrom_host_staging_bytes.restype = sz
        L.laplace_nystrom_host_staging_bytes.argtypes = [pp]
        L.laplace_nystrom_fwd_bwd_host.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp, sz, vp, vp]
        L.ns_pinv_workspace_bytes.restype = sz
        L.ns_pinv_workspace_bytes.argtypes = [i32, i32, i32]
        L.ns_pinv.argtypes = [i32, i32, vp, i32, f32, f32, vp, vp, vp, vp, sz, vp]
        L.ns_pinv_bwd.argtypes = [i32, i32, vp, i32, f32, f32, vp, vp, vp, vp, sz, vp]
        L.l1_kernel.argtypes = [i32, i32, i32, i32, vp, vp, i32, f32, vp, vp, vp]
        L.l1_kernel_bwd_workspace_bytes.restype = sz
        L.l1_kernel_bwd_workspace_bytes.argtypes = [i32, i32, i32, i32]
        L.l1_kernel_bwd.argtypes = [i32, i32, i32, i32, vp, vp, i32, f32, vp, vp, vp, vp, vp, sz, vp]
        L.landmarks_pool.argtypes = [pp, vp, vp, vp]
        L.landmarks_pool_bwd.argtypes = [pp, vp, vp, vp]
        L.ns_pinv_static_scratch_bytes.restype = sz
        L.ns_pinv_static_scratch_bytes.argtypes = []
        L.ns_pinv_static.argtypes = [i32, i32, vp, i32, f32, f32, vp, vp, vp]
        L.ln_trace_end.argtypes = [i32, ctypes.POINTER(i32), ctypes.POINTER(f32), ctypes.POINTER(ctypes.c_char_p)]
        L.ln_set_overlap.argtypes = [i32]
        L.ln_set_fused_sign.argtypes = [i32]
        L.ln_launch_count.restype = ctypes.c_uint64
        L.ln_launch_count.argtypes = []
        L.laplace_nystrom_whiten_stats_workspace_bytes.restype = sz
        L.laplace_nystrom_whiten_stats_workspace_bytes.argtypes = [ctypes.POINTER(_CProblem)]
        L.laplace_nystrom_whiten_stats.argtypes = [ctypes.POINTER(_CProblem), vp, f32, vp, vp, sz, vp]
        L.laplace_nystrom_saved_array.argtypes = [pp, ctypes.c_char_p, ctypes.POINTER(ctypes.c_int64)]
        L.ln_selftest_wait_timeout.argtypes = [i32, vp, vp]
        L.ln_fp32_add_probe.argtypes = [i32, i32, i32, vp, vp]
        L.ln_fp32_add_probe_lane_ops.restype = ctypes.c_int64
        L.ln_fp32_add_probe_lane_ops.argtypes = [i32, i32, i32]
        L.laplace_exact_fwd.argtypes = [i32, i32, i32, i32, f32, i32, vp, vp, vp, vp, vp]
        pb = ctypes.POINTER(_CBlock)
        L.laplace_attention_block_saved_bytes.restype = sz
        L.laplace_attention_block_saved_bytes.argtypes = [pp, pb]
        L.laplace_attention_block_workspace_bytes.restype = sz
        L.laplace_attention_block_workspace_bytes.argtypes = [pp, pb]
        L.laplace_attention_block_fwd.argtypes = [pp, pb, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.laplace_attention_block_bwd.argtypes = [pp, pb, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("tensor must live on a CUDA device (there is no CPU path)")
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise LnError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LN_F32
    if t.dtype == torch.bfloat16:
        return LN_BF16
    raise ValueError(f"unsupported storage dtype {t.dtype}")


def _bytes(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------------------------------ sizes
def laplace_nystrom_saved_bytes(p: Problem) -> int:
    cp = p.c()
    return int(lib().laplace_nystrom_saved_bytes(ctypes.byref(cp)))


def laplace_nystrom_workspace_bytes(p: Problem, with_saved: bool) -> int:
    cp = p.c()
    return int(lib().laplace_nystrom_workspace_bytes(ctypes.byref(cp), int(with_saved)))


# ------------------------------------------------------------------------------------------ attention
def laplace_nystrom_fwd(p: Problem, Q, K, V, L=None, O=None, saved=None, ws=None, dev_status=None, stream=None):
    """O = Z Y (Alg. 1 + Alg. 2 + Prop. 3).  ``saved``: a uint8 tensor of laplace_nystrom_saved_bytes(p)
    for training, or None for inference.  Returns O."""
    if O is None:
        O = torch.empty_like(Q)
    if ws is None:
        ws = _bytes(laplace_nystrom_workspace_bytes(p, saved is not None), Q.device)
    cp = p.c()
    st = lib().laplace_nystrom_fwd(ctypes.byref(cp), _ptr(Q), _ptr(K), _ptr(V), _ptr(L), _ptr(O), _ptr(saved),
                                   _ptr(ws), ws.numel(), _ptr(dev_status), _stream(stream))
    _check(st, "laplace_nystrom_fwd")
    return O


def laplace_nystrom_bwd(p: Problem, Q, K, V, dO, saved, L=None, dQ=None, dK=None, dV=None, dL=None, ws=None,
                        dev_status=None, stream=None):
    """Exact adjoint of laplace_nystrom_fwd.  Returns dQ, dK, dV, dL (dL is None when lm_mode == 1).
    ``dev_status``: optional int32 [B*H] device tensor that receives the per-head flags."""
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(V) if dV is None else dV
    if p.lm_mode == 0 and dL is None:
        dL = torch.empty_like(L)
    if p.lm_filter is not None and p.lm_filter_grad is None:       # the filter's gradient is left in p.lm_filter_grad
        p.lm_filter_grad = torch.empty_like(p.lm_filter)
    if ws is None:
        ws = _bytes(laplace_nystrom_workspace_bytes(p, True), Q.device)
    cp = p.c()
    st = lib().laplace_nystrom_bwd(ctypes.byref(cp), _ptr(Q), _ptr(K), _ptr(V), _ptr(L), _ptr(dO), _ptr(saved),
                                   _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dL), _ptr(ws), ws.numel(), _ptr(dev_status),
                                   _stream(stream))
    _check(st, "laplace_nystrom_bwd")
    return dQ, dK, dV, dL


class HostStep:
    """Device buffers of laplace_nystrom_fwd_bwd_host for one problem: staging, saved context, workspace."""

    def __init__(self, p: Problem, device):
        cp = p.c()
        self.p = p
        self.staging = _bytes(lib().laplace_nystrom_host_staging_bytes(ctypes.byref(cp)), device)
        self.saved = _bytes(laplace_nystrom_saved_bytes(p), device)
        self.ws = _bytes(laplace_nystrom_workspace_bytes(p, True), device)


def _host_ptr(t: torch.Tensor):
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("laplace_nystrom_fwd_bwd_host takes contiguous host tensors")
    return ctypes.c_void_p(t.data_ptr())


def laplace_nystrom_fwd_bwd_host(p: Problem, bufs: HostStep, hQ, hK, hV, hdO, hO, hdQ, hdK, hdV, stream=None,
                                 dev_status=None):
    """One training step on host tensors (pinned for asynchronous copies): copies in, forward, backward, copies
    out, all enqueued on `stream`; the host outputs are valid after the stream has been synchronised."""
    cp = p.c()
    st = lib().laplace_nystrom_fwd_bwd_host(ctypes.byref(cp), _host_ptr(hQ), _host_ptr(hK), _host_ptr(hV),
                                            _host_ptr(hdO), _host_ptr(hO), _host_ptr(hdQ), _host_ptr(hdK),
                                            _host_ptr(hdV), _ptr(bufs.staging), bufs.staging.numel(),
                                            _ptr(bufs.saved), _ptr(bufs.ws), bufs.ws.numel(), _ptr(dev_status),
                                            _stream(stream))
    _check(st, "laplace_nystrom_fwd_bwd_host")


# ------------------------------------------------------------------------------------------ Newton-Schulz
def ns_pinv(W, iters: int, ridge_eps: float = 0.0, alpha: float = 0.0, want_hist=False, want_resid=False,
            stream=None):
    """T-step Newton-Schulz iterate of (W + eps I)^-1 (Alg. 2).  W: device fp32 [batch, m, m]."""
    batch, m, _ = W.shape
    X = torch.empty_like(W)
    hist = torch.empty((batch, iters + 1, m, m), dtype=torch.float32, device=W.device) if want_hist else None
    resid = torch.empty((batch,), dtype=torch.float32, device=W.device) if want_resid else None
    ws = _bytes(lib().ns_pinv_workspace_bytes(batch, m, iters), W.device)
    st = lib().ns_pinv(batch, m, _ptr(W), iters, ridge_eps, alpha, _ptr(X), _ptr(hist), _ptr(resid), _ptr(ws),
                       ws.numel(), _stream(stream))
    _check(st, "ns_pinv")
    return X, hist, resid


def ns_pinv_bwd(W, iters: int, ridge_eps: float, alpha: float, dX, X_hist=None, stream=None):
    batch, m, _ = W.shape
    dW = torch.empty_like(W)
    ws = _bytes(lib().ns_pinv_workspace_bytes(batch, m, iters), W.device)
    st = lib().ns_pinv_bwd(batch, m, _ptr(W), iters, ridge_eps, alpha, _ptr(X_hist), _ptr(dX), _ptr(dW), _ptr(ws),
                           ws.numel(), _stream(stream))
    _check(st, "ns_pinv_bwd")
    return dW


def ns_pinv_static(W, iters: int, X, ridge_eps: float = 0.0, alpha: float = 0.0, resid=None, stream=None):
    """ns_pinv for callers that cannot allocate: the scratch lives inside the library, so the caller
    hands in only W and the output X (and optionally resid), all allocated beforehand.  Raises
    LnError(-5) when the problem does not fit the library's fixed scratch.  Calls that overlap on
    the GPU share that scratch and must be serialised by the caller."""
    batch, m, _ = W.shape
    st = lib().ns_pinv_static(batch, m, _ptr(W), iters, ridge_eps, alpha, _ptr(X), _ptr(resid), _stream(stream))
    _check(st, "ns_pinv_static")
    return X


# ------------------------------------------------------------------------------------------ kernel block
def l1_kernel(A, Bm, lam: float, want_rowsum=False, stream=None):
    """K[b,i,j] = exp(-||A[b,i]-Bm[b,j]||_1 / lam) (Sec. 1, Eq. 8).  A [batch,na,d], Bm [batch,nb,d]."""
    batch, na, d = A.shape
    nb = Bm.shape[1]
    Kout = torch.empty((batch, na, nb), dtype=torch.float32, device=A.device)
    rs = torch.empty((batch, na), dtype=torch.float32, device=A.device) if want_rowsum else None
    st = lib().l1_kernel(batch, na, nb, d, _ptr(A), _ptr(Bm), _dtype_code(A), lam, _ptr(Kout), _ptr(rs),
                         _stream(stream))
    _check(st, "l1_kernel")
    return (Kout, rs) if want_rowsum else Kout


def l1_kernel_bwd(A, Bm, lam: float, dK, Kmat=None, stream=None):
    batch, na, d = A.shape
    nb = Bm.shape[1]
    dA, dB = torch.empty_like(A), torch.empty_like(Bm)
    ws = _bytes(lib().l1_kernel_bwd_workspace_bytes(batch, na, nb, d), A.device)
    st = lib().l1_kernel_bwd(batch, na, nb, d, _ptr(A), _ptr(Bm), _dtype_code(A), lam, _ptr(Kmat), _ptr(dK),
                             _ptr(dA), _ptr(dB), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "l1_kernel_bwd")
    return dA, dB


# ------------------------------------------------------------------------------------------ landmarks
def landmarks_pool(p: Problem, K, stream=None):
    L = torch.empty((p.B, p.H, p.m, p.d), dtype=torch.float32, device=K.device)
    cp = p.c()
    _check(lib().landmarks_pool(ctypes.byref(cp), _ptr(K), _ptr(L), _stream(stream)), "landmarks_pool")
    return L


def landmarks_pool_bwd(p: Problem, dL, stream=None):
    dK = torch.empty((p.B, p.H, p.n, p.d), dtype=p.torch_dtype, device=dL.device)
    cp = p.c()
    _check(lib().landmarks_pool_bwd(ctypes.byref(cp), _ptr(dL), _ptr(dK), _stream(stream)), "landmarks_pool_bwd")
    return dK


def set_overlap(enabled: bool) -> bool:
    """Whether the per-head kernels run on the library's second stream beside the token-sized ones
    (default on); returns the previous setting."""
    return bool(lib().ln_set_overlap(1 if enabled else 0))


class Block:
    """The steps around the path inside the attention block: rotary embedding base (0 = off) and the depth-wise
    convolution filters (device fp32 [H, d, ks, ks] or None)."""

    def __init__(self, dwc_w: Optional[torch.Tensor] = None, rope_base: float = 0.0):
        self.dwc_w, self.rope_base = dwc_w, float(rope_base)
        if dwc_w is not None:
            assert dwc_w.is_cuda and dwc_w.dtype == torch.float32 and dwc_w.is_contiguous() and dwc_w.dim() == 4
            assert dwc_w.shape[2] == dwc_w.shape[3]

    def c(self) -> _CBlock:
        return _CBlock(None if self.dwc_w is None else self.dwc_w.data_ptr(), 0 if self.dwc_w is None else int(self.dwc_w.shape[-1]),
                       self.rope_base)


def laplace_attention_block_fwd(p: Problem, blk: Block, Q, K, V, saved=None, ws=None, O=None, dev_status=None, stream=None):
    """O = Z(rope(Q), rope(K)) Y + DWC(V) (Eq. 7, Sec. 5.1).  Returns O, saved, ws (allocated when not given)."""
    cp, cb = p.c(), blk.c()
    if saved is None:
        saved = _bytes(lib().laplace_attention_block_saved_bytes(ctypes.byref(cp), ctypes.byref(cb)), Q.device)
    if ws is None:
        ws = _bytes(lib().laplace_attention_block_workspace_bytes(ctypes.byref(cp), ctypes.byref(cb)), Q.device)
    if O is None:
        O = torch.empty_like(Q)
    _check(lib().laplace_attention_block_fwd(ctypes.byref(cp), ctypes.byref(cb), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(saved),
                                             _ptr(ws), ws.numel(), _ptr(dev_status), _stream(stream)), "laplace_attention_block_fwd")
    return O, saved, ws


def laplace_attention_block_bwd(p: Problem, blk: Block, Q, K, V, dO, saved, ws, dev_status=None, stream=None):
    """Adjoint of laplace_attention_block_fwd: dQ, dK, dV, dWd (None without the convolution branch)."""
    cp, cb = p.c(), blk.c()
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    dWd = None if blk.dwc_w is None else torch.empty_like(blk.dwc_w)
    _check(lib().laplace_attention_block_bwd(ctypes.byref(cp), ctypes.byref(cb), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(saved),
                                             _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dWd), _ptr(ws), ws.numel(), _ptr(dev_status),
                                             _stream(stream)), "laplace_attention_block_bwd")
    return dQ, dK, dV, dWd


def laplace_exact_fwd(Q, K, V, lam: float, map_mode: int = 1, stream=None):
    """Exact (m = n) Laplacian-kernel attention of Q, K, V [B, H, n, d] (Eq. 4 + Eq. 7, full kernel matrix on chip)."""
    B, H, n, d = Q.shape
    O = torch.empty_like(Q)
    _check(lib().laplace_exact_fwd(B * H, n, d, _dtype_code(Q), lam, map_mode, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _stream(stream)),
           "laplace_exact_fwd")
    return O


def set_fused_sign(enabled: bool) -> bool:
    """Whether the bf16 sign passes form their upstream factor on the tensor cores themselves (default) or read it
    from the workspace, where separate product kernels left it; returns the previous setting.  Set it before the
    workspace is sized."""
    return bool(lib().ln_set_fused_sign(1 if enabled else 0))


def laplace_nystrom_whiten_stats(p: Problem, saved, eps_w: float = 1e-5, out=None, ws=None, stream=None):
    """Whitening scale s [H, m] (Eq. 5-6) from the kernel block a forward call left in ``saved``."""
    if saved is None or not saved.is_cuda:
        raise ValueError("saved must be the CUDA context buffer of a forward call")
    cp = p.c()
    need = lib().laplace_nystrom_whiten_stats_workspace_bytes(ctypes.byref(cp))
    if ws is None:
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=saved.device)
    if out is None:
        out = torch.empty((p.H, p.m), dtype=torch.float32, device=saved.device)
    _check(lib().laplace_nystrom_whiten_stats(ctypes.byref(cp), _ptr(saved), eps_w, _ptr(out), _ptr(ws), ws.numel(),
                                              _stream(stream)), "laplace_nystrom_whiten_stats")
    return out


def saved_array(p: Problem, saved: torch.Tensor, name: str) -> torch.Tensor:
    """A strided fp32 view [B*H, rows, cols] of a named intermediate inside the forward context ``saved``
    (laplace_nystrom_saved_array): "L", "C", "Rt", "mu", "W", "X", "M", "Yt", "ybar"."""
    info = (ctypes.c_int64 * 5)()
    cp = p.c()
    _check(lib().laplace_nystrom_saved_array(ctypes.byref(cp), name.encode(), info), "laplace_nystrom_saved_array")
    off, rows, cols, ld, stride = (int(v) for v in info)
    flat = saved.view(torch.float32)
    return torch.as_strided(flat, (p.B * p.H, rows, cols), (stride, ld, 1), off)


def selftest_wait_timeout(dev_status: torch.Tensor, probes: int = 1000, stream=None):
    """Run the bounded-wait self-test: ORs bit 1 into dev_status[0] once the wait has given up."""
    _check(lib().ln_selftest_wait_timeout(probes, _ptr(dev_status), _stream(stream)), "ln_selftest_wait_timeout")


def fp32_add_probe(blocks: int, iters: int, mode: int, sink: torch.Tensor, stream=None) -> int:
    """Launch the FP32 rate probe (mode 0 scalar adds, 1 packed adds, 2 sign-pass mix, 3 l1-forward mix); returns the
    lane-operations the launch performs."""
    _check(lib().ln_fp32_add_probe(blocks, iters, int(mode), _ptr(sink), _stream(stream)), "ln_fp32_add_probe")
    return int(lib().ln_fp32_add_probe_lane_ops(blocks, iters, int(mode)))


def launch_count() -> int:
    """Kernels the library has launched in this process so far."""
    return int(lib().ln_launch_count())


# ------------------------------------------------------------------------------------------ profiling aid
def trace_begin():
    """Start bracketing every library launch with CUDA events (profiling only)."""
    _check(lib().ln_trace_begin(), "ln_trace_begin")


def trace_end(capacity: int = 2048):
    """Stop tracing; returns [(kernel name, milliseconds), ...] in launch order (synchronises)."""
    cnt = ctypes.c_int32(0)
    ms = (ctypes.c_float * capacity)()
    names = (ctypes.c_char_p * capacity)()
    _check(lib().ln_trace_end(capacity, ctypes.byref(cnt), ms, names), "ln_trace_end")
    k = min(cnt.value, capacity)
    return [(names[i].decode(), float(ms[i])) for i in range(k)]
