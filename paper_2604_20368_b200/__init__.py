"""B200 (sm_100a) Nystrom-approximated Laplacian-kernel attention, forward and backward.

The work is done by hand-written CUDA kernels behind the C ABI declared in
``include/laplace_nystrom.h``; ``binding`` marshals arguments to it.  ``synth`` draws the seeded
synthetic inputs.  The shared library is loaded on first use and there is no CPU fallback.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    LN_BF16, LN_F32, LnError, Problem, l1_kernel, l1_kernel_bwd, landmarks_pool, landmarks_pool_bwd,
    laplace_nystrom_bwd, laplace_nystrom_fwd, laplace_nystrom_saved_bytes, laplace_nystrom_workspace_bytes,
    ns_pinv, ns_pinv_bwd, ns_pinv_static, trace_begin, trace_end, HostStep, laplace_nystrom_fwd_bwd_host,
    set_overlap, set_fused_sign, laplace_exact_fwd, Block, laplace_attention_block_fwd, laplace_attention_block_bwd, launch_count, laplace_nystrom_whiten_stats, saved_array, selftest_wait_timeout, fp32_add_probe,
)


def problem_from_config(cfg: "synth.Config", whiten=None, map_mode: int = 1) -> Problem:
    """The ln_problem of a synthetic workload (landmarks pooled from the keys)."""
    return Problem(B=cfg.B, H=cfg.H, n=cfg.n, d=cfg.d, m=cfg.m, lam=cfg.lam, ns_iters=cfg.T,
                   ridge_eps=cfg.ridge_eps, dtype=LN_F32 if cfg.dtype == "f32" else LN_BF16,
                   map_mode=map_mode, whiten=whiten, lm_mode=1, prefix=cfg.prefix, gh=cfg.gh, gw=cfg.gw,
                   mh=cfg.mh, mw=cfg.mw)
