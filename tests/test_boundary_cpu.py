"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes are sane, and argument errors are reported before anything is launched."""
import ctypes
import os
import re

import pytest
import torch

import paper_2604_20368_b200 as ln
from paper_2604_20368_b200 import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "laplace_nystrom.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:int|size_t|uint64_t|int64_t|const char\*)\s+(\w+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    syms = declared_symbols()
    assert set(syms) == set(binding.EXPORTS)
    for s in syms:
        assert hasattr(lib, s), s
    assert lib.ln_status_string(0) == b"ok"
    assert lib.ln_status_string(-3) == b"workspace too small"


def _problem(**kw):
    cfg = synth.CONFIGS["cfg2"]
    p = ln.problem_from_config(cfg)
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_sizes_positive_and_monotone():
    p = _problem()
    sb = ln.laplace_nystrom_saved_bytes(p)
    assert sb > 0
    assert ln.laplace_nystrom_workspace_bytes(p, True) > 0
    assert ln.laplace_nystrom_workspace_bytes(p, False) >= sb
    assert ln.laplace_nystrom_saved_bytes(_problem(B=128)) > sb
    assert binding.lib().ns_pinv_workspace_bytes(4, 64, 6) > 0
    assert binding.lib().ns_pinv_workspace_bytes(0, 64, 6) == 0
    assert binding.lib().l1_kernel_bwd_workspace_bytes(2, 100, 30, 64) > 0


@pytest.mark.parametrize("kw", [
    dict(lam=0.0), dict(lam=float("nan")), dict(ns_iters=-1), dict(ridge_eps=-1.0), dict(m=500),
    dict(n=196), dict(mh=6), dict(dtype=7), dict(map_mode=2), dict(B=0), dict(gh=0),
])
def test_invalid_problem_is_rejected_on_the_host(kw):
    p = _problem(**kw)
    assert ln.laplace_nystrom_saved_bytes(p) == 0
    cp = p.c()
    fake = ctypes.c_void_p(4096)   # never dereferenced: validation fails first
    st = binding.lib().laplace_nystrom_fwd(ctypes.byref(cp), fake, fake, fake, None, fake, None, fake, 1 << 40,
                                          None, None)
    assert st in (-1, -2)


def test_unsupported_envelope_and_null_and_workspace():
    lib = binding.lib()
    fake = ctypes.c_void_p(4096)
    cp = _problem(d=48).c()
    assert lib.laplace_nystrom_fwd(ctypes.byref(cp), fake, fake, fake, None, fake, None, fake, 1 << 40, None, None) == -2
    cp = _problem().c()
    assert lib.laplace_nystrom_fwd(ctypes.byref(cp), None, fake, fake, None, fake, None, fake, 1 << 40, None, None) == -1
    assert lib.laplace_nystrom_fwd(ctypes.byref(cp), fake, fake, fake, None, fake, None, fake, 16, None, None) == -3
    # lm_mode 1 forbids a landmark tensor, misaligned pointers are refused
    assert lib.laplace_nystrom_fwd(ctypes.byref(cp), fake, fake, fake, fake, fake, None, fake, 1 << 40, None, None) == -1
    odd = ctypes.c_void_p(4100)
    assert lib.laplace_nystrom_fwd(ctypes.byref(cp), odd, fake, fake, None, fake, None, fake, 1 << 40, None, None) == -1
    assert lib.ns_pinv(1, 300, fake, 2, 0.0, 0.0, fake, None, None, fake, 1 << 40, None) == -2
    assert lib.ns_pinv(1, 8, fake, 2, 0.0, 0.0, fake, None, None, fake, 8, None) == -3
    assert lib.l1_kernel(1, 4, 4, 0, fake, fake, 0, 1.0, fake, None, None) == -1
    assert lib.l1_kernel_bwd(1, 4, 4, 48, fake, fake, 0, 1.0, None, fake, fake, fake, fake, 1 << 40, None) == -2


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(ValueError):
        ln.l1_kernel(torch.zeros(1, 4, 8), torch.zeros(1, 4, 8), 1.0)


def test_config_table_matches_the_workloads():
    c = synth.CONFIGS
    assert (c["cfg1"].n, c["cfg1"].m, c["cfg1"].dtype, c["cfg1"].backward) == (196, 32, "f32", False)
    assert (c["cfg2"].n, c["cfg2"].m, c["cfg2"].B * c["cfg2"].H) == (197, 49, 384)
    assert (c["cfg3"].n, c["cfg3"].m) == (3136, 64)
    assert [c[k].n for k in ("cfg4a", "cfg4b", "cfg4c")] == [3136, 12544, 50176]
    assert c["cfg5_m256_T12"].n == 4096 and c["cfg5_m256_T12"].d == 128
    for cfg in c.values():
        assert cfg.mh * cfg.mw == cfg.m and cfg.lam == cfg.d


def test_generator_is_seeded_and_duplicates_bins():
    import torch
    cfg = synth.shrink(synth.CONFIGS["cfg5_m64_T4"], B=1, H=2)
    a, b = synth.make_inputs(cfg), synth.make_inputs(cfg)
    for k in a:
        assert torch.equal(a[k], b[k])
    assert a["Q"].dtype == torch.bfloat16 and a["whiten"].shape == (2, 64)
    # about 10 % of the keys are copies: count rows that occur more than once
    K = a["K"][0, 0].to(torch.float32)
    uniq = torch.unique(K, dim=0).shape[0]
    ndup_tokens = K.shape[0] - uniq
    assert ndup_tokens == 7 * 64          # ceil(0.1*64) = 7 bins of 8x8 tokens


def test_host_step_argument_errors_without_gpu():
    """The host-buffer entry point validates before it touches CUDA: sizes, NULL pointers, lm_mode."""
    lib = binding.lib()
    p = _problem()
    cp = p.c()
    one = 64 * 6 * 197 * 64 * 2
    need = lib.laplace_nystrom_host_staging_bytes(ctypes.byref(cp))
    assert need >= 8 * one and need % 256 == 0
    bad = _problem(lm_mode=0).c()
    buf = ctypes.create_string_buffer(96)
    a = ctypes.c_void_p((ctypes.addressof(buf) + 15) // 16 * 16)      # 16-byte aligned, never dereferenced
    call = lambda prob, staging, nbytes: lib.laplace_nystrom_fwd_bwd_host(
        ctypes.byref(prob), a, a, a, a, a, a, a, a, staging, nbytes, a, a, 1 << 40, None, None)
    assert call(bad, a, need) == -2                     # landmarks must come from pooling
    assert call(cp, None, need) == -1                   # NULL staging
    assert call(cp, a, need - 1) == -3                  # staging too small
    assert lib.laplace_nystrom_host_staging_bytes(ctypes.byref(_problem(n=0).c())) == 0


def test_filter_selection_argument_errors_without_gpu():
    """The landmark-selection filter (Sec. 4.2) needs regions that divide the grid, one pooled tensor, and in the
    backward pass a buffer for its gradient: refused on the host before anything is enqueued."""
    lib = binding.lib()
    buf = ctypes.create_string_buffer(96)
    a = ctypes.c_void_p((ctypes.addressof(buf) + 15) // 16 * 16)      # 16-byte aligned, never dereferenced

    def with_filter(cfg_name, lm_mode, grad):
        cp = ln.problem_from_config(synth.CONFIGS[cfg_name]).c()
        cp.lm_mode, cp.lm_filter, cp.lm_filter_grad = lm_mode, a.value, (a.value if grad else None)
        return cp
    fwd = lambda cp: lib.laplace_nystrom_fwd(ctypes.byref(cp), a, a, a, None, a, a, a, 0, None, None)
    bwd = lambda cp: lib.laplace_nystrom_bwd(ctypes.byref(cp), a, a, a, None, a, a, a, a, a, None, a, 0, None, None)
    assert fwd(with_filter("cfg2", 1, False)) == -3                 # valid problem: only the (empty) workspace is refused
    assert fwd(with_filter("cfg4a", 1, False)) == -1                # 56 columns do not divide into 16 regions
    assert fwd(with_filter("cfg2", 3, False)) == -2                 # two landmark sets: not with a filter
    assert fwd(with_filter("cfg2", 0, False)) == -1                 # given landmarks: nothing is selected
    assert bwd(with_filter("cfg2", 1, False)) == -1                 # no buffer for the filter's gradient
    assert bwd(with_filter("cfg2", 1, True)) == -3
    odd = with_filter("cfg2", 1, False); odd.lm_filter = a.value + 4
    assert fwd(odd) == -1                                           # not 16-byte aligned


def test_solver_argument_errors_without_gpu():
    """ln_problem.solver: 0 (Newton-Schulz) or 1 (conjugate gradients, Sec. 5.3); conjugate gradients need the symmetric
    matrix of one landmark set."""
    lib = binding.lib()
    buf = ctypes.create_string_buffer(96)
    a = ctypes.c_void_p((ctypes.addressof(buf) + 15) // 16 * 16)      # 16-byte aligned, never dereferenced

    def with_solver(solver, lm_mode):
        cp = ln.problem_from_config(synth.CONFIGS["cfg2"]).c()
        cp.solver, cp.lm_mode = solver, lm_mode
        return cp
    fwd = lambda cp: lib.laplace_nystrom_fwd(ctypes.byref(cp), a, a, a, None, a, a, a, 0, None, None)
    assert fwd(with_solver(1, 1)) == -3                             # valid: only the (empty) workspace is refused
    assert fwd(with_solver(1, 2)) == -3
    assert fwd(with_solver(2, 1)) == -1
    assert fwd(with_solver(-1, 1)) == -1
    assert fwd(with_solver(1, 3)) == -2                             # W = k(pool Q, pool K) is not symmetric
    bw = with_solver(1, 1); bw.whiten_mode, bw.whiten, bw.whiten_batch = 1, None, a.value
    assert fwd(bw) == -2                                            # batch-statistic whitening with this solver: not built
    # the solver's scratch is part of the workspace the caller is told to bring
    p0, p1 = with_solver(0, 1), with_solver(1, 1)
    for with_saved in (0, 1):
        assert lib.laplace_nystrom_workspace_bytes(ctypes.byref(p1), with_saved) > lib.laplace_nystrom_workspace_bytes(ctypes.byref(p0), with_saved)


def test_overlap_switch_and_launch_counter_without_gpu():
    """ln_set_overlap returns the previous setting (default on); the launch counter is readable and has not moved
    without a launch."""
    assert ln.set_overlap(False) is True
    assert ln.set_overlap(True) is False
    assert ln.set_overlap(True) is True
    c0 = ln.launch_count()
    assert c0 >= 0 and ln.launch_count() == c0


def test_whiten_stats_argument_errors_without_gpu():
    p = _problem()
    cp = p.c()
    lib = binding.lib()
    assert lib.laplace_nystrom_whiten_stats_workspace_bytes(ctypes.byref(cp)) > 0
    # NULL buffers are refused on the host before anything is enqueued
    assert lib.laplace_nystrom_whiten_stats(ctypes.byref(cp), None, 1e-5, None, None, 0, None) == -1
    with pytest.raises(ValueError):
        ln.laplace_nystrom_whiten_stats(p, torch.empty(16, dtype=torch.uint8))


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg4a", "cfg5_m256_T12"])
def test_saved_array_views_lie_inside_the_context(name):
    """The inspection entry point is pure host arithmetic: every named intermediate lies inside the saved buffer,
    heads do not overlap, and an unknown name is an argument error."""
    cfg = synth.CONFIGS[name]
    p = ln.problem_from_config(cfg)
    total = ln.laplace_nystrom_saved_bytes(p) // 4
    cp = p.c()
    info = (ctypes.c_int64 * 5)()
    BH = cfg.B * cfg.H
    spans = []
    for nm, rows, cols in (("L", cfg.m, cfg.d), ("C", cfg.n, cfg.m), ("Rt", cfg.n, cfg.m), ("mu", 1, cfg.n),
                           ("W", cfg.m, cfg.m), ("X", cfg.m, cfg.m), ("M", cfg.m, cfg.d), ("Yt", cfg.m, cfg.d),
                           ("ybar", 1, cfg.d)):
        assert binding.lib().laplace_nystrom_saved_array(ctypes.byref(cp), nm.encode(), info) == 0
        off, r, c, ld, stride = (int(v) for v in info)
        assert (r, c) == (rows, cols) and ld >= c and stride >= (r - 1) * ld + c
        assert 0 <= off and off + (BH - 1) * stride + (r - 1) * ld + c <= total
        spans.append((off, off + (BH - 1) * stride + (r - 1) * ld + c, nm))
    spans.sort()
    for (a0, a1, na), (b0, b1, nb) in zip(spans, spans[1:]):
        assert a1 <= b0 or {na, nb} == {"X"}, (na, nb)
    assert binding.lib().laplace_nystrom_saved_array(ctypes.byref(cp), b"nope", info) == -1
