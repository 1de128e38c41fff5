"""ctypes marshalling for ``include/sfda.h``.  Same names, same argument order."""
import ctypes
import os

import torch

SFDA_F32, SFDA_BF16 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

_vp, _ci, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t


class SfdaError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s failed: %d (%s)" % (where, status, sfda_status_string(status)))


def lib_path() -> str:
    return os.path.join(_HERE, "libsfda.so")


def load():
    """Load ``libsfda.so``; raise if it has not been built (no fallback exists).  A library that was not built from
    the sources now in the tree is rebuilt first: an out-of-date kernel must never be what a test or a benchmark runs."""
    global _LIB
    if _LIB is None:
        path = lib_path()
        from . import build as _build
        if os.path.abspath(path) == os.path.abspath(_build.LIB) and os.path.exists(path) and _build.is_stale():
            if int(os.environ.get("LOCAL_RANK", "0")) == 0:
                _build.build(force=True)
            else:                                   # several ranks on one node: the first one builds, the others wait for it
                import time
                for _ in range(1800):
                    if not _build.is_stale():
                        break
                    time.sleep(1.0)
        _LIB = load_library(path)
    return _LIB


def load_library(path):
    """Open a build of the library at `path` and declare the argument types of its entry points."""
    if not os.path.exists(path):
        raise ImportError("%s is missing: run `python -m paper_2607_11897_b200.build` "
                          "(or __graft_entry__.build()) first" % path)
    lib = ctypes.CDLL(path)
    lib.sfda_status_string.restype = ctypes.c_char_p
    lib.sfda_status_string.argtypes = [_ci]
    lib.sfda_plan.argtypes = [_ci, _ci, ctypes.POINTER(_ci), ctypes.POINTER(_ci)]
    lib.sfda_workspace_bytes.restype = _sz
    lib.sfda_workspace_bytes.argtypes = [_ci] * 7
    lib.sfda_forward_partition.argtypes = [_ci] * 7 + [_sz, _ci] + [ctypes.POINTER(_ci)] * 3
    lib.sfda_forward.argtypes = [_vp] * 10 + [_ci] * 7 + [_vp, _sz, _vp]
    lib.sfda_forward_simt.argtypes = [_vp] * 10 + [_ci] * 7 + [_vp]
    lib.sfda_forward_phase.argtypes = [_vp] * 11 + [_ci] * 7 + [_vp, _sz, _vp]
    lib.sfda_forward_withheld_handoff.argtypes = [_vp] * 10 + [_ci] * 8 + [ctypes.c_uint, _vp, _sz, _vp]
    lib.sfda_chunk_factors.argtypes = [_vp] * 9 + [_ci] * 6 + [_vp]
    lib.sfda_step.argtypes = [_vp] * 9 + [_ci] * 5 + [_vp]
    lib.sfda_forward_host_arena_bytes.restype = _sz
    lib.sfda_forward_host_arena_bytes.argtypes = [_ci] * 10
    lib.sfda_forward_host.argtypes = [_vp] * 10 + [_ci] * 7 + [_vp, _sz, _vp, ctypes.POINTER(_sz),
                                                          ctypes.POINTER(_sz)]
    lib.sfda_last_launch_count.restype = _ci
    lib.sfda_forward_noalloc.argtypes = [_vp] * 10 + [_ci] * 7 + [_vp]
    lib.sfda_noalloc_status.argtypes = [_vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.sfda_workspace_status.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_uint32)]
    _cf = ctypes.c_float
    lib.sfda_frontend.argtypes = [_vp] * 4 + [_cf] * 4 + [_vp] * 4 + [_ci] * 5 + [_vp]
    lib.sfda_forward_fused_workspace_bytes.restype = _sz
    lib.sfda_forward_fused_workspace_bytes.argtypes = [_ci] * 7
    lib.sfda_forward_fused.argtypes = [_vp] * 6 + [_cf] * 4 + [_vp] * 4 + [_ci] * 7 + [_vp, _sz, _vp]
    lib.sfda_step_fused.argtypes = [_vp] * 6 + [_cf] * 4 + [_vp] * 3 + [_ci] * 5 + [_vp]
    lib.sfda_backward_workspace_bytes.restype = _sz
    lib.sfda_backward_workspace_bytes.argtypes = [_ci] * 6
    lib.sfda_backward.argtypes = [_vp] * 17 + [_ci] * 6 + [_vp, _sz, _vp]
    lib.sfda_forward_two_level_workspace_bytes.restype = _sz
    lib.sfda_forward_two_level_workspace_bytes.argtypes = [_ci] * 8
    lib.sfda_forward_two_level.argtypes = [_vp] * 10 + [_ci] * 8 + [_vp, _sz, _vp]
    lib.sfda_step_decoupled.argtypes = [_vp] * 11 + [_ci] * 5 + [_vp]
    lib.sfda_forward_decoupled.argtypes = [_vp] * 12 + [_ci] * 6 + [_vp]
    lib.sfda_frontend_backward.argtypes = [_vp] * 4 + [_cf] * 4 + [_vp] * 8 + [_ci] * 5 + [_vp]
    lib.sfda_step_blocks.argtypes = [_vp] * 12 + [_ci] * 6 + [_vp]
    lib.sfda_forward_blocks.argtypes = [_vp] * 13 + [_ci] * 7 + [_vp]
    return lib


def sfda_status_string(status: int) -> str:
    return load().sfda_status_string(int(status)).decode()


def last_launch_count() -> int:
    return int(load().sfda_last_launch_count())


def sfda_plan(T: int, chunk: int):
    n, tail = _ci(), _ci()
    rc = load().sfda_plan(T, chunk, ctypes.byref(n), ctypes.byref(tail))
    if rc != 0:
        raise SfdaError(rc, "sfda_plan")
    return n.value, tail.value


def sfda_workspace_bytes(B, T, H, d_k, d_v, chunk, dtype) -> int:
    return int(load().sfda_workspace_bytes(B, T, H, d_k, d_v, chunk, dtype))


def sfda_forward_partition(B, T, H, d_k, d_v, chunk, dtype, workspace_bytes, n_sm):
    """(slices, balanced, ctas) that sfda_forward would use on a device of n_sm multiprocessors (host only)."""
    q, b, c = _ci(), _ci(), _ci()
    rc = load().sfda_forward_partition(B, T, H, d_k, d_v, chunk, dtype, workspace_bytes, n_sm, ctypes.byref(q),
                                       ctypes.byref(b), ctypes.byref(c))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_partition")
    return q.value, b.value, c.value


def _ptr(t):
    return None if t is None else _vp(t.data_ptr())


def _dtype_code(t):
    if t.dtype == torch.float32:
        return SFDA_F32
    if t.dtype == torch.bfloat16:
        return SFDA_BF16
    raise TypeError("q, k, v must be float32 or bfloat16")


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return _vp(s.cuda_stream)


def _check(t, name, dtype=None, device="cuda"):
    if t is None:
        return
    if not t.is_contiguous():
        raise ValueError(name + " must be contiguous")
    if t.device.type != device:
        raise ValueError("%s must live on %s" % (name, device))
    if dtype is not None and t.dtype != dtype:
        raise TypeError("%s must be %s" % (name, dtype))


def _forward_common(fn_name, q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, workspace, stream):
    lib = load()
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    dt = _dtype_code(q)
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (beta, "beta"), (S0, "S0"), (S_T, "S_T")):
        _check(t, n, torch.float32)
    if fn_name == "sfda_forward_noalloc":
        rc = lib.sfda_forward_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0),
                                      _ptr(o), _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v, chunk, dt, _stream(stream))
    elif fn_name == "sfda_forward":
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        rc = lib.sfda_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0), _ptr(o),
                              _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v, chunk, dt, _ptr(workspace), ws_bytes,
                              _stream(stream))
    else:
        rc = lib.sfda_forward_simt(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0),
                                   _ptr(o), _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v, chunk, dt, _stream(stream))
    if rc != 0:
        raise SfdaError(rc, fn_name)


def sfda_forward(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, workspace=None, stream=None):
    """``sfda_forward`` of ``include/sfda.h``; tensors are CUDA tensors the caller allocated."""
    _forward_common("sfda_forward", q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, workspace, stream)


def sfda_forward_phase(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, phase_turns, chunk, workspace, stream=None):
    """``sfda_forward_phase`` of ``include/sfda.h``: the tensor-core forward that also writes the chunk-closing
    integer phase ``phase_turns`` ([B][H][NC][m], int32 tensor holding the uint32 bit patterns)."""
    lib = load()
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (beta, "beta"), (S0, "S0"), (S_T, "S_T")):
        _check(t, n, torch.float32)
    _check(phase_turns, "phase_turns", torch.int32)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.sfda_forward_phase(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0), _ptr(o),
                                _ptr(o_im), _ptr(S_T), _ptr(phase_turns), B, T, H, d_k, d_v, chunk, _dtype_code(q),
                                _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_phase")


def sfda_forward_withheld_handoff(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, slices, wait_ticks, workspace,
                                  stream=None):
    """``sfda_forward_withheld_handoff`` of ``include/sfda.h``: the diagnostic launch whose time slices never
    announce their boundary states, so that every later slice's bounded wait runs out."""
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().sfda_forward_withheld_handoff(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0),
                                              _ptr(o), _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v, chunk, _dtype_code(q),
                                              int(slices), int(wait_ticks), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_withheld_handoff")


def sfda_workspace_status(workspace, stream=None) -> int:
    """``sfda_workspace_status``: 0, or raises SfdaError(-7) when a device-side wait ran out."""
    word = ctypes.c_uint32()
    rc = load().sfda_workspace_status(_ptr(workspace), _stream(stream), ctypes.byref(word))
    if rc != 0:
        raise SfdaError(rc, "sfda_workspace_status")
    return int(word.value)


def sfda_forward_noalloc(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, stream=None):
    """``sfda_forward_noalloc`` of ``include/sfda.h``: the forward on the library's own static scratch block,
    for callers that may not allocate device memory.  Same tensors as ``sfda_forward``, no workspace."""
    _forward_common("sfda_forward_noalloc", q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, None, stream)


def sfda_noalloc_status(stream=None) -> int:
    """``sfda_noalloc_status``: 0, or raises SfdaError(-7) when a device-side wait of the last
    ``sfda_forward_noalloc`` call ran out.  Synchronises the stream."""
    word = ctypes.c_uint32()
    rc = load().sfda_noalloc_status(_stream(stream), ctypes.byref(word))
    if rc != 0:
        raise SfdaError(rc, "sfda_noalloc_status")
    return int(word.value)


def sfda_forward_simt(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, stream=None):
    """``sfda_forward_simt`` of ``include/sfda.h`` (fp32 CUDA-core path for any dtype)."""
    _forward_common("sfda_forward_simt", q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, None, stream)


def sfda_chunk_factors(k, alpha, theta, beta, Gamma, Y, M, W, phase_turns, chunk, stream=None):
    """``sfda_chunk_factors`` of ``include/sfda.h``; any output may be None."""
    B, T, H, d_k = k.shape
    _check(k, "k")
    for t, n in ((alpha, "alpha"), (theta, "theta"), (beta, "beta"), (Gamma, "Gamma"), (Y, "Y"), (M, "M"),
                 (W, "W")):
        _check(t, n, torch.float32)
    _check(phase_turns, "phase_turns", torch.int32)
    rc = load().sfda_chunk_factors(_ptr(k), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(Gamma), _ptr(Y), _ptr(M),
                                   _ptr(W), _ptr(phase_turns), B, T, H, d_k, chunk, _dtype_code(k),
                                   _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_chunk_factors")


def sfda_step(q, k, v, alpha, theta, beta, S, o, o_im, stream=None):
    """``sfda_step`` of ``include/sfda.h``; S is updated in place."""
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (beta, "beta"), (S, "S")):
        _check(t, n, torch.float32)
    rc = load().sfda_step(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S), _ptr(o),
                          _ptr(o_im), B, H, d_k, d_v, _dtype_code(q), _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_step")


def sfda_forward_host(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, arena, stream=None):
    """``sfda_forward_host``: q..S_T are HOST tensors (pinned), arena a CUDA byte tensor.

    Returns (bytes_h2d, bytes_d2h) the call copied.
    """
    lib = load()
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    dt = _dtype_code(q)
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype, "cpu")
    for t, n in ((alpha, "alpha"), (theta, "theta"), (beta, "beta"), (S0, "S0"), (S_T, "S_T")):
        _check(t, n, torch.float32, "cpu")
    _check(arena, "arena")
    h2d, d2h = _sz(), _sz()
    rc = lib.sfda_forward_host(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0), _ptr(o),
                               _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v, chunk, dt, _ptr(arena),
                               arena.numel() * arena.element_size(), _stream(stream), ctypes.byref(h2d),
                               ctypes.byref(d2h))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_host")
    return h2d.value, d2h.value


def sfda_forward_host_arena_bytes(B, T, H, d_k, d_v, chunk, dtype, want_o_im, have_S0, want_S_T) -> int:
    return int(load().sfda_forward_host_arena_bytes(B, T, H, d_k, d_v, chunk, dtype, int(want_o_im), int(have_S0),
                                                    int(want_S_T)))


def sfda_frontend(a_raw, b_raw, c_raw, k_raw, alpha_min, alpha_max, theta_max, eps, alpha, theta, beta, k,
                  stream=None):
    """``sfda_frontend`` of ``include/sfda.h``: the stable parameterisation as a kernel of its own."""
    B, T, H, d_k = k_raw.shape
    _check(k_raw, "k_raw")
    _check(k, "k", k_raw.dtype)
    for t, n in ((a_raw, "a_raw"), (b_raw, "b_raw"), (c_raw, "c_raw"), (alpha, "alpha"), (theta, "theta"),
                 (beta, "beta")):
        _check(t, n, torch.float32)
    rc = load().sfda_frontend(_ptr(a_raw), _ptr(b_raw), _ptr(c_raw), _ptr(k_raw), alpha_min, alpha_max, theta_max,
                              eps, _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(k), B, T, H, d_k,
                              _dtype_code(k_raw), _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_frontend")


def sfda_forward_fused_workspace_bytes(B, T, H, d_k, d_v, chunk, dtype) -> int:
    return int(load().sfda_forward_fused_workspace_bytes(B, T, H, d_k, d_v, chunk, dtype))


def sfda_forward_fused(q, k_raw, v, a_raw, b_raw, c_raw, alpha_min, alpha_max, theta_max, eps, S0, o, o_im, S_T,
                       chunk, workspace=None, stream=None):
    """``sfda_forward_fused`` of ``include/sfda.h``: the forward on the raw inputs of the stable parameterisation."""
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k_raw, "k_raw"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((a_raw, "a_raw"), (b_raw, "b_raw"), (c_raw, "c_raw"), (S0, "S0"), (S_T, "S_T")):
        _check(t, n, torch.float32)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().sfda_forward_fused(_ptr(q), _ptr(k_raw), _ptr(v), _ptr(a_raw), _ptr(b_raw), _ptr(c_raw), alpha_min,
                                   alpha_max, theta_max, eps, _ptr(S0), _ptr(o), _ptr(o_im), _ptr(S_T), B, T, H,
                                   d_k, d_v, chunk, _dtype_code(q), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_fused")


def sfda_step_fused(q, k_raw, v, a_raw, b_raw, c_raw, alpha_min, alpha_max, theta_max, eps, S, o, o_im, stream=None):
    """``sfda_step_fused`` of ``include/sfda.h``: one decode step on the raw inputs; S is updated in place."""
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k_raw, "k_raw"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((a_raw, "a_raw"), (b_raw, "b_raw"), (c_raw, "c_raw"), (S, "S")):
        _check(t, n, torch.float32)
    rc = load().sfda_step_fused(_ptr(q), _ptr(k_raw), _ptr(v), _ptr(a_raw), _ptr(b_raw), _ptr(c_raw), alpha_min,
                                alpha_max, theta_max, eps, _ptr(S), _ptr(o), _ptr(o_im), B, H, d_k, d_v,
                                _dtype_code(q), _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_step_fused")


def sfda_backward_workspace_bytes(B, T, H, d_k, d_v, dtype) -> int:
    return int(load().sfda_backward_workspace_bytes(B, T, H, d_k, d_v, dtype))


def sfda_backward(q, k, v, alpha, theta, beta, S0, d_o, d_o_im, dS_T, dq, dk, dv, dalpha, dtheta, dbeta, dS0,
                  workspace, stream=None):
    """``sfda_backward`` of ``include/sfda.h``: gradients of a real loss through the recurrence."""
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (d_o, "d_o"), (d_o_im, "d_o_im"), (dq, "dq"), (dk, "dk"), (dv, "dv")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (beta, "beta"), (S0, "S0"), (dS_T, "dS_T"), (dalpha, "dalpha"),
                 (dtheta, "dtheta"), (dbeta, "dbeta"), (dS0, "dS0")):
        _check(t, n, torch.float32)
    _check(workspace, "workspace")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().sfda_backward(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0), _ptr(d_o),
                              _ptr(d_o_im), _ptr(dS_T), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dalpha), _ptr(dtheta),
                              _ptr(dbeta), _ptr(dS0), B, T, H, d_k, d_v, _dtype_code(q), _ptr(workspace), ws_bytes,
                              _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_backward")


def sfda_forward_two_level_workspace_bytes(B, T, H, d_k, d_v, chunk, dtype, n_slices=0) -> int:
    return int(load().sfda_forward_two_level_workspace_bytes(B, T, H, d_k, d_v, chunk, dtype, n_slices))


def sfda_forward_two_level(q, k, v, alpha, theta, beta, S0, o, o_im, S_T, chunk, n_slices, workspace, stream=None):
    """``sfda_forward_two_level`` of ``include/sfda.h``: the forward as a two-level scan over time slices."""
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (beta, "beta"), (S0, "S0"), (S_T, "S_T")):
        _check(t, n, torch.float32)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().sfda_forward_two_level(_ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta), _ptr(S0),
                                       _ptr(o), _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v, chunk, _dtype_code(q),
                                       int(n_slices), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_two_level")


def sfda_step_decoupled(q, k, r, v, alpha, theta, eta, beta, S, o, o_im, stream=None):
    """``sfda_step_decoupled`` of ``include/sfda.h``: one decode step of the write-decoupled variant."""
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (r, "r"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (eta, "eta"), (beta, "beta"), (S, "S")):
        _check(t, n, torch.float32)
    rc = load().sfda_step_decoupled(_ptr(q), _ptr(k), _ptr(r), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(eta),
                                    _ptr(beta), _ptr(S), _ptr(o), _ptr(o_im), B, H, d_k, d_v, _dtype_code(q),
                                    _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_step_decoupled")


def sfda_forward_decoupled(q, k, r, v, alpha, theta, eta, beta, S0, o, o_im, S_T, stream=None):
    """``sfda_forward_decoupled`` of ``include/sfda.h``: the write-decoupled variant over whole sequences."""
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (r, "r"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (eta, "eta"), (beta, "beta"), (S0, "S0"), (S_T, "S_T")):
        _check(t, n, torch.float32)
    rc = load().sfda_forward_decoupled(_ptr(q), _ptr(k), _ptr(r), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(eta),
                                       _ptr(beta), _ptr(S0), _ptr(o), _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v,
                                       _dtype_code(q), _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_decoupled")


ERASE_COMPLEX, ERASE_REAL = 0, 1


def sfda_step_blocks(q, k, r, v, alpha, theta, flip, eta, beta, S, o, o_im, erase=ERASE_COMPLEX, stream=None):
    """``sfda_step_blocks`` of ``include/sfda.h``: one decode step with 2 x 2 rotation / reflection control blocks
    (``flip``: uint8 [B, H, m] or None) and the complex or the real rank-one erase."""
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (r, "r"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (eta, "eta"), (beta, "beta"), (S, "S")):
        _check(t, n, torch.float32)
    _check(flip, "flip", torch.uint8)
    rc = load().sfda_step_blocks(_ptr(q), _ptr(k), _ptr(r), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(flip), _ptr(eta),
                                 _ptr(beta), _ptr(S), _ptr(o), _ptr(o_im), B, H, d_k, d_v, _dtype_code(q), int(erase),
                                 _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_step_blocks")


def sfda_forward_blocks(q, k, r, v, alpha, theta, flip, eta, beta, S0, o, o_im, S_T, erase=ERASE_COMPLEX, stream=None):
    """``sfda_forward_blocks`` of ``include/sfda.h``: whole sequences with 2 x 2 rotation / reflection control
    blocks (``flip``: uint8 [B, T, H, m] or None) and the complex or the real rank-one erase."""
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    for t, n in ((q, "q"), (k, "k"), (r, "r"), (v, "v"), (o, "o"), (o_im, "o_im")):
        _check(t, n, q.dtype)
    for t, n in ((alpha, "alpha"), (theta, "theta"), (eta, "eta"), (beta, "beta"), (S0, "S0"), (S_T, "S_T")):
        _check(t, n, torch.float32)
    _check(flip, "flip", torch.uint8)
    rc = load().sfda_forward_blocks(_ptr(q), _ptr(k), _ptr(r), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(flip),
                                    _ptr(eta), _ptr(beta), _ptr(S0), _ptr(o), _ptr(o_im), _ptr(S_T), B, T, H, d_k, d_v,
                                    _dtype_code(q), int(erase), _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_forward_blocks")


def sfda_frontend_backward(a_raw, b_raw, c_raw, k_raw, alpha_min, alpha_max, theta_max, eps, dalpha, dtheta, dbeta, dk,
                           da, db, dc, dk_raw, stream=None):
    """``sfda_frontend_backward`` of ``include/sfda.h``: gradients with respect to the raw inputs of the stable
    parameterisation from the gradients with respect to alpha, theta, beta and the normalised key."""
    B, T, H, d_k = k_raw.shape
    _check(k_raw, "k_raw")
    for t, n in ((dk, "dk"), (dk_raw, "dk_raw")):
        _check(t, n, k_raw.dtype)
    for t, n in ((a_raw, "a_raw"), (b_raw, "b_raw"), (c_raw, "c_raw"), (dalpha, "dalpha"), (dtheta, "dtheta"),
                 (dbeta, "dbeta"), (da, "da"), (db, "db"), (dc, "dc")):
        _check(t, n, torch.float32)
    rc = load().sfda_frontend_backward(_ptr(a_raw), _ptr(b_raw), _ptr(c_raw), _ptr(k_raw), alpha_min, alpha_max,
                                       theta_max, eps, _ptr(dalpha), _ptr(dtheta), _ptr(dbeta), _ptr(dk), _ptr(da),
                                       _ptr(db), _ptr(dc), _ptr(dk_raw), B, T, H, d_k, _dtype_code(k_raw),
                                       _stream(stream))
    if rc != 0:
        raise SfdaError(rc, "sfda_frontend_backward")
