"""ctypes front end of ``sfda_recurrence.c`` (test infrastructure only).

The arithmetic is all in the C file; this module only marshals numpy arrays.
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.oracle_sfda_recurrence.argtypes = [dp] * 10 + [
            ctypes.c_long, ctypes.c_long, ctypes.c_int, ctypes.c_int]
        lib.oracle_sfda_recurrence.restype = ctypes.c_int
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the C loop spreads whole sequences over."""
    return int(_load().oracle_num_threads())


def _as(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float64)
    if a.shape != tuple(shape):
        raise ValueError("expected shape %s, got %s" % (tuple(shape), a.shape))
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None \
        else ctypes.POINTER(ctypes.c_double)()


def sfda_recurrence(q, k, v, alpha, theta, beta, S0=None):
    """Run the per-token recurrence of Eq. "sfda" on N independent sequences.

    q, k: [N,T,2m] (pairs Re,Im); v: [N,T,dv]; alpha, theta: [N,T,m];
    beta: [N,T]; S0: [N,2m,dv] or None (zero).  All are converted to float64.
    Returns ``(o_re, o_im, S_T)`` as float64 arrays, ``o = S_t^* q_t`` read from
    the state *after* token t's update, ``S_T`` in the paired-row layout of S0.
    """
    q = np.asarray(q)
    N, T, dk = q.shape
    if dk % 2:
        raise ValueError("key width must be even")
    m = dk // 2
    dv = np.asarray(v).shape[-1]
    q = _as(q, (N, T, dk))
    k = _as(k, (N, T, dk))
    v = _as(v, (N, T, dv))
    alpha = _as(alpha, (N, T, m))
    theta = _as(theta, (N, T, m))
    beta = _as(beta, (N, T))
    S0 = None if S0 is None else _as(S0, (N, dk, dv))
    o_re = np.empty((N, T, dv), np.float64)
    o_im = np.empty((N, T, dv), np.float64)
    S_T = np.empty((N, dk, dv), np.float64)
    rc = _load().oracle_sfda_recurrence(
        _ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(theta), _ptr(beta),
        _ptr(S0), _ptr(o_re), _ptr(o_im), _ptr(S_T), N, T, m, dv)
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return o_re, o_im, S_T
