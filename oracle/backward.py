"""Reverse-mode derivative of the per-token recurrence (test infrastructure only).

The paper names the backward pass only as something to be timed (App. E, kernel benchmark protocol); what it must
compute is fixed by Eq. "sfda" itself: for a real loss L that depends on the outputs o_t = S_t^* q_t and on the final
state S_T, the gradients of L with respect to every input of

    S_t = (I - beta_t k_t k_t^*) Lambda_t S_{t-1} + beta_t k_t v_t^T,    Lambda_t = diag(alpha_t e^{i theta_t}).

Conventions.  Complex quantities X carry a cotangent Xb with dL = Re sum conj(Xb) dX; for an array stored as
(Re, Im) pairs this is the ordinary gradient with respect to the two real numbers.  Upstream: do_re, do_im
(cotangents of Re and Im of S_t^* q_t) and dS_T in the paired-row layout of the state.

One step, written with Z = Lambda_t S_{t-1}, u^T = v_t^T - k_t^* Z, so that S_t = Z + beta_t k_t u^T, and with
G the cotangent of S_t (including the output term q_t yb_t^*, yb_t = do_re + i do_im):

    qb   = S_t yb                       p   = G^* k                      vb   = beta Re p
    betab = Re(u^T p)                   kb  = beta (G conj(u) - Z p)     Zb   = G - beta k p^*
    lamb_j = sum_c conj(S_{t-1,jc}) Zb_jc       alphab = Re(conj(lamb) e^{i theta})     thetab = -Im(conj(lamb) lam)
    cotangent of S_{t-1}:  conj(lam) Zb (row-wise)

Plain complex128 numpy, one Python iteration per token; states are recomputed from checkpoints every `seg` tokens so
that long sequences fit in memory.  The pins (finite differences of the forward oracle, closed forms) are in
tests/test_oracle_pins.py.
"""
import numpy as np


def _pair(x):
    x = np.asarray(x, dtype=np.float64)
    return x[..., 0::2] + 1j * x[..., 1::2]


def _unpair(z):
    out = np.empty(z.shape[:-1] + (2 * z.shape[-1],), np.float64)
    out[..., 0::2] = z.real
    out[..., 1::2] = z.imag
    return out


def _state_pair(S):      # [N, 2m, dv] paired rows -> complex [N, m, dv]
    S = np.asarray(S, dtype=np.float64)
    return S[:, 0::2, :] + 1j * S[:, 1::2, :]


def _state_unpair(Z):
    out = np.empty((Z.shape[0], 2 * Z.shape[1], Z.shape[2]), np.float64)
    out[:, 0::2, :] = Z.real
    out[:, 1::2, :] = Z.imag
    return out


def _step(S, lam, k, v, beta):
    """S_{t-1} -> (Z, u, S_t) for N sequences: S [N,m,dv], lam, k [N,m], v [N,dv], beta [N]."""
    Z = lam[:, :, None] * S
    u = v - np.einsum("nj,njc->nc", k.conj(), Z)
    return Z, u, Z + beta[:, None, None] * k[:, :, None] * u[:, None, :]


def sfda_backward(q, k, v, alpha, theta, beta, S0, do_re, do_im, dS_T, seg=64):
    """Gradients of L for N independent sequences.

    q, k [N,T,2m] (pairs), v [N,T,dv], alpha, theta [N,T,m], beta [N,T], S0 [N,2m,dv] or None;
    do_re, do_im [N,T,dv] (do_im may be None), dS_T [N,2m,dv] or None.
    Returns dq, dk [N,T,2m], dv [N,T,dv], dalpha, dtheta [N,T,m], dbeta [N,T], dS0 [N,2m,dv], all float64.
    """
    qc, kc = _pair(q), _pair(k)
    v = np.asarray(v, dtype=np.float64)
    alpha = np.asarray(alpha, dtype=np.float64)
    theta = np.asarray(theta, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    N, T, m = qc.shape
    dv_ = v.shape[-1]
    lam = alpha * np.exp(1j * theta)
    yb = np.asarray(do_re, dtype=np.float64) + (0.0 if do_im is None else 1j * np.asarray(do_im, dtype=np.float64))
    S = np.zeros((N, m, dv_), np.complex128) if S0 is None else _state_pair(S0)

    # forward sweep: keep the state at the start of every segment
    starts = list(range(0, T, seg))
    check = []
    for t in range(T):
        if t % seg == 0:
            check.append(S.copy())
        _, _, S = _step(S, lam[:, t], kc[:, t], v[:, t], beta[:, t])

    G = np.zeros((N, m, dv_), np.complex128) if dS_T is None else _state_pair(dS_T)
    dq = np.zeros((N, T, m), np.complex128)
    dk = np.zeros((N, T, m), np.complex128)
    dvv = np.zeros((N, T, dv_))
    dal = np.zeros((N, T, m))
    dth = np.zeros((N, T, m))
    dbe = np.zeros((N, T))
    for si in reversed(range(len(starts))):
        t0, t1 = starts[si], min(starts[si] + seg, T)
        prev = []                                   # S_{t-1} for every token of the segment
        S = check[si]
        for t in range(t0, t1):
            prev.append(S)
            _, _, S = _step(S, lam[:, t], kc[:, t], v[:, t], beta[:, t])
        for t in reversed(range(t0, t1)):
            Sp = prev[t - t0]
            l, kk, b = lam[:, t], kc[:, t], beta[:, t]
            Z, u, St = _step(Sp, l, kk, v[:, t], b)
            G = G + qc[:, t][:, :, None] * yb[:, t].conj()[:, None, :]
            dq[:, t] = np.einsum("njc,nc->nj", St, yb[:, t])
            p = np.einsum("njc,nj->nc", G.conj(), kk)
            dvv[:, t] = b[:, None] * p.real
            dbe[:, t] = np.einsum("nc,nc->n", u, p).real
            dk[:, t] = b[:, None] * (np.einsum("njc,nc->nj", G, u.conj()) - np.einsum("njc,nc->nj", Z, p))
            Zb = G - b[:, None, None] * kk[:, :, None] * p.conj()[:, None, :]
            lamb = np.einsum("njc,njc->nj", Sp.conj(), Zb)
            dal[:, t] = (lamb.conj() * np.exp(1j * theta[:, t])).real
            dth[:, t] = -(lamb.conj() * l).imag
            G = l.conj()[:, :, None] * Zb
    return _unpair(dq), _unpair(dk), dvv, dal, dth, dbe, _state_unpair(G)
