"""The write-decoupled variant of the recurrence (test infrastructure only).

Section 3, paragraph "Write-decoupled variant" (Eq. "sfda-decoupled-main"): the erase direction and strength
(k_t, eta_t) are separated from the write direction and strength (r_t, beta_t),

    S_t = (I - eta_t k_t k_t^*) Lambda_t S_{t-1} + beta_t r_t v_t^*,        o_t = S_t^* q_t,

and the tied model is r_t = k_t, eta_t = beta_t.  Plain complex128 numpy, one Python iteration per token, same
layouts as the tied oracle (q, k, r as (Re, Im) pairs, S with paired rows, v real).
"""
import numpy as np


def sfda_decoupled_recurrence(q, k, r, v, alpha, theta, eta, beta, S0=None):
    """q, k, r [N,T,2m]; v [N,T,dv]; alpha, theta [N,T,m]; eta, beta [N,T]; S0 [N,2m,dv] or None.
    Returns (o_re, o_im, S_T) as float64, o read from the state after token t's update."""
    q, k, r = (np.asarray(x, dtype=np.float64) for x in (q, k, r))
    qc, kc, rc = (x[..., 0::2] + 1j * x[..., 1::2] for x in (q, k, r))
    v = np.asarray(v, dtype=np.float64)
    lam = np.asarray(alpha, dtype=np.float64) * np.exp(1j * np.asarray(theta, dtype=np.float64))
    eta = np.asarray(eta, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    N, T, m = qc.shape
    dv = v.shape[-1]
    S = np.zeros((N, m, dv), np.complex128)
    if S0 is not None:
        S0 = np.asarray(S0, dtype=np.float64)
        S = S0[:, 0::2] + 1j * S0[:, 1::2]
    o = np.empty((N, T, dv), np.complex128)
    for t in range(T):
        Z = lam[:, t][:, :, None] * S                                           # Lambda_t S_{t-1}
        c = np.einsum("nj,njc->nc", kc[:, t].conj(), Z)                         # k_t^* Z
        S = Z - eta[:, t][:, None, None] * kc[:, t][:, :, None] * c[:, None, :] \
            + beta[:, t][:, None, None] * rc[:, t][:, :, None] * v[:, t][:, None, :]
        o[:, t] = np.einsum("njc,nj->nc", S.conj(), qc[:, t])                   # S_t^* q_t
    S_T = np.empty((N, 2 * m, dv))
    S_T[:, 0::2], S_T[:, 1::2] = S.real, S.imag
    return o.real, o.imag, S_T
