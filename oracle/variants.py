"""Variants of the recurrence (test infrastructure only): the write-decoupled one in complex arithmetic, and the
real-coordinate model with aligned 2 x 2 orthogonal control blocks (rotations and reflections) and a choice of
erase term.

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


def sfda_block_control_recurrence(q, k, r, v, alpha, theta, flip, eta, beta, S0=None, real_erase=False):
    """The layer in real coordinates (Eq. "intro-sfda-real"), written with explicit real matrices:

        S_t = (I - eta_t P_t) U_t D_t S_{t-1} + beta_t r_t v_t^T,      S_t in R^{2m x d_v},

    where U_t D_t is a direct sum of 2 x 2 blocks alpha_j R(theta_j) F^{flip_j}, R a planar rotation and
    F = diag(1, -1) the reflection (Theorem "Dihedral phase-orientation memory" and the remark after it: aligned
    2 x 2 orthogonal blocks; flip = 0 everywhere is the complex-diagonal family of Lemma "Real-to-complex phase
    equivalence").  The erase projector P_t is either the realification of the complex rank-one k k^*, i.e. the
    real rank-two k k^T + (Jk)(Jk)^T with J(x, y) = (-y, x) per pair (real_erase=False: the model of Eq.
    "sfda-decoupled-main"), or the real rank-one k k^T on R^{2m} that Eq. "intro-sfda-real" writes
    (real_erase=True).  Outputs: o_re = S_t^T q_t and o_im = -S_t^T (J q_t), which are Re and Im of S_t^* q_t under
    the identification of a row pair with a complex row.

    q, k, r [N,T,2m]; v [N,T,dv]; alpha, theta [N,T,m]; flip [N,T,m] (0/1) or None; eta, beta [N,T];
    S0 [N,2m,dv] or None.  float64, dense 2m x 2m matrices, one Python iteration per token and sequence.
    """
    q, k, r, v = (np.asarray(x, dtype=np.float64) for x in (q, k, r, v))
    alpha, theta = np.asarray(alpha, dtype=np.float64), np.asarray(theta, dtype=np.float64)
    eta, beta = np.asarray(eta, dtype=np.float64), np.asarray(beta, dtype=np.float64)
    N, T, d = q.shape
    m, dv = d // 2, v.shape[-1]
    flip = np.zeros((N, T, m), np.int64) if flip is None else np.asarray(flip).astype(np.int64)

    def J(x):
        y = np.empty_like(x)
        y[0::2], y[1::2] = -x[1::2], x[0::2]
        return y

    o_re, o_im = np.empty((N, T, dv)), np.empty((N, T, dv))
    S_T = np.empty((N, d, dv))
    for n in range(N):
        S = np.zeros((d, dv)) if S0 is None else np.array(S0[n], dtype=np.float64)
        for t in range(T):
            A = np.zeros((d, d))
            for j in range(m):
                c, s_ = np.cos(theta[n, t, j]), np.sin(theta[n, t, j])
                R = np.array([[c, -s_], [s_, c]])
                F = np.diag([1.0, -1.0]) if flip[n, t, j] else np.eye(2)
                A[2 * j:2 * j + 2, 2 * j:2 * j + 2] = alpha[n, t, j] * (R @ F)
            kk = k[n, t]
            P = np.outer(kk, kk)
            if not real_erase:
                P = P + np.outer(J(kk), J(kk))
            S = (np.eye(d) - eta[n, t] * P) @ (A @ S) + beta[n, t] * np.outer(r[n, t], v[n, t])
            o_re[n, t] = S.T @ q[n, t]
            o_im[n, t] = -S.T @ J(q[n, t])
        S_T[n] = S
    return o_re, o_im, S_T
