"""The reverse-mode derivative of the recurrence in chunk form (test infrastructure only).

`oracle/backward.py` is the definition (the adjoint of Eq. "sfda", token by token).  This module reaches the same
gradients chunk by chunk with the matrices of the constructive chunk-WY form (Theorem "constructive chunk-WY" and
the corollary "chunk output formula"): it is the statement, checked in tests/test_oracle_pins.py against the
token-level adjoint, of what a chunked backward pass computes -- every step is a product with a C x C, m x C or
m x d_v matrix of the chunk.  It needs alpha > 0 (it divides by the cumulative decay, as the forward chunk form does).

One chunk of C tokens, complex notation, gamma_t = prod_{s <= t} lambda_s:

  forward   W_t = conj(gamma_t) k_t,  Qt_t = conj(gamma_t) q_t,  Kc_t = k_t / gamma_t          (rows of C x m matrices)
            Kt = stril(conj(W) Kc^T),  Aq = tril(conj(Qt) Kc^T)                               (C x C)
            U  = (I + Kt D_beta)^{-1} (V - conj(W) S_0),  E = D_beta U      (rows u_t^T = v_t^T - k_t^* Lambda_t S_{t-1})
            S_C = gamma_C . (S_0 + Kc^T E)
  backward  with G_C the cotangent of S_C, Gt = conj(gamma_C) . G_C, rows Yc_t = yb_t^* of the output cotangents:
            Pc = (I + Kt^H D_beta)^{-1} (conj(Kc) Gt + Aq^H Yc)        (rows p_t^* = k_t^* Ghat_t; an upper-triangular solve)
            G_0 = Gt + Qt^T Yc - W^T D_beta Pc                          (the cotangent of S_0)
  with X_t = S_0 + sum_{i<t} Kc_i e_i^T (so S_{t-1} = gamma_{t-1} . X_t) and
       Xi_t = Gt + sum_{i>=t} Qt_i Yc_i - sum_{i>t} W_i beta_i Pc_i (so Ghat_t = Xi_t / conj(gamma_t)):
            dv_t = beta_t Re p_t,   dbeta_t = Re(u_t^T p_t),   dq_t = gamma_t . (X_{t+1} yb_t),
            dk_t = beta_t (Xi_t conj(u_t) / conj(gamma_t) - gamma_t . (X_t p_t)),
            D_t  = rowdot(S_{t-1}, G_{t-1}) = D_{t+1} + Qt_t . conj(X_t yb_t) - beta_t W_t . conj(X_t p_t)
                                                      - beta_t conj(Kc_t) . (Xi'_{t+1} conj(u_t)),
            D_{C+1} = rowdot(S_C, G_C),   dalpha_t = Re D_t / alpha_t,   dtheta_t = Im D_t.
  The vectors X_t yb_t, X_t p_t, Xi_t conj(u_t) of all tokens are S_0 Yb^T, S_0 P^T, Gt conj(U)^T corrected by
  Kc^T, Qt^T, W^T times triangular parts of the C x C products E Yb^T and E P^T.
"""
import numpy as np

from .backward import _pair, _state_pair, _state_unpair, _unpair


def _chunk_forward(S0, lam, k, v, beta):
    """Chunk matrices and the final state: returns (gam, W, Kc, Kt, U, E, S_C)."""
    C = lam.shape[0]
    gam = np.cumprod(lam, axis=0)
    W = gam.conj() * k
    Kc = k / gam
    Kt = np.tril(W.conj() @ Kc.T, -1)
    R = v - W.conj() @ S0
    U = np.linalg.solve(np.eye(C) + Kt * beta[None, :], R)
    E = beta[:, None] * U
    S_C = gam[-1][:, None] * (S0 + Kc.T @ E)
    return gam, W, Kc, Kt, U, E, S_C


def _chunk_backward(S0, S_C, G_C, lam, alpha, q, k, beta, yb, fwd):
    gam, W, Kc, Kt, U, E, _ = fwd
    C = lam.shape[0]
    Qt = gam.conj() * q
    Aq = np.tril(Qt.conj() @ Kc.T)
    Gt = gam[-1].conj()[:, None] * G_C
    Yc = yb.conj()
    Pc = np.linalg.solve(np.eye(C) + Kt.conj().T * beta[None, :], Kc.conj() @ Gt + Aq.conj().T @ Yc)
    P = Pc.conj()                                           # rows p_t
    G_0 = Gt + Qt.T @ Yc - W.T @ (beta[:, None] * Pc)

    dv = beta[:, None] * P.real
    dbeta = np.einsum("tc,tc->t", U, P).real
    # C x C couplings (index [i, t]) and the m x C products with the boundary matrices
    B1 = E @ yb.T                                           # e_i . yb_t
    B2 = E @ P.T                                            # e_i . p_t
    B3 = Yc @ U.conj().T                                    # yb_i^* conj(u_t)
    B4 = (beta[:, None] * Pc) @ U.conj().T                  # beta_i p_i^* conj(u_t)
    XY = S0 @ yb.T + Kc.T @ np.triu(B1, 1)                  # column t: X_t yb_t
    XP = S0 @ P.T + Kc.T @ np.triu(B2, 1)                   # column t: X_t p_t
    XiU = Gt @ U.conj().T + Qt.T @ np.tril(B3, -1) - W.T @ np.tril(B4, -1)     # column t: Xi'_{t+1} conj(u_t)
    dq = gam * (XY.T + Kc * np.diag(B1)[:, None])           # gamma_t . X_{t+1} yb_t
    dk = beta[:, None] * ((XiU.T + Qt * np.diag(B3)[:, None]) / gam.conj() - gam * XP.T)
    delta = Qt * XY.T.conj() - beta[:, None] * W * XP.T.conj() - beta[:, None] * Kc.conj() * XiU.T
    D_end = np.einsum("jc,jc->j", S_C.conj(), G_C)
    D = D_end[None, :] + np.cumsum(delta[::-1], axis=0)[::-1]
    return dq, dk, dv, D.real / alpha, D.imag, dbeta, G_0


def sfda_backward_chunked(q, k, v, alpha, theta, beta, S0, do_re, do_im, dS_T, chunk):
    """Same arguments and results as oracle.backward.sfda_backward, plus the chunk size (T a multiple of it)."""
    qc, kc = _pair(q), _pair(k)
    v = np.asarray(v, dtype=np.float64)
    alpha = np.asarray(alpha, dtype=np.float64)
    theta = np.asarray(theta, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    N, T, m = qc.shape
    dv_ = v.shape[-1]
    assert T % chunk == 0
    lam = alpha * np.exp(1j * theta)
    yb = np.asarray(do_re, dtype=np.float64) + (0.0 if do_im is None else 1j * np.asarray(do_im, dtype=np.float64))
    S_all = np.zeros((N, m, dv_), np.complex128) if S0 is None else _state_pair(S0)
    G_all = np.zeros((N, m, dv_), np.complex128) if dS_T is None else _state_pair(dS_T)
    out = [np.zeros((N, T, m), np.complex128), np.zeros((N, T, m), np.complex128), np.zeros((N, T, dv_)),
           np.zeros((N, T, m)), np.zeros((N, T, m)), np.zeros((N, T))]
    G_out = np.zeros_like(G_all)
    for n in range(N):
        starts, fwds, S = [], [], S_all[n]
        for t0 in range(0, T, chunk):                      # forward: the state at the start of every chunk
            sl = slice(t0, t0 + chunk)
            fwd = _chunk_forward(S, lam[n, sl], kc[n, sl], v[n, sl], beta[n, sl])
            starts.append(S)
            fwds.append(fwd)
            S = fwd[-1]
        G = G_all[n]
        for ci in reversed(range(len(starts))):            # backward: the cotangent from the last chunk to the first
            sl = slice(ci * chunk, (ci + 1) * chunk)
            res = _chunk_backward(starts[ci], fwds[ci][-1], G, lam[n, sl], alpha[n, sl], qc[n, sl], kc[n, sl],
                                  beta[n, sl], yb[n, sl], fwds[ci])
            for dst, val in zip(out, res[:6]):
                dst[n, sl] = val
            G = res[6]
        G_out[n] = G
    return _unpair(out[0]), _unpair(out[1]), out[2], out[3], out[4], out[5], _state_unpair(G_out)
