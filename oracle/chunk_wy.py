"""Naive chunked SFDA path in numpy complex128 (test infrastructure only).

It takes the steps of the paper in the paper's order and notation, one token at
a time, with no blocking or fusion (written from the theorems' equations):

* Algorithm 1 ("Constructive SFDA-WY chunk summary") / Theorem "Constructive
  left-to-right chunk-WY recursion": the factors (Gamma, Y, W, M) of
  ``P_t = A_t ... A_1 = Gamma_t - Y_t M_t W_t^*``;
* the zero-state recurrence of Theorem "Exact affine chunk transfer" for the
  write summary ``B_t^chunk``;
* Eq. "apply-transfer": ``S_out = Gamma S_in - Y (M (W^* S_in)) + B``;
* Theorem "Prefix outputs inside a chunk": ``o_r = S_r^* q_r`` with
  ``S_r = P_r S_0 + B_r^chunk``;
* the boundary-state scan: the state after a chunk enters the next chunk.

It shares no code with ``sfda_recurrence.c``; the two are compared in the pins.
Complex vectors are given here already paired: ``x_c[j] = x[2j] + 1j*x[2j+1]``.
"""
import numpy as np


def pair(x):
    """[..., 2m] real pairs -> [..., m] complex (channel 2j = Re, 2j+1 = Im)."""
    x = np.asarray(x, dtype=np.float64)
    return x[..., 0::2] + 1j * x[..., 1::2]


def unpair_rows(S):
    """[m, dv] complex -> [2m, dv] real with row 2j = Re, row 2j+1 = Im."""
    out = np.empty((2 * S.shape[0], S.shape[1]), np.float64)
    out[0::2] = S.real
    out[1::2] = S.imag
    return out


def pair_rows(S):
    """[2m, dv] real paired rows -> [m, dv] complex."""
    S = np.asarray(S, dtype=np.float64)
    return S[0::2] + 1j * S[1::2]


def chunk_factor_steps(k, alpha, theta, beta):
    """Factors of P_t = A_t ... A_1 = Gamma_t - Y_t M_t W_t^* for t = 1..C, from the four equations of Theorem
    "Constructive left-to-right chunk-WY recursion" (u_t = beta_t k_t, r_t = Lambda_t^* k_t):

      Gamma_t = Lambda_t Gamma_{t-1}                         Eq. "constructive-Gamma"
      Y_t     = [Lambda_t Y_{t-1} | u_t]                     Eq. "constructive-Y"
      W_t     = [W_{t-1} | Gamma_{t-1}^* r_t]                Eq. "constructive-W"
      M_t     = [[M_{t-1}, 0], [-r_t^* Y_{t-1} M_{t-1}, 1]]  Eq. "constructive-M"

    k: [C, m] complex; alpha, theta: [C, m]; beta: [C].  Yields (Gamma_t [m], Y_t [m, t], W_t [m, t], M_t [t, t])
    after every token.  The factors live in arrays of the chunk's full size that grow by one column (and one row of
    M) per token; W_t and M_t are leading blocks of the final ones, Y_t is not (its old columns are multiplied by
    Lambda_t every step), so what is yielded are copies of the current leading blocks.
    """
    k = np.asarray(k, dtype=np.complex128)
    C, m = k.shape
    lam = np.asarray(alpha, np.float64) * np.exp(1j * np.asarray(theta, np.float64))     # diagonal of Lambda_t, [C, m]
    u_all = np.asarray(beta, np.float64)[:, None] * k                                   # rows u_t
    r_all = np.conj(lam) * k                                                            # rows r_t
    gamma = np.cumprod(lam, axis=0)                                                     # rows diag(Gamma_t)
    Y = np.zeros((m, C), np.complex128)
    W = np.zeros((m, C), np.complex128)
    M = np.eye(C, dtype=np.complex128)
    for t in range(C):
        if t > 0:
            # row t of M first: it needs Y_{t-1} and M_{t-1}, both still untouched by this step
            M[t, :t] = -(np.conj(r_all[t]) @ Y[:, :t]) @ M[:t, :t]
            Y[:, :t] *= lam[t][:, None]
            W[:, t] = np.conj(gamma[t - 1]) * r_all[t]
        else:
            W[:, 0] = r_all[0]                            # Gamma_0 = I
        Y[:, t] = u_all[t]
        n = t + 1
        yield gamma[t].copy(), Y[:, :n].copy(), W[:, :n].copy(), M[:n, :n].copy()


def chunk_factors(k, alpha, theta, beta):
    """(Gamma_C, Y_C, W_C, M_C) of one chunk (the last step of the recursion)."""
    out = None
    for out in chunk_factor_steps(k, alpha, theta, beta):
        pass
    return out


def forward_chunked(q, k, v, alpha, theta, beta, S0, chunk):
    """Chunked forward of ONE sequence.

    q, k: [T, 2m] real pairs; v: [T, dv]; alpha, theta: [T, m]; beta: [T];
    S0: [2m, dv] paired rows or None.  Returns (o_re [T,dv], o_im [T,dv],
    S_T [2m,dv]).  A short last chunk is simply a shorter chunk.
    """
    qc, kc = pair(q), pair(k)
    v = np.asarray(v, dtype=np.float64)
    alpha = np.asarray(alpha, dtype=np.float64)
    theta = np.asarray(theta, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    T, m = kc.shape
    dv = v.shape[1]
    S_in = np.zeros((m, dv), np.complex128) if S0 is None else pair_rows(S0)
    o = np.zeros((T, dv), np.complex128)
    for start in range(0, T, chunk):
        stop = min(start + chunk, T)
        sl = slice(start, stop)
        Sbar = np.zeros((m, dv), np.complex128)          # zero-state recurrence
        steps = chunk_factor_steps(kc[sl], alpha[sl], theta[sl], beta[sl])
        S_r = S_in
        for i, (Gamma, Y, W, M) in enumerate(steps):
            t = start + i
            lam = alpha[t] * np.exp(1j * theta[t])
            u = beta[t] * kc[t]
            r = np.conj(lam) * kc[t]
            # Sbar_t = A_t Sbar_{t-1} + B_t with A_t = Lambda_t - u_t r_t^*, B_t = beta_t k_t v_t^*
            Sbar = lam[:, None] * Sbar - u[:, None] * (np.conj(r)[None, :] @ Sbar) \
                + beta[t] * kc[t][:, None] * v[t][None, :]
            # S_r = Gamma_r S_0 - Y_r (M_r (W_r^* S_0)) + B_r^chunk
            S_r = Gamma[:, None] * S_in - Y @ (M @ (W.conj().T @ S_in)) + Sbar
            o[t] = S_r.conj().T @ qc[t]                  # o_r = S_r^* q_r
        S_in = S_r                                       # boundary-state scan
    return o.real.copy(), o.imag.copy(), unpair_rows(S_in)
