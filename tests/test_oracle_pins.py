"""Pins for the CPU oracle: every check compares ``oracle/`` with something that
does not come from it -- dense brute force written here, closed forms, special
cases that reduce to separately written textbook loops, invariants the paper
proves.  A dropped term, a wrong sign or index, a missing conjugate or a
transposed operand in the oracle fails at least one of them.
"""
import os

import numpy as np
import pytest

from oracle import backward, backward_chunk, bookkeeping, chunk_wy, frontend, recurrence

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------
# helpers written independently of oracle/ (dense matrices, no structure used)
# ----------------------------------------------------------------------------
def rand_inputs(seed, N, T, m, dv, alpha_lo=0.5, s0=True, unit_k=True):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((N, T, 2 * m))
    k = rng.standard_normal((N, T, 2 * m))
    if unit_k:
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.standard_normal((N, T, dv))
    alpha = rng.uniform(alpha_lo, 1.0, (N, T, m))
    theta = rng.uniform(-np.pi, np.pi, (N, T, m))
    beta = rng.uniform(0.0, 1.0, (N, T))
    S0 = rng.standard_normal((N, 2 * m, dv)) if s0 else None
    return q, k, v, alpha, theta, beta, S0


def cplx(x):
    return x[..., 0::2] + 1j * x[..., 1::2]


def dense_A(kc, alpha, theta, beta):
    """A_t = (I - beta k k^H) diag(alpha e^{i theta}) as a dense m x m matrix (Eq. AtBt)."""
    m = kc.shape[0]
    Lam = np.diag(alpha * np.exp(1j * theta))
    return (np.eye(m) - beta * np.outer(kc, kc.conj())) @ Lam


def dense_forward(q, k, v, alpha, theta, beta, S0):
    """One sequence, dense matrices only.  Returns o [T,dv] complex, all states, all A_t."""
    T = q.shape[0]
    qc, kc = cplx(q), cplx(k)
    S = np.zeros((kc.shape[1], v.shape[1]), complex) if S0 is None else S0[0::2] + 1j * S0[1::2]
    o, states, As = [], [], []
    for t in range(T):
        A = dense_A(kc[t], alpha[t], theta[t], beta[t])
        B = beta[t] * np.outer(kc[t], v[t])            # beta k v^* with v real
        S = A @ S + B
        o.append(S.conj().T @ qc[t])
        states.append(S)
        As.append(A)
    return np.array(o), states, As


def run_rec(q, k, v, alpha, theta, beta, S0):
    return recurrence.sfda_recurrence(q, k, v, alpha, theta, beta, S0)


# ----------------------------------------------------------------------------
# P1: dense brute force (Theorem "Constructive left-to-right chunk-WY recursion")
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("seed,m,dv,T", [(1, 3, 2, 12), (2, 8, 5, 32), (3, 1, 1, 7)])
def test_both_oracles_match_dense_brute_force(seed, m, dv, T):
    q, k, v, al, th, be, S0 = rand_inputs(seed, 2, T, m, dv)
    o_re, o_im, ST = run_rec(q, k, v, al, th, be, S0)
    for n in range(2):
        o, states, _ = dense_forward(q[n], k[n], v[n], al[n], th[n], be[n], S0[n])
        assert np.abs(o_re[n] - o.real).max() < 1e-12
        assert np.abs(o_im[n] - o.imag).max() < 1e-12
        assert np.abs(ST[n][0::2] - states[-1].real).max() < 1e-12
        assert np.abs(ST[n][1::2] - states[-1].imag).max() < 1e-12
        for C in (4, 5, T):
            a, b, c = chunk_wy.forward_chunked(q[n], k[n], v[n], al[n], th[n], be[n], S0[n], C)
            assert np.abs(a - o.real).max() < 1e-12
            assert np.abs(b - o.imag).max() < 1e-12
            assert np.abs(c[0::2] - states[-1].real).max() < 1e-12
            assert np.abs(c[1::2] - states[-1].imag).max() < 1e-12


@pytest.mark.parametrize("seed,m,C", [(4, 4, 9), (5, 8, 16), (6, 2, 6)])
def test_prefix_products_equal_factor_form(seed, m, C):
    """P_t = A_t ... A_1 = Gamma_t - Y_t M_t W_t^* for every t (Eq. constructive-invariant)."""
    _, k, _, al, th, be, _ = rand_inputs(seed, 1, C, m, 1)
    kc = cplx(k[0])
    P = np.eye(m, dtype=complex)
    worst = 0.0
    for t, (G, Y, W, M) in enumerate(chunk_wy.chunk_factor_steps(kc, al[0], th[0], be[0])):
        P = dense_A(kc[t], al[0, t], th[0, t], be[0, t]) @ P
        F = np.diag(G) - Y @ M @ W.conj().T
        worst = max(worst, np.abs(P - F).max())
        assert Y.shape == (m, t + 1) and W.shape == (m, t + 1) and M.shape == (t + 1, t + 1)
        assert np.allclose(np.triu(M, 1), 0) and np.allclose(np.diag(M), 1)
    assert worst < 1e-13          # the paper prints 1.9e-15 for this identity (Table 8)


def test_single_step_diag_plus_rank_one():
    """A_t = Lambda_t - u_t w_t^*, u = beta k, w = Lambda^* k (Eq. single-step-wy)."""
    _, k, _, al, th, be, _ = rand_inputs(7, 1, 1, 5, 1)
    kc = cplx(k[0, 0])
    lam = al[0, 0] * np.exp(1j * th[0, 0])
    A = dense_A(kc, al[0, 0], th[0, 0], be[0, 0])
    G, Y, W, M = chunk_wy.chunk_factors(kc[None], al[0], th[0], be[0])
    assert np.allclose(Y[:, 0], be[0, 0] * kc)
    assert np.allclose(W[:, 0], np.conj(lam) * kc)
    assert np.allclose(A, np.diag(lam) - np.outer(Y[:, 0], W[:, 0].conj()))


# ----------------------------------------------------------------------------
# P2: theta = 0 reduces to KDA (Prop. "KDA is a special case")
# ----------------------------------------------------------------------------
def real_kda(q, k, v, alpha, beta, S0):
    """Textbook real KDA of dimension m: S = (I - b k k^T) diag(a) S + b k v^T; o = S^T q."""
    T, m = k.shape
    S = S0.copy()
    o = np.zeros((T, v.shape[1]))
    for t in range(T):
        S = alpha[t][:, None] * S
        S = S - beta[t] * np.outer(k[t], k[t] @ S) + beta[t] * np.outer(k[t], v[t])
        o[t] = S.T @ q[t]
    return o, S


def test_theta_zero_real_channels_is_real_kda():
    N, T, m, dv = 2, 50, 6, 4
    q, k, v, al, th, be, S0 = rand_inputs(11, N, T, m, dv)
    th[:] = 0.0
    q[..., 1::2] = 0.0
    k[..., 1::2] = 0.0
    S0[:, 1::2] = 0.0
    o_re, o_im, ST = run_rec(q, k, v, al, th, be, S0)
    for n in range(N):
        o, S = real_kda(q[n][:, 0::2], k[n][:, 0::2], v[n], al[n], be[n], S0[n][0::2])
        assert np.abs(o_re[n] - o).max() < 1e-13
        assert np.abs(o_im[n]).max() == 0.0
        assert np.abs(ST[n][0::2] - S).max() < 1e-13
        assert np.abs(ST[n][1::2]).max() == 0.0
        a, b, c = chunk_wy.forward_chunked(q[n], k[n], v[n], al[n], th[n], be[n], S0[n], 16)
        assert np.abs(a - o).max() < 1e-12 and np.abs(b).max() < 1e-13
        assert np.abs(c[0::2] - S).max() < 1e-12


def test_theta_zero_general_is_complex_kda():
    T, m, dv = 30, 5, 3
    q, k, v, al, th, be, S0 = rand_inputs(12, 1, T, m, dv)
    th[:] = 0.0
    o_re, o_im, ST = run_rec(q, k, v, al, th, be, S0)
    qc, kc = cplx(q[0]), cplx(k[0])
    S = S0[0][0::2] + 1j * S0[0][1::2]
    for t in range(T):
        S = (np.eye(m) - be[0, t] * np.outer(kc[t], kc[t].conj())) @ np.diag(al[0, t]) @ S \
            + be[0, t] * np.outer(kc[t], v[0, t])
        o = S.conj().T @ qc[t]
        assert np.abs(o_re[0, t] - o.real).max() < 1e-13
        assert np.abs(o_im[0, t] - o.imag).max() < 1e-13


# ----------------------------------------------------------------------------
# P3/P4: beta = 0 gives pure diagonal phase-decay (Prop. "Interpolation ...")
# ----------------------------------------------------------------------------
def test_beta_zero_closed_form():
    N, T, m, dv = 1, 64, 4, 3
    q, k, v, al, th, be, S0 = rand_inputs(13, N, T, m, dv)
    be[:] = 0.0
    o_re, o_im, ST = run_rec(q, k, v, al, th, be, S0)
    gam = np.cumprod(al[0] * np.exp(1j * th[0]), axis=0)        # global cumulative product
    S0c = S0[0][0::2] + 1j * S0[0][1::2]
    qc = cplx(q[0])
    for t in range(T):
        o = S0c.conj().T @ (np.conj(gam[t]) * qc[t])
        assert np.abs(o_re[0, t] - o.real).max() < 1e-12
        assert np.abs(o_im[0, t] - o.imag).max() < 1e-12
    S_T = gam[-1][:, None] * S0c
    assert np.abs(ST[0][0::2] - S_T.real).max() < 1e-12
    assert np.abs(ST[0][1::2] - S_T.imag).max() < 1e-12
    a, b, c = chunk_wy.forward_chunked(q[0], k[0], v[0], al[0], th[0], be[0], S0[0], 16)
    assert np.abs(c[0::2] - S_T.real).max() < 1e-12 and np.abs(c[1::2] - S_T.imag).max() < 1e-12


def test_unit_decay_no_write_preserves_row_norms():
    """alpha = 1, beta = 0: |z_t| = |z_0| (Prop. "Bounded cyclic phase memory")."""
    N, T, m, dv = 1, 4096, 3, 2
    q, k, v, al, th, be, S0 = rand_inputs(14, N, T, m, dv)
    al[:] = 1.0
    be[:] = 0.0
    _, _, ST = run_rec(q, k, v, al, th, be, S0)
    n0 = np.hypot(S0[0][0::2], S0[0][1::2])
    nT = np.hypot(ST[0][0::2], ST[0][1::2])
    assert np.abs(nT - n0).max() < 1e-12          # the paper prints 3.0e-14 drift at T = 16384


# ----------------------------------------------------------------------------
# P5: quantised phases 2 pi a / p (Prop. "Bounded cyclic phase memory")
# ----------------------------------------------------------------------------
def test_constant_quantised_phase_returns_after_p_steps():
    m, dv = 4, 2
    p = np.array([2, 3, 5, 7])
    a = np.array([1, 2, 3, 4])
    lcm = 210
    T = 2 * lcm
    rng = np.random.default_rng(15)
    q = rng.standard_normal((1, T, 2 * m))
    k = rng.standard_normal((1, T, 2 * m))
    v = rng.standard_normal((1, T, dv))
    S0 = rng.standard_normal((1, 2 * m, dv))
    al = np.ones((1, T, m))
    th = np.broadcast_to(2 * np.pi * a / p, (1, T, m)).copy()
    be = np.zeros((1, T))
    for Tcut in (lcm, 2 * lcm):
        _, _, ST = run_rec(q[:, :Tcut], k[:, :Tcut], v[:, :Tcut], al[:, :Tcut], th[:, :Tcut], be[:, :Tcut], S0)
        assert np.abs(ST - S0).max() < 1e-11
    # after p_j steps coordinate j alone is back
    for j in range(m):
        _, _, ST = run_rec(q[:, :p[j]], k[:, :p[j]], v[:, :p[j]], al[:, :p[j]], th[:, :p[j]], be[:, :p[j]], S0)
        assert np.abs(ST[0, 2 * j:2 * j + 2] - S0[0, 2 * j:2 * j + 2]).max() < 1e-13


def test_mod5_counter_fixture():
    """z_t = exp(2 pi i (sum a_s mod 5) / 5) z_0: the symbols and residues of the
    fixture were written by hand from the closed form of Prop. "Bounded cyclic
    phase memory"; nothing in it comes from the oracle."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "mod5_counter.txt")) if l.strip() and l[0] != "#"]
    a = np.array([int(r[0]) for r in rows])
    resid = np.array([int(r[1]) for r in rows])
    T = len(a)
    q = np.zeros((1, T, 2))
    q[..., 0] = 1.0                                   # q = 1 reads conj(z_t)
    k = np.zeros((1, T, 2))
    v = np.zeros((1, T, 1))
    al = np.ones((1, T, 1))
    th = (2 * np.pi * a / 5).reshape(1, T, 1)
    be = np.zeros((1, T))
    S0 = np.array([[[1.0], [0.0]]])                   # z_0 = 1
    o_re, o_im, ST = run_rec(q, k, v, al, th, be, S0)
    z = o_re[0, :, 0] - 1j * o_im[0, :, 0]            # o = conj(z) * 1
    want = np.exp(2j * np.pi * resid / 5)
    assert np.abs(z - want).max() < 1e-13
    a2, b2, _ = chunk_wy.forward_chunked(q[0], k[0], v[0], al[0], th[0], be[0], S0[0], 4)
    assert np.abs((a2[:, 0] - 1j * b2[:, 0]) - want).max() < 1e-13


def test_random_quantised_phase_tracks_integer_sum():
    T, m, dv = 500, 4, 1
    p = np.array([2, 3, 5, 7])
    rng = np.random.default_rng(16)
    a = rng.integers(0, p, size=(T, m))
    th = (2 * np.pi * a / p)[None]
    q = rng.standard_normal((1, T, 2 * m))
    k = rng.standard_normal((1, T, 2 * m))
    v = rng.standard_normal((1, T, dv))
    S0 = rng.standard_normal((1, 2 * m, dv))
    _, _, ST = run_rec(q, k, v, np.ones((1, T, m)), th, np.zeros((1, T)), S0)
    resid = a.sum(0) % p                               # exact integer bookkeeping
    S0c = S0[0][0::2] + 1j * S0[0][1::2]
    want = np.exp(2j * np.pi * resid / p)[:, None] * S0c
    assert np.abs(ST[0][0::2] - want.real).max() < 1e-11      # paper: modular error 3.0e-12
    assert np.abs(ST[0][1::2] - want.imag).max() < 1e-11


# ----------------------------------------------------------------------------
# P6: register write (Theorem on register memory): Lambda = I, beta = 1, k = e_i
# ----------------------------------------------------------------------------
def test_register_overwrite():
    m, dv = 5, 3
    rng = np.random.default_rng(17)
    S0 = rng.standard_normal((1, 2 * m, dv))
    i = 2
    k = np.zeros((1, 1, 2 * m))
    k[0, 0, 2 * i] = 1.0
    a = rng.standard_normal((1, 1, dv))
    q = rng.standard_normal((1, 1, 2 * m))
    _, _, ST = run_rec(q, k, a, np.ones((1, 1, m)), np.zeros((1, 1, m)), np.ones((1, 1)), S0)
    want = S0[0].copy()
    want[2 * i] = a[0, 0]
    want[2 * i + 1] = 0.0
    assert np.abs(ST[0] - want).max() < 1e-15


# ----------------------------------------------------------------------------
# P7: chunk-size invariance and split-sequence continuation (Theorem "Chunk-bounded exactness")
# ----------------------------------------------------------------------------
def test_chunk_size_invariance_and_continuation():
    N, T, m, dv = 1, 96, 6, 4
    q, k, v, al, th, be, S0 = rand_inputs(18, N, T, m, dv)
    ref = run_rec(q, k, v, al, th, be, S0)
    for C in (16, 32, 64, 7):
        got = chunk_wy.forward_chunked(q[0], k[0], v[0], al[0], th[0], be[0], S0[0], C)
        for g, r in zip(got, ref):
            assert np.abs(g - r[0]).max() < 1e-12
    T1 = 37
    o1 = run_rec(q[:, :T1], k[:, :T1], v[:, :T1], al[:, :T1], th[:, :T1], be[:, :T1], S0)
    o2 = run_rec(q[:, T1:], k[:, T1:], v[:, T1:], al[:, T1:], th[:, T1:], be[:, T1:], o1[2])
    assert np.abs(np.concatenate([o1[0], o2[0]], 1) - ref[0]).max() < 1e-13
    assert np.abs(np.concatenate([o1[1], o2[1]], 1) - ref[1]).max() < 1e-13
    assert np.abs(o2[2] - ref[2]).max() < 1e-13


# ----------------------------------------------------------------------------
# P8: affine transfer (Theorem "Exact affine chunk transfer")
# ----------------------------------------------------------------------------
def test_affine_transfer_against_dense_sum():
    T, m, dv = 12, 5, 3
    q, k, v, al, th, be, S0 = rand_inputs(19, 1, T, m, dv)
    kc = cplx(k[0])
    _, states, As = dense_forward(q[0], k[0], v[0], al[0], th[0], be[0], S0[0])
    # B^chunk = sum_i A_{C:i+1} B_i with dense products
    Bc = np.zeros((m, dv), complex)
    for i in range(T):
        P = np.eye(m, dtype=complex)
        for s in range(i + 1, T):
            P = As[s] @ P
        Bc += P @ (be[0, i] * np.outer(kc[i], v[0, i]))
    G, Y, W, M = chunk_wy.chunk_factors(kc, al[0], th[0], be[0])
    S0c = S0[0][0::2] + 1j * S0[0][1::2]
    S_out = G[:, None] * S0c - Y @ (M @ (W.conj().T @ S0c)) + Bc
    assert np.abs(S_out - states[-1]).max() < 1e-13
    # zero-state run of the C oracle gives the same write summary
    _, _, ST0 = run_rec(q, k, v, al, th, be, None)
    assert np.abs((ST0[0][0::2] + 1j * ST0[0][1::2]) - Bc).max() < 1e-13


# ----------------------------------------------------------------------------
# P9/P10: rank and stability (Cor. "SFDA admits exact constructive block-WY products",
# Prop. "Basic numerical stability")
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("m,C", [(8, 4), (8, 8), (6, 10)])
def test_correction_rank(m, C):
    _, k, _, al, th, be, _ = rand_inputs(20, 1, C, m, 1)
    be = np.maximum(be, 0.2)
    G, Y, W, M = chunk_wy.chunk_factors(cplx(k[0]), al[0], th[0], be[0])
    corr = Y @ M @ W.conj().T
    assert np.linalg.matrix_rank(corr, tol=1e-10) == min(C, m)


def test_spectral_and_frobenius_bounds():
    N, T, m, dv = 1, 200, 6, 4
    q, k, v, al, th, be, S0 = rand_inputs(21, N, T, m, dv, alpha_lo=0.0)
    kc = cplx(k[0])
    worst = 0.0
    for t in range(T):
        worst = max(worst, np.linalg.norm(dense_A(kc[t], al[0, t], th[0, t], be[0, t]), 2))
    assert worst <= 1.0 + 1e-12
    bound = np.linalg.norm(S0[0]) + np.cumsum(be[0] * np.linalg.norm(k[0], axis=1) * np.linalg.norm(v[0], axis=1))
    for Tcut in (1, 50, 200):
        _, _, ST = run_rec(q[:, :Tcut], k[:, :Tcut], v[:, :Tcut], al[:, :Tcut], th[:, :Tcut], be[:, :Tcut], S0)
        assert np.linalg.norm(ST[0]) <= bound[Tcut - 1] + 1e-9


# ----------------------------------------------------------------------------
# P11: block-WY closure (Theorem "Block-WY closure") on two exported chunk tuples
# ----------------------------------------------------------------------------
def test_closure_of_two_chunks():
    m, C = 6, 5
    _, k, _, al, th, be, _ = rand_inputs(22, 1, 2 * C, m, 1)
    kc = cplx(k[0])
    G1, Y1, W1, M1 = chunk_wy.chunk_factors(kc[:C], al[0, :C], th[0, :C], be[0, :C])
    G2, Y2, W2, M2 = chunk_wy.chunk_factors(kc[C:], al[0, C:], th[0, C:], be[0, C:])
    G21 = G2 * G1
    Y21 = np.concatenate([G2[:, None] * Y1, Y2], 1)
    W21 = np.concatenate([W1, np.conj(G1)[:, None] * W2], 1)
    M21 = np.block([[M1, np.zeros((C, C))], [-M2 @ W2.conj().T @ Y1 @ M1, M2]])
    P = np.eye(m, dtype=complex)
    for t in range(2 * C):
        P = dense_A(kc[t], al[0, t], th[0, t], be[0, t]) @ P
    assert np.abs(np.diag(G21) - Y21 @ M21 @ W21.conj().T - P).max() < 1e-13
    # and the 2C-token recursion yields exactly these composed factors
    G, Y, W, M = chunk_wy.chunk_factors(kc, al[0], th[0], be[0])
    assert np.abs(G - G21).max() < 1e-13 and np.abs(Y - Y21).max() < 1e-13
    assert np.abs(W - W21).max() < 1e-13 and np.abs(M - M21).max() < 1e-12


# ----------------------------------------------------------------------------
# P12: realification (Prop. "Complex phases are real block rotations")
# ----------------------------------------------------------------------------
def test_real_block_formulation():
    """Same map on R^{2m}: 2x2 blocks alpha R(theta); the complex rank-one k k^*
    is the real rank-two projector k k^T + (Jk)(Jk)^T."""
    T, m, dv = 25, 4, 3
    q, k, v, al, th, be, S0 = rand_inputs(23, 1, T, m, dv)
    o_re, o_im, ST = run_rec(q, k, v, al, th, be, S0)
    S = S0[0].copy()
    J = np.kron(np.eye(m), np.array([[0.0, -1.0], [1.0, 0.0]]))
    for t in range(T):
        Lam = np.zeros((2 * m, 2 * m))
        for j in range(m):
            c, s = np.cos(th[0, t, j]), np.sin(th[0, t, j])
            Lam[2 * j:2 * j + 2, 2 * j:2 * j + 2] = al[0, t, j] * np.array([[c, -s], [s, c]])
        kr = k[0, t]
        Jk = J @ kr
        E = np.eye(2 * m) - be[0, t] * (np.outer(kr, kr) + np.outer(Jk, Jk))
        S = E @ Lam @ S + be[0, t] * np.outer(kr, v[0, t])
        assert np.abs(o_re[0, t] - S.T @ q[0, t]).max() < 1e-12
        assert np.abs(o_im[0, t] + S.T @ (J @ q[0, t])).max() < 1e-12
    assert np.abs(ST[0] - S).max() < 1e-12


# ----------------------------------------------------------------------------
# closed forms the GPU kernels use, checked against the literal recursion
# ----------------------------------------------------------------------------
def test_closed_form_factors():
    m, C = 7, 12
    _, k, _, al, th, be, _ = rand_inputs(24, 1, C, m, 1)
    kc = cplx(k[0])
    G, Y, W, M = chunk_wy.chunk_factors(kc, al[0], th[0], be[0])
    gam = np.cumprod(al[0] * np.exp(1j * th[0]), axis=0)           # gamma_t
    assert np.abs(G - gam[-1]).max() < 1e-14
    assert np.abs(W - (np.conj(gam) * kc).T).max() < 1e-14
    assert np.abs(Y - ((gam[-1] / gam) * be[0][:, None] * kc).T).max() < 1e-13
    Kt = np.zeros((C, C), complex)
    for t in range(C):
        for i in range(t):
            Kt[t, i] = np.sum(np.conj(kc[t]) * (gam[t] / gam[i]) * kc[i])
    N = Kt * be[0][None, :]
    assert np.abs(M - np.linalg.inv(np.eye(C) + N)).max() < 1e-12


# ----------------------------------------------------------------------------
# integer bookkeeping
# ----------------------------------------------------------------------------
PI50 = "3.14159265358979323846264338327950288419716939937510"


def test_phase_turns_match_exact_rational_rounding():
    from decimal import Decimal, getcontext, ROUND_HALF_EVEN
    getcontext().prec = 60
    rng = np.random.default_rng(25)
    th = np.concatenate([rng.uniform(-np.pi, np.pi, 2000), [0.0, np.pi, -np.pi, 1e-9, -1e-9, 100.0, -7.5]]).astype(np.float32)
    got = bookkeeping.phase_to_turns(th)
    scale = Decimal(2 ** 32) / (2 * Decimal(PI50))
    exact_mismatch = 0
    for x, g in zip(th, got):
        e = int((Decimal(float(x)) * scale).to_integral_value(rounding=ROUND_HALF_EVEN)) % 2 ** 32
        d = (int(g) - e) % 2 ** 32
        assert d in (0, 1, 2 ** 32 - 1)        # double rounding may move a near-tie by one unit
        exact_mismatch += d != 0
    assert exact_mismatch <= 2
    assert np.array_equal(bookkeeping.phase_to_turns(-th), (-got.astype(np.int64) & 0xFFFFFFFF).astype(np.uint32))


def test_cumulative_turns_are_chunk_local_integer_sums():
    rng = np.random.default_rng(26)
    T, m, C = 50, 3, 16
    th = rng.uniform(-np.pi, np.pi, (2, T, m)).astype(np.float32)
    u = bookkeeping.phase_to_turns(th)
    cum = bookkeeping.cumulative_phase_turns(th, C)
    for n in range(2):
        for j in range(m):
            acc = 0
            for t in range(T):
                if t % C == 0:
                    acc = 0
                acc = (acc + int(u[n, t, j])) % 2 ** 32
                assert int(cum[n, t, j]) == acc
    # quantised phases: p steps of 2 pi / p come back to within p rounding units of zero
    for p in (2, 3, 5, 7):
        thp = np.full((1, p, 1), 2 * np.pi / p, np.float32)
        last = int(bookkeeping.cumulative_phase_turns(thp, 64)[0, -1, 0])
        dist = min(last, 2 ** 32 - last)
        assert dist <= 2 ** 32 * 2.0 ** -24 * p      # float32 spacing of theta, p times
    assert int(bookkeeping.cumulative_phase_turns(np.full((1, 2, 1), np.pi, np.float32), 64)[0, -1, 0]) \
        == (2 * int(bookkeeping.phase_to_turns(np.float32(np.pi)))) % 2 ** 32


def test_single_precision_phase_turns_match_exact_rational_arithmetic():
    """phase_to_turns_f32 against its definition in exact arithmetic: the float32 nearest to the exact product of
    the two float32 factors (ties to even), then the nearest integer (ties to even), modulo 2**32."""
    from fractions import Fraction
    rng = np.random.default_rng(27)
    th = np.concatenate([rng.uniform(-np.pi, np.pi, 3000), rng.uniform(-40.0, 40.0, 500),
                         [0.0, np.pi, -np.pi, 1e-9, -1e-9, 100.0, -7.5, 2 * np.pi / 3, 2 * np.pi / 7]]).astype(np.float32)
    got = bookkeeping.phase_to_turns_f32(th)
    c = Fraction(float(bookkeeping.TURNS_PER_RADIAN_F32))
    assert abs(float(c) - 2 ** 32 / (2 * np.pi)) <= 32.0           # float32 spacing there is 64

    def round_to_f32(x):            # nearest float32 (24-bit significand) to the rational x, ties to even
        if x == 0:
            return Fraction(0)
        sign, a = (-1 if x < 0 else 1), abs(x)
        e = 0
        while a >= 2 ** 24:
            a /= 2
            e += 1
        while a < 2 ** 23:
            a *= 2
            e -= 1
        n = a.numerator // a.denominator
        rem = a - n
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
            n += 1
        return sign * Fraction(n) * Fraction(2) ** e

    def round_half_even(x):
        n = x.numerator // x.denominator
        rem = x - n
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
            n += 1
        return n

    for x, g in zip(th, got):
        want = round_half_even(round_to_f32(Fraction(float(x)) * c)) % 2 ** 32
        assert int(g) == want
    # odd symmetry, and closeness to the double-precision conversion: within 2^-24 of the angle (plus one unit)
    assert np.array_equal(bookkeeping.phase_to_turns_f32(-th), (-got.astype(np.int64) & 0xFFFFFFFF).astype(np.uint32))
    d = (got.astype(np.int64) - bookkeeping.phase_to_turns(th).astype(np.int64) + 2 ** 31) % 2 ** 32 - 2 ** 31
    assert np.all(np.abs(d) <= np.abs(th.astype(np.float64)) * bookkeeping.TURNS_PER_RADIAN * 2.0 ** -23 + 1)


def test_chunk_closing_turns_are_integer_sums_over_each_chunk():
    rng = np.random.default_rng(28)
    T, m, C = 150, 3, 64
    th = rng.uniform(-np.pi, np.pi, (2, T, m)).astype(np.float32)
    u = bookkeeping.phase_to_turns_f32(th)
    close = bookkeeping.chunk_closing_turns_f32(th, C)
    assert close.shape == (2, 3, m) and close.dtype == np.uint32
    for n in range(2):
        for j in range(m):
            for c in range(3):
                acc = 0
                for t in range(c * C, min((c + 1) * C, T)):
                    acc = (acc + int(u[n, t, j])) % 2 ** 32
                assert int(close[n, c, j]) == acc
    # p steps of 2 pi / p close a chunk within p rounding units of a whole turn
    for p_ in (2, 3, 5, 7):
        last = int(bookkeeping.chunk_closing_turns_f32(np.full((1, p_, 1), 2 * np.pi / p_, np.float32), 64)[0, 0, 0])
        assert min(last, 2 ** 32 - last) <= 2 ** 32 * 2.0 ** -23 * p_


def test_chunk_plan():
    assert bookkeeping.chunk_plan(256, 16) == (16, 16)
    assert bookkeeping.chunk_plan(257, 16) == (17, 1)
    assert bookkeeping.chunk_plan(5, 64) == (1, 5)
    assert bookkeeping.chunk_plan(131072, 64) == (2048, 64)
    with pytest.raises(ValueError):
        bookkeeping.chunk_plan(0, 16)


# ----------------------------------------------------------------------------
# stable parameterisation (paragraph "Stable parameterization", Section 3)
# ----------------------------------------------------------------------------
def test_parameterisation_special_values_and_ranges():
    """Values the formulas fix by themselves: sigmoid(0) = 1/2, tanh(0) = 0, the limits, the symmetry of the
    sigmoid, and a key of norm n mapped to norm n / (n + eps) without changing its direction."""
    import math
    z1, z0 = np.zeros((1, 3)), np.zeros(1)
    k1 = np.array([[3.0, 0.0, 4.0, 0.0]])
    al, th, be, k = frontend.stable_parameterisation(z1, z1, z0, k1, 0.2, 0.9, 2.5, 1e-3)
    assert np.allclose(al, 0.55) and np.allclose(th, 0.0) and np.allclose(be, 0.5)
    assert np.allclose(k, k1 / (5.0 + 1e-3), rtol=0, atol=1e-15)
    big = np.full((1, 3), 40.0)
    al, th, be, _ = frontend.stable_parameterisation(big, big, np.full(1, 40.0), k1, 0.2, 0.9, 2.5, 1e-3)
    assert np.allclose(al, 0.9) and np.allclose(th, 2.5) and np.allclose(be, 1.0)
    al, th, be, _ = frontend.stable_parameterisation(-big, -big, np.full(1, -40.0), k1, 0.2, 0.9, 2.5, 1e-3)
    assert np.allclose(al, 0.2) and np.allclose(th, -2.5) and np.allclose(be, 0.0, atol=1e-15)
    # against the standard library, written with other functions than the oracle uses
    rng = np.random.default_rng(7)
    a, b, c = rng.normal(0, 3, (5, 4)), rng.normal(0, 2, (5, 4)), rng.normal(0, 3, 5)
    kr = rng.normal(0, 1, (5, 8))
    al, th, be, k = frontend.stable_parameterisation(a, b, c, kr, 0.1, 1.0, math.pi, 1e-6)
    for i in range(5):
        for j in range(4):
            assert math.isclose(al[i, j], 0.1 + 0.9 * 0.5 * (1.0 + math.tanh(0.5 * a[i, j])), rel_tol=1e-12)
            assert math.isclose(th[i, j], math.pi * math.expm1(2 * b[i, j]) / (math.expm1(2 * b[i, j]) + 2.0), rel_tol=1e-12)
        assert math.isclose(be[i] + float(frontend.sigmoid(-c[i])), 1.0, rel_tol=1e-14)
        n = math.sqrt(sum(x * x for x in kr[i]))
        assert math.isclose(math.sqrt(sum(x * x for x in k[i])), n / (n + 1e-6), rel_tol=1e-12)
        assert np.allclose(k[i] * kr[i, 0], kr[i] * k[i, 0], rtol=0, atol=1e-14) and np.all(k[i] * kr[i] >= 0)   # same direction


def test_parameterisation_gives_the_stability_assumptions():
    """||Lambda|| <= 1, 0 <= beta ||k||^2 <= 1 (the sentence after Eq. "param-key"), on heavy-tailed raw inputs; and a
    recurrence driven by them never grows a state beyond the bound of Prop. "Basic numerical stability"."""
    rng = np.random.default_rng(11)
    N, T, m, dv = 2, 40, 3, 4
    a, b, c = rng.standard_cauchy((N, T, m)), rng.standard_cauchy((N, T, m)), rng.standard_cauchy((N, T))
    kr = rng.standard_cauchy((N, T, 2 * m))
    al, th, be, k = frontend.stable_parameterisation(a, b, c, kr, 0.0, 1.0, np.pi, 1e-6)
    assert np.all((al >= 0) & (al <= 1)) and np.all(np.abs(th) <= np.pi) and np.all((be >= 0) & (be <= 1))
    n2 = np.sum(k * k, axis=-1)
    assert np.all(n2 <= 1.0) and np.all(be * n2 <= 1.0)
    q, v = rng.standard_normal((N, T, 2 * m)), rng.standard_normal((N, T, dv))
    _, _, S_T = recurrence.sfda_recurrence(q, k, v, al, th, be, None)
    bound = np.sum(np.sqrt(be)[..., None] * np.linalg.norm(v, axis=-1)[..., None], axis=1)   # sum_t sqrt(beta_t) ||v_t||
    assert np.all(np.linalg.norm(S_T.reshape(N, -1), axis=-1) <= bound[:, 0] + 1e-9)


def test_parameterisation_backward_matches_central_differences():
    """The gradients with respect to the raw inputs against (L(x + h e) - L(x - h e)) / 2h of the forward
    parameterisation, L = <dalpha, alpha> + <dtheta, theta> + <dbeta, beta> + <dk, k>, entry by entry; a zero key
    passes s dk through; and the key's gradient is orthogonal to the key when eps = 0 (k does not depend on the
    length of k_raw then)."""
    rng = np.random.default_rng(61)
    a, b, c = rng.normal(0, 2, (3, 4)), rng.normal(0, 1.5, (3, 4)), rng.normal(0, 2, 3)
    kr = rng.normal(0, 1, (3, 8))
    up = [rng.normal(size=x.shape) for x in (a, b, c, kr)]
    par = (0.1, 0.95, 2.0, 1e-3)

    def loss(a_, b_, c_, k_):
        out = frontend.stable_parameterisation(a_, b_, c_, k_, *par)
        return float(sum(np.sum(u * o) for u, o in zip(up, out)))

    got = frontend.stable_parameterisation_backward(a, b, c, kr, *par, *up)
    h = 1e-6
    for idx_arr, (x, g) in enumerate(zip((a, b, c, kr), got)):
        for idx in np.ndindex(x.shape):
            args_p, args_m = [a.copy(), b.copy(), c.copy(), kr.copy()], [a.copy(), b.copy(), c.copy(), kr.copy()]
            args_p[idx_arr][idx] += h
            args_m[idx_arr][idx] -= h
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(fd - g[idx]) <= 1e-7 * max(1.0, abs(fd)), (idx_arr, idx, fd, g[idx])
    z = np.zeros((1, 8))
    dk = rng.normal(size=(1, 8))
    g0 = frontend.stable_parameterisation_backward(a[:1], b[:1], c[:1], z, *par, up[0][:1], up[1][:1], up[2][:1], dk)[3]
    assert np.allclose(g0, dk / 1e-3)
    g1 = frontend.stable_parameterisation_backward(a, b, c, kr, 0.1, 0.95, 2.0, 0.0, *up)[3]
    assert np.allclose(np.sum(g1 * kr, axis=-1), 0.0, atol=1e-12)


# ----------------------------------------------------------------------------
# backward pass: the gradient of a scalar loss through Eq. "sfda"
# ----------------------------------------------------------------------------
def _loss_inputs(seed, N=2, T=7, m=3, dv=4, s0=True):
    rng = np.random.default_rng(seed)
    x = dict(q=rng.standard_normal((N, T, 2 * m)), k=0.6 * rng.standard_normal((N, T, 2 * m)),
             v=rng.standard_normal((N, T, dv)), alpha=rng.uniform(0.5, 1.0, (N, T, m)),
             theta=rng.uniform(-np.pi, np.pi, (N, T, m)), beta=rng.uniform(0.1, 0.9, (N, T)),
             S0=(rng.standard_normal((N, 2 * m, dv)) if s0 else None))
    up = dict(do_re=rng.standard_normal((N, T, dv)), do_im=rng.standard_normal((N, T, dv)),
              dS_T=rng.standard_normal((N, 2 * m, dv)))
    return x, up


def _loss(x, up):
    """L = sum do_re . Re o + do_im . Im o + <dS_T, S_T>, evaluated by the forward oracle."""
    o_re, o_im, S_T = recurrence.sfda_recurrence(x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], x["S0"])
    return float(np.sum(up["do_re"] * o_re) + np.sum(up["do_im"] * o_im) + np.sum(up["dS_T"] * S_T))


def test_backward_matches_central_differences_of_the_forward_oracle():
    """Every gradient, entry by entry on a sample, against (L(x + h e) - L(x - h e)) / 2h of the independently
    written forward oracle (C, per token); also across a segment boundary of the checkpointing."""
    for seed, seg in ((0, 64), (1, 3)):
        x, up = _loss_inputs(seed)
        g = dict(zip(("q", "k", "v", "alpha", "theta", "beta", "S0"),
                     backward.sfda_backward(x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], x["S0"],
                                            up["do_re"], up["do_im"], up["dS_T"], seg=seg)))
        rng = np.random.default_rng(100 + seed)
        h = 1e-6
        for name in g:
            flat = x[name].reshape(-1)
            for idx in rng.choice(flat.size, size=min(12, flat.size), replace=False):
                keep = flat[idx]
                flat[idx] = keep + h
                lp = _loss(x, up)
                flat[idx] = keep - h
                lm = _loss(x, up)
                flat[idx] = keep
                fd = (lp - lm) / (2 * h)
                assert abs(fd - g[name].reshape(-1)[idx]) <= 2e-7 * max(1.0, abs(fd)), (name, idx, fd, g[name].reshape(-1)[idx])


def test_backward_without_writes_is_the_adjoint_of_the_diagonal_scan():
    """beta = 0: S_t = Gamma_t S_0 and o_t = S_0^* conj(Gamma_t) q_t (Prop. "Interpolation ..."), so
    dS0 = sum_t conj(Gamma_t)^{-1}... written out: dS0_j = sum_t conj(gamma_tj) (q_tj yb_t^*) + conj(gamma_Tj) dS_T,j,
    dq_t = Gamma_t S_0 yb_t, and dv = dbeta-free terms vanish (dv = 0)."""
    x, up = _loss_inputs(3, N=1, T=6)
    x["beta"][:] = 0.0
    dq, dk, dv, dal, dth, dbe, dS0 = backward.sfda_backward(x["q"], x["k"], x["v"], x["alpha"], x["theta"],
                                                             x["beta"], x["S0"], up["do_re"], up["do_im"], up["dS_T"])
    lam = x["alpha"][0] * np.exp(1j * x["theta"][0])                 # [T, m]
    gam = np.cumprod(lam, axis=0)
    S0 = x["S0"][0, 0::2] + 1j * x["S0"][0, 1::2]
    yb = up["do_re"][0] + 1j * up["do_im"][0]
    qc = x["q"][0, :, 0::2] + 1j * x["q"][0, :, 1::2]
    GT = up["dS_T"][0, 0::2] + 1j * up["dS_T"][0, 1::2]
    want_dS0 = gam[-1].conj()[:, None] * GT + sum(gam[t].conj()[:, None] * np.outer(qc[t], yb[t].conj()) for t in range(6))
    assert np.allclose(dS0[0, 0::2] + 1j * dS0[0, 1::2], want_dS0, rtol=0, atol=1e-12)
    for t in range(6):
        want_dq = (gam[t][:, None] * S0) @ yb[t]
        assert np.allclose(dq[0, t, 0::2] + 1j * dq[0, t, 1::2], want_dq, rtol=0, atol=1e-12)
    assert np.all(dv == 0) and np.all(dk == 0)


def test_backward_is_linear_in_the_upstream_and_additive_over_a_split():
    """The cotangents are linear in (do, dS_T); and running the second half first, then feeding its dS0 to the
    first half as dS_T, gives the gradients of the whole sequence (Theorem "Chunk-bounded exactness", transposed)."""
    x, up = _loss_inputs(5, N=2, T=9)
    full = backward.sfda_backward(x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], x["S0"],
                                  up["do_re"], up["do_im"], up["dS_T"])
    twice = backward.sfda_backward(x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], x["S0"],
                                   2 * up["do_re"], 2 * up["do_im"], 2 * up["dS_T"])
    for a, b in zip(full, twice):
        assert np.allclose(2 * a, b, rtol=1e-13, atol=1e-13)
    T1 = 4
    _, _, S_mid = recurrence.sfda_recurrence(x["q"][:, :T1], x["k"][:, :T1], x["v"][:, :T1], x["alpha"][:, :T1],
                                             x["theta"][:, :T1], x["beta"][:, :T1], x["S0"])
    second = backward.sfda_backward(x["q"][:, T1:], x["k"][:, T1:], x["v"][:, T1:], x["alpha"][:, T1:],
                                    x["theta"][:, T1:], x["beta"][:, T1:], S_mid, up["do_re"][:, T1:],
                                    up["do_im"][:, T1:], up["dS_T"])
    first = backward.sfda_backward(x["q"][:, :T1], x["k"][:, :T1], x["v"][:, :T1], x["alpha"][:, :T1],
                                   x["theta"][:, :T1], x["beta"][:, :T1], x["S0"], up["do_re"][:, :T1],
                                   up["do_im"][:, :T1], second[6])
    for i in range(6):
        assert np.allclose(np.concatenate([first[i], second[i]], axis=1), full[i], rtol=1e-12, atol=1e-12)
    assert np.allclose(first[6], full[6], rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("chunk,T", [(1, 5), (4, 12), (8, 8), (6, 18)])
def test_chunked_backward_equals_the_token_level_adjoint(chunk, T):
    """The chunk form of the backward pass (triangular solves with the forward's Gram matrix, state-sized products
    with S_0 and with the cotangent of S_C, C x C couplings) against the adjoint taken token by token -- and, for two
    of the gradients, directly against central differences of the forward oracle.  Includes beta = 0 and beta = 1
    tokens, a missing initial state, a missing Im cotangent and a missing final-state cotangent."""
    x, up = _loss_inputs(40 + chunk, N=2, T=T)
    x["beta"][0, 1] = 0.0
    x["beta"][1, 2] = 1.0
    args = (x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"])
    want = backward.sfda_backward(*args, x["S0"], up["do_re"], up["do_im"], up["dS_T"])
    got = backward_chunk.sfda_backward_chunked(*args, x["S0"], up["do_re"], up["do_im"], up["dS_T"], chunk)
    for name, a, b in zip(("dq", "dk", "dv", "dalpha", "dtheta", "dbeta", "dS0"), got, want):
        assert np.allclose(a, b, rtol=1e-10, atol=1e-10), name
    want = backward.sfda_backward(*args, None, up["do_re"], None, None)
    got = backward_chunk.sfda_backward_chunked(*args, None, up["do_re"], None, None, chunk)
    for name, a, b in zip(("dq", "dk", "dv", "dalpha", "dtheta", "dbeta", "dS0"), got, want):
        assert np.allclose(a, b, rtol=1e-10, atol=1e-10), name
    # independent of the token-level adjoint: finite differences of the forward oracle
    g = dict(zip(("q", "k", "v", "alpha", "theta", "beta", "S0"),
                 backward_chunk.sfda_backward_chunked(*args, x["S0"], up["do_re"], up["do_im"], up["dS_T"], chunk)))
    h = 1e-6
    for key, idx in (("theta", (1, T - 2, 1)), ("k", (0, 0, 3)), ("alpha", (0, T // 2, 0))):
        xp, xm = {n: np.array(a, copy=True) for n, a in x.items()}, {n: np.array(a, copy=True) for n, a in x.items()}
        xp[key][idx] += h
        xm[key][idx] -= h
        fd = (_loss(xp, up) - _loss(xm, up)) / (2 * h)
        assert abs(fd - g[key][idx]) <= 1e-6 * max(1.0, abs(fd)), (key, fd, g[key][idx])


# ----------------------------------------------------------------------------
# identities the CUDA path leans on, checked on the oracle alone
# ----------------------------------------------------------------------------
def test_key_normalisation_is_a_rescaling_of_beta_and_v():
    """Eq. "sfda" with k = s k_raw equals Eq. "sfda" with k_raw, beta s^2 in place of beta and v / s in place of v
    (erase term beta s^2 k_raw k_raw^*, write term (beta s^2) k_raw (v / s)^*): states and outputs agree.  The fused
    forward never divides the key and relies on exactly this."""
    rng = np.random.default_rng(21)
    N, T, m, dv = 2, 30, 4, 5
    q = rng.standard_normal((N, T, 2 * m))
    k_raw = rng.standard_normal((N, T, 2 * m)) * np.exp(rng.standard_normal((N, T, 1)))
    v = rng.standard_normal((N, T, dv))
    alpha, theta = rng.uniform(0.6, 1.0, (N, T, m)), rng.uniform(-np.pi, np.pi, (N, T, m))
    beta = rng.uniform(0.0, 1.0, (N, T))
    S0 = rng.standard_normal((N, 2 * m, dv))
    s = 1.0 / (np.linalg.norm(k_raw, axis=-1) + 1e-6)
    a = recurrence.sfda_recurrence(q, k_raw * s[..., None], v, alpha, theta, beta, S0)
    b = recurrence.sfda_recurrence(q, k_raw, v / s[..., None], alpha, theta, beta * s * s, S0)
    for x, y in zip(a, b):
        assert np.allclose(x, y, rtol=1e-11, atol=1e-11)


def test_time_slice_transfer_from_the_identity_state_and_the_zero_state():
    """Over a time slice S_out = P S_in + B (Theorem "Exact affine chunk transfer"): B is what the slice reaches from
    a zero state, and P is read off the first m columns of what it reaches with v = 0 from the state [I | 0].
    Scanning S_{i+1} = P_i S_i + B_i over the slices reproduces the states of the whole sequence, and the outputs of
    every slice from its scanned state are those of the whole sequence: the two-level scan is exact."""
    rng = np.random.default_rng(22)
    N, T, m, dv, n = 2, 24, 3, 4, 4
    q, k = rng.standard_normal((N, T, 2 * m)), 0.7 * rng.standard_normal((N, T, 2 * m))
    v = rng.standard_normal((N, T, dv))
    alpha, theta = rng.uniform(0.6, 1.0, (N, T, m)), rng.uniform(-np.pi, np.pi, (N, T, m))
    beta = rng.uniform(0.0, 1.0, (N, T))
    S0 = rng.standard_normal((N, 2 * m, dv))
    o_re, o_im, S_T = recurrence.sfda_recurrence(q, k, v, alpha, theta, beta, S0)
    L = T // n
    ident = np.zeros((N, 2 * m, m))                    # complex identity in paired rows: Re row 2j, column j
    for j in range(m):
        ident[:, 2 * j, j] = 1.0
    S = S0[:, 0::2] + 1j * S0[:, 1::2]
    for i in range(n):
        sl = slice(i * L, (i + 1) * L)
        S_in = np.empty((N, 2 * m, dv))
        S_in[:, 0::2], S_in[:, 1::2] = S.real, S.imag
        got_re, got_im, _ = recurrence.sfda_recurrence(q[:, sl], k[:, sl], v[:, sl], alpha[:, sl], theta[:, sl],
                                                       beta[:, sl], S_in)
        assert np.allclose(got_re, o_re[:, sl], atol=1e-11) and np.allclose(got_im, o_im[:, sl], atol=1e-11)
        _, _, Bp = recurrence.sfda_recurrence(q[:, sl], k[:, sl], v[:, sl], alpha[:, sl], theta[:, sl], beta[:, sl], None)
        _, _, Pp = recurrence.sfda_recurrence(q[:, sl], k[:, sl], np.zeros((N, L, m)), alpha[:, sl], theta[:, sl],
                                              beta[:, sl], ident)
        P = Pp[:, 0::2] + 1j * Pp[:, 1::2]            # [N, m, m]
        Bc = Bp[:, 0::2] + 1j * Bp[:, 1::2]
        S = np.einsum("njl,nlc->njc", P, S) + Bc
    assert np.allclose(S.real, S_T[:, 0::2], atol=1e-11) and np.allclose(S.imag, S_T[:, 1::2], atol=1e-11)


# ----------------------------------------------------------------------------
# write-decoupled variant (Eq. "sfda-decoupled-main")
# ----------------------------------------------------------------------------
def _decoupled_inputs(seed, N=2, T=12, m=3, dv=4):
    rng = np.random.default_rng(seed)
    return dict(q=rng.standard_normal((N, T, 2 * m)), k=0.6 * rng.standard_normal((N, T, 2 * m)),
                r=0.6 * rng.standard_normal((N, T, 2 * m)), v=rng.standard_normal((N, T, dv)),
                alpha=rng.uniform(0.5, 1.0, (N, T, m)), theta=rng.uniform(-np.pi, np.pi, (N, T, m)),
                eta=rng.uniform(0.1, 0.9, (N, T)), beta=rng.uniform(0.1, 0.9, (N, T)),
                S0=rng.standard_normal((N, 2 * m, dv)))


def test_decoupled_variant_reduces_to_the_tied_model():
    """r = k and eta = beta is Eq. "sfda" (checked against the C oracle); r = k with eta != beta is Eq. "sfda" with
    beta := eta and v := (beta / eta) v."""
    from oracle import variants
    x = _decoupled_inputs(31)
    a = variants.sfda_decoupled_recurrence(x["q"], x["k"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], x["beta"], x["S0"])
    b = recurrence.sfda_recurrence(x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], x["S0"])
    for u, w in zip(a, b):
        assert np.allclose(u, w, rtol=1e-12, atol=1e-12)
    a = variants.sfda_decoupled_recurrence(x["q"], x["k"], x["k"], x["v"], x["alpha"], x["theta"], x["eta"], x["beta"], x["S0"])
    b = recurrence.sfda_recurrence(x["q"], x["k"], x["v"] * (x["beta"] / x["eta"])[..., None], x["alpha"], x["theta"],
                                   x["eta"], x["S0"])
    for u, w in zip(a, b):
        assert np.allclose(u, w, rtol=1e-12, atol=1e-12)


def test_decoupled_variant_against_explicit_matrices_and_limits():
    """Dense brute force S_t = A_t S_{t-1} + B_t with explicit m x m matrices; eta = 0 leaves a decayed sum of the
    writes, S_T = Gamma_T S_0 + sum_t (Gamma_T / Gamma_t) beta_t r_t v_t^T; beta = 0 never increases the Frobenius
    norm when eta |k|^2 <= 1 (the erase factor is a contraction, Prop. "Basic numerical stability")."""
    from oracle import variants
    x = _decoupled_inputs(32, N=1, T=7)
    o_re, o_im, S_T = variants.sfda_decoupled_recurrence(**x)
    m = 3
    kc, rc, qc = (x[n][0, :, 0::2] + 1j * x[n][0, :, 1::2] for n in ("k", "r", "q"))
    lam = x["alpha"][0] * np.exp(1j * x["theta"][0])
    S = x["S0"][0, 0::2] + 1j * x["S0"][0, 1::2]
    for t in range(7):
        A = (np.eye(m) - x["eta"][0, t] * np.outer(kc[t], kc[t].conj())) @ np.diag(lam[t])
        S = A @ S + x["beta"][0, t] * np.outer(rc[t], x["v"][0, t])
        assert np.allclose(S.conj().T @ qc[t], o_re[0, t] + 1j * o_im[0, t], atol=1e-12)
    assert np.allclose(S, S_T[0, 0::2] + 1j * S_T[0, 1::2], atol=1e-12)
    # eta = 0
    y = dict(x, eta=np.zeros_like(x["eta"]))
    _, _, S_T0 = variants.sfda_decoupled_recurrence(**y)
    gam = np.cumprod(lam, axis=0)
    want = gam[-1][:, None] * (x["S0"][0, 0::2] + 1j * x["S0"][0, 1::2]) + sum(
        (gam[-1] / gam[t])[:, None] * x["beta"][0, t] * np.outer(rc[t], x["v"][0, t]) for t in range(7))
    assert np.allclose(S_T0[0, 0::2] + 1j * S_T0[0, 1::2], want, atol=1e-12)
    # beta = 0, eta |k|^2 <= 1
    z = dict(x, beta=np.zeros_like(x["beta"]))
    z["k"] = z["k"] / np.linalg.norm(z["k"], axis=-1, keepdims=True)
    norms = [np.linalg.norm(x["S0"][0])]
    for T_ in range(1, 8):
        _, _, S_p = variants.sfda_decoupled_recurrence(**{n: (v if n == "S0" else v[:, :T_]) for n, v in z.items()})
        norms.append(np.linalg.norm(S_p[0]))
    assert all(b <= a + 1e-12 for a, b in zip(norms[:-1], norms[1:]))


# ----------------------------------------------------------------------------
# real-coordinate model with 2 x 2 orthogonal control blocks (rotations, reflections) and a real rank-one erase
# ----------------------------------------------------------------------------
def test_block_controls_without_reflections_are_the_complex_model():
    """Lemma "Real-to-complex phase equivalence": with rotation blocks only and the realified complex erase, the
    real-coordinate recurrence (dense real matrices) is the complex write-decoupled recurrence."""
    from oracle import variants
    x = _decoupled_inputs(50, N=2, T=9)
    a = variants.sfda_decoupled_recurrence(**x)
    b = variants.sfda_block_control_recurrence(x["q"], x["k"], x["r"], x["v"], x["alpha"], x["theta"], None, x["eta"],
                                               x["beta"], x["S0"])
    for u, w in zip(a, b):
        assert np.allclose(u, w, rtol=1e-12, atol=1e-12)


def test_reflection_block_is_complex_conjugation():
    """F = diag(1, -1) on a row pair is z -> conj(z): a token whose blocks are alpha R(theta) F maps the complex row
    S_j to alpha e^{i theta} conj(S_j) (then the same erase and write as before)."""
    from oracle import variants
    x = _decoupled_inputs(51, N=1, T=6)
    rng = np.random.default_rng(51)
    flip = rng.integers(0, 2, (1, 6, 3))
    flip[0, 0] = 1
    o_re, o_im, S_T = variants.sfda_block_control_recurrence(x["q"], x["k"], x["r"], x["v"], x["alpha"], x["theta"],
                                                             flip, x["eta"], x["beta"], x["S0"])
    kc, rc, qc = (x[n][0, :, 0::2] + 1j * x[n][0, :, 1::2] for n in ("k", "r", "q"))
    lam = x["alpha"][0] * np.exp(1j * x["theta"][0])
    S = x["S0"][0, 0::2] + 1j * x["S0"][0, 1::2]
    for t in range(6):
        Z = lam[t][:, None] * np.where(flip[0, t][:, None] == 1, S.conj(), S)
        S = Z - x["eta"][0, t] * np.outer(kc[t], kc[t].conj() @ Z) + x["beta"][0, t] * np.outer(rc[t], x["v"][0, t])
        assert np.allclose(S.conj().T @ qc[t], o_re[0, t] + 1j * o_im[0, t], atol=1e-12)
    assert np.allclose(S, S_T[0, 0::2] + 1j * S_T[0, 1::2], atol=1e-12)


def test_dihedral_group_is_tracked_exactly():
    """Theorem "Dihedral phase-orientation memory": beta = 0, one row pair, d_v = 2, S_0 = I; the symbols R (rotation
    by 2 pi / n), F (reflection) and RF drive S_t = rho(sigma_t ... sigma_1).  The expected matrix comes from integer
    arithmetic in D_n, (R^a F^f)(R^b F^g) = R^{a + (-1)^f b} F^{f + g}; also F^2 = I and F R F = R^{-1}."""
    from oracle import variants
    n, T = 7, 40
    rng = np.random.default_rng(52)
    sym = rng.integers(0, 3, T)                       # 0: R, 1: F, 2: R F
    theta = np.where(sym == 1, 0.0, 2 * np.pi / n)[None, :, None]
    flip = (sym >= 1).astype(np.int64)[None, :, None]
    one, zero = np.ones((1, T)), np.zeros((1, T))
    zq = np.zeros((1, T, 2))
    _, _, S_T = variants.sfda_block_control_recurrence(zq, zq, zq, np.zeros((1, T, 2)), np.ones((1, T, 1)), theta, flip,
                                                       zero, zero, np.eye(2)[None])
    a, f = 0, 0                                       # group element R^a F^f, multiplied from the left
    for s in sym:
        b, g = (1, 0) if s == 0 else (0, 1) if s == 1 else (1, 1)
        a, f = (b + (-1) ** g * a) % n, (g + f) % 2   # (R^b F^g)(R^a F^f)
    ang = 2 * np.pi * a / n
    R = np.array([[np.cos(ang), -np.sin(ang)], [np.sin(ang), np.cos(ang)]])
    want = R @ (np.diag([1.0, -1.0]) if f else np.eye(2))
    assert np.allclose(S_T[0], want, atol=1e-12)
    assert abs(np.linalg.norm(S_T[0], 2) - 1.0) < 1e-12          # orthogonal: bounded norm

    def run(symbols):
        th = np.array([0.0 if s == 1 else 2 * np.pi / n for s in symbols])[None, :, None]
        fl = np.array([1 if s >= 1 else 0 for s in symbols])[None, :, None]
        L = len(symbols)
        z = np.zeros((1, L, 2))
        return variants.sfda_block_control_recurrence(z, z, z, z, np.ones((1, L, 1)), th, fl, np.zeros((1, L)),
                                                      np.zeros((1, L)), np.eye(2)[None])[2][0]
    assert np.allclose(run([1, 1]), np.eye(2), atol=1e-15)                        # F^2 = I
    assert np.allclose(run([1, 0, 1]) @ run([0]), np.eye(2), atol=1e-12)          # F R F = R^{-1}


def test_real_rank_one_erase_is_the_real_delta_rule():
    """With the erase k k^T on R^{2m} (Eq. "intro-sfda-real" read literally): theta = 0 and no reflections give the
    textbook real gated delta rule S <- (I - beta k k^T) Diag(a) S + beta k v^T of dimension 2m (Prop. "KDA is a
    special case"); a unit key with beta = 1 stores its value exactly, k_t^T S_t = v_t^T; and the real and the
    complex erase differ by exactly eta (Jk)(Jk)^T applied to the controlled state."""
    from oracle import variants
    x = _decoupled_inputs(53, N=1, T=8)
    x["k"] = x["k"] / np.linalg.norm(x["k"], axis=-1, keepdims=True)
    zero_th = np.zeros_like(x["theta"])
    o_re, _, S_T = variants.sfda_block_control_recurrence(x["q"], x["k"], x["k"], x["v"], x["alpha"], zero_th, None,
                                                          x["beta"], x["beta"], x["S0"], real_erase=True)
    S = x["S0"][0].copy()
    for t in range(8):
        a = np.repeat(x["alpha"][0, t], 2)
        kk, b = x["k"][0, t], x["beta"][0, t]
        S = a[:, None] * S
        S = S - b * np.outer(kk, kk @ S) + b * np.outer(kk, x["v"][0, t])
        assert np.allclose(S.T @ x["q"][0, t], o_re[0, t], atol=1e-12)
    assert np.allclose(S, S_T[0], atol=1e-12)
    # exact storage
    ones = np.ones_like(x["beta"])
    for T_ in (1, 5, 8):
        _, _, S_p = variants.sfda_block_control_recurrence(x["q"][:, :T_], x["k"][:, :T_], x["k"][:, :T_], x["v"][:, :T_],
                                                           x["alpha"][:, :T_], x["theta"][:, :T_], None, ones[:, :T_],
                                                           ones[:, :T_], x["S0"], real_erase=True)
        assert np.allclose(x["k"][0, T_ - 1] @ S_p[0], x["v"][0, T_ - 1], atol=1e-12)
    # one step: the two erase terms differ by eta (Jk)(Jk)^T Z
    args = [x[n][:, :1] for n in ("q", "k", "r", "v", "alpha", "theta")] + [None, x["eta"][:, :1], x["beta"][:, :1], x["S0"]]
    S_c = variants.sfda_block_control_recurrence(*args)[2][0]
    S_r = variants.sfda_block_control_recurrence(*args, real_erase=True)[2][0]
    lam = x["alpha"][0, 0] * np.exp(1j * x["theta"][0, 0])
    Zc = lam[:, None] * (x["S0"][0, 0::2] + 1j * x["S0"][0, 1::2])
    Z = np.empty_like(x["S0"][0])
    Z[0::2], Z[1::2] = Zc.real, Zc.imag
    Jk = np.empty(6)
    Jk[0::2], Jk[1::2] = -x["k"][0, 0, 1::2], x["k"][0, 0, 0::2]
    assert np.allclose(S_r - S_c, x["eta"][0, 0] * np.outer(Jk, Jk @ Z), atol=1e-12)
