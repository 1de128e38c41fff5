"""Integer bookkeeping of the chunked path (test infrastructure only).

The paper fixes no representation for the cumulative phase; the reading taken
here makes it exact: a phase is stored as an unsigned 32-bit count of
``2*pi / 2**32`` turns, so the chunk-local prefix product of Eq.
"constructive-Gamma" (``Gamma_t = Lambda_t Gamma_{t-1}``) becomes, for its unit
modulus part, a prefix *sum* modulo 2**32 that has one right answer whatever
order a scan adds it in.
"""
import numpy as np

# 2**32 / (2*pi) as the nearest double; the product below is one IEEE double
# multiply followed by round-to-nearest-even to an integer.
TURNS_PER_RADIAN = 4294967296.0 / (2.0 * np.pi)


def chunk_plan(T: int, chunk: int):
    """Number of chunks and length of the last one for T tokens."""
    if T < 1 or chunk < 1:
        raise ValueError("T and chunk must be positive")
    n_chunks = -(-T // chunk)
    tail = T - (n_chunks - 1) * chunk
    return n_chunks, tail


def phase_to_turns(theta):
    """theta (float32 radians) -> uint32 turns: rint(double(theta) * 2**32/(2 pi)) mod 2**32."""
    th = np.asarray(theta, dtype=np.float32).astype(np.float64)
    r = np.rint(th * TURNS_PER_RADIAN)          # round half to even, like llrint
    return (r.astype(np.int64) & 0xFFFFFFFF).astype(np.uint32)


def cumulative_phase_turns(theta, chunk: int):
    """Chunk-local inclusive prefix sum (mod 2**32) of the per-token turns.

    theta: [..., T, m] with the token axis second to last.  Token t of chunk c
    gets sum_{s = c*chunk .. t} turns_s  mod 2**32.
    """
    u = phase_to_turns(theta).astype(np.uint64)
    T = u.shape[-2]
    out = np.empty(u.shape, np.uint32)
    for start in range(0, T, chunk):
        stop = min(start + chunk, T)
        acc = np.cumsum(u[..., start:stop, :], axis=-2, dtype=np.uint64)
        out[..., start:stop, :] = (acc & 0xFFFFFFFF).astype(np.uint32)
    return out


# The same constant rounded to single precision (the nearest float32 to 683565275.57...), for the
# single-precision variant of the conversion.
TURNS_PER_RADIAN_F32 = np.float32(683565275.6)


def phase_to_turns_f32(theta):
    """Single-precision variant: the product theta * 2**32/(2 pi) is ONE float32 multiply (round to
    nearest even), then rounded to the nearest integer (ties to even) and wrapped modulo 2**32."""
    th = np.asarray(theta, dtype=np.float32)
    prod = th * TURNS_PER_RADIAN_F32                       # float32 * float32 -> float32, IEEE
    assert prod.dtype == np.float32
    r = np.rint(prod.astype(np.float64))                   # exact widening, then ties-to-even rounding
    return (r.astype(np.int64) & 0xFFFFFFFF).astype(np.uint32)


def chunk_closing_turns_f32(theta, chunk: int):
    """Phase every chunk closes with (Eq. "constructive-Gamma" at t = C, unit-modulus part), in 2**-32 turns:
    the sum modulo 2**32 of phase_to_turns_f32 over the chunk's tokens.

    theta: [..., T, m]  ->  [..., NC, m] uint32 with NC = ceil(T / chunk); a short last chunk sums
    the tokens it has (missing tokens are neutral: phase 0).
    """
    u = phase_to_turns_f32(theta).astype(np.uint64)
    T = u.shape[-2]
    n_chunks, _ = chunk_plan(T, chunk)
    out = np.empty(u.shape[:-2] + (n_chunks, u.shape[-1]), np.uint32)
    for c in range(n_chunks):
        seg = u[..., c * chunk:min((c + 1) * chunk, T), :]
        out[..., c, :] = (seg.sum(axis=-2, dtype=np.uint64) & 0xFFFFFFFF).astype(np.uint32)
    return out
