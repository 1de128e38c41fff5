"""Seeded synthetic inputs for the five workload configurations.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only draws random tensors with the shapes
and value distributions the configurations name, and rounds to bfloat16 where
the configuration stores bf16.  numpy only.

Recipe (every stream is ``numpy.random.default_rng([seed, *key])``, PCG64):

* forward configs: one stream per batch element ``b`` (key ``(b,)``) drawn in the
  fixed order q, k, v, beta, alpha, theta, S0, each with shape ``[T, H, ...]``
  (S0: ``[H, d_k, d_v]``), float32 draws; k is L2-normalised over its d_k real
  channels (= the complex norm) in float32 *before* bf16 rounding.
* config 3 draws its per-(head, pair) modulus p from the stream with key
  ``(10**6,)``; p is fixed over time and over the batch.
* raw inputs of the stable parameterisation (``forward_raw_*``): one stream per batch element with key
  ``(7 * 10**6 + b,)`` drawn in the order q, k_raw, key scale, v, a_raw, b_raw, c_raw, S0: a_raw ~ N(3, 1)
  (so that alpha_min = 0, alpha_max = 1 reproduces the "sigmoid(n(3,1))" decay of the forward configs),
  b_raw ~ N(0, 1.5), c_raw ~ N(0, 1), k_raw = N(0, 1) times a log-normal scale exp(N(0, 0.5)) per token and
  head (unnormalised keys of varying length).  Nothing is transformed here.
* decode config: S0 from key ``(2**20,)``; step ``s`` from key ``(s,)`` in the order
  q, k, v, beta, alpha, theta with shape ``[B, H, ...]``.
"""
import os
from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Config:
    name: str
    B: int
    T: int
    H: int
    d_k: int
    d_v: int
    chunk: int
    dtype: str            # "f32" or "bf16": storage type of q, k, v, o
    alpha: str            # "u(0.9,1)", "sigmoid(n(3,1))", "u(0.999,1)"
    theta: str            # "u(-pi,pi)", "quantised"
    beta: str             # "u(0,1)", "sigmoid(n(0,1))", "bernoulli(0.05)"
    s0_std: float         # 0 -> zero initial state
    seed: int
    steps: int = 0        # decode only

    @property
    def m(self):
        return self.d_k // 2

    def scaled(self, **kw):
        """Same distributions at other sizes (for tests)."""
        return replace(self, **kw)


CONFIGS = [
    Config("cfg0_tiny_fp32", 1, 256, 2, 64, 64, 16, "f32", "u(0.9,1)", "u(-pi,pi)", "u(0,1)", 0.0, 0),
    Config("cfg1_bf16_4k", 4, 4096, 16, 128, 128, 64, "bf16", "sigmoid(n(3,1))", "u(-pi,pi)", "sigmoid(n(0,1))", 0.0, 1),
    Config("cfg2_headline", 8, 8192, 32, 128, 128, 64, "bf16", "sigmoid(n(3,1))", "u(-pi,pi)", "sigmoid(n(0,1))", 0.02, 2),
    Config("cfg3_long_context", 1, 131072, 16, 128, 128, 64, "bf16", "u(0.999,1)", "quantised", "bernoulli(0.05)", 0.0, 3),
    Config("cfg4_decode", 256, 1, 32, 128, 128, 64, "bf16", "sigmoid(n(3,1))", "u(-pi,pi)", "sigmoid(n(0,1))", 0.02, 4,
           steps=1024),
]


def bf16_round(x):
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    bias = ((bits >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((bits + bias) & np.uint32(0xFFFF0000)).view(np.float32)
    return out.reshape(x.shape)


def _sigmoid(x):
    return (1.0 / (1.0 + np.exp(-x.astype(np.float64)))).astype(np.float32)


def _store(cfg, x):
    return bf16_round(x) if cfg.dtype == "bf16" else x.astype(np.float32)


def _draw_alpha(cfg, rng, shape):
    if cfg.alpha == "u(0.9,1)":
        return rng.uniform(0.9, 1.0, shape).astype(np.float32)
    if cfg.alpha == "u(0.999,1)":
        return rng.uniform(0.999, 1.0, shape).astype(np.float32)
    if cfg.alpha == "sigmoid(n(3,1))":
        return _sigmoid(3.0 + rng.standard_normal(shape, dtype=np.float32))
    if cfg.alpha.startswith("u("):               # "u(lo,hi)" for edge-case tests
        lo, hi = (float(t) for t in cfg.alpha[2:-1].split(","))
        return rng.uniform(lo, hi, shape).astype(np.float32)
    raise ValueError(cfg.alpha)


def _draw_beta(cfg, rng, shape):
    if cfg.beta == "u(0,1)":
        return rng.uniform(0.0, 1.0, shape).astype(np.float32)
    if cfg.beta == "sigmoid(n(0,1))":
        return _sigmoid(rng.standard_normal(shape, dtype=np.float32))
    if cfg.beta == "bernoulli(0.05)":
        return (rng.uniform(0.0, 1.0, shape) < 0.05).astype(np.float32)
    raise ValueError(cfg.beta)


def moduli(cfg):
    """Per-(head, pair) modulus p in {2,3,5,7} of the quantised-phase configuration."""
    rng = np.random.default_rng([cfg.seed, 10 ** 6])
    return rng.choice(np.array([2, 3, 5, 7]), size=(cfg.H, cfg.m))


def _draw_theta(cfg, rng, shape):
    if cfg.theta == "u(-pi,pi)":
        return rng.uniform(-np.pi, np.pi, shape).astype(np.float32)
    if cfg.theta == "zero":
        return np.zeros(shape, np.float32)
    if cfg.theta == "quantised":
        p = moduli(cfg)                                    # [H, m], broadcast over leading axes
        j = np.floor(rng.uniform(0.0, 1.0, shape) * p).astype(np.int64)
        j = np.minimum(j, p - 1)
        th = 2.0 * np.pi * j / p
        th = np.where(th > np.pi, th - 2.0 * np.pi, th)    # wrap to (-pi, pi]
        return th.astype(np.float32)
    raise ValueError(cfg.theta)


def _unit_keys(k):
    n = np.sqrt(np.sum(k.astype(np.float32) ** 2, axis=-1, keepdims=True, dtype=np.float32))
    return (k / n).astype(np.float32)


def forward_batch_element(cfg, b):
    """Inputs of batch element b: dict of float32 arrays q,k [T,H,d_k], v [T,H,d_v],
    beta [T,H], alpha, theta [T,H,m], S0 [H,d_k,d_v] or None.  q, k, v hold values that are
    exactly representable in cfg.dtype."""
    rng = np.random.default_rng([cfg.seed, b])
    T, H = cfg.T, cfg.H
    q = _store(cfg, rng.standard_normal((T, H, cfg.d_k), dtype=np.float32))
    k = _store(cfg, _unit_keys(rng.standard_normal((T, H, cfg.d_k), dtype=np.float32)))
    v = _store(cfg, rng.standard_normal((T, H, cfg.d_v), dtype=np.float32))
    beta = _draw_beta(cfg, rng, (T, H))
    alpha = _draw_alpha(cfg, rng, (T, H, cfg.m))
    theta = _draw_theta(cfg, rng, (T, H, cfg.m))
    S0 = None
    if cfg.s0_std > 0:
        S0 = (cfg.s0_std * rng.standard_normal((H, cfg.d_k, cfg.d_v), dtype=np.float32)).astype(np.float32)
    return dict(q=q, k=k, v=v, beta=beta, alpha=alpha, theta=theta, S0=S0)


def forward_inputs(cfg, batch=None):
    """Stack batch elements (all of them by default) into [B, T, H, ...] arrays."""
    bs = list(range(cfg.B) if batch is None else batch)
    if len(bs) > 1 and cfg.T * cfg.H >= 1 << 16:     # big tensors: numpy's generators release the GIL
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=min(len(bs), os.cpu_count() or 1)) as pool:
            parts = list(pool.map(lambda b: forward_batch_element(cfg, b), bs))
    else:
        parts = [forward_batch_element(cfg, b) for b in bs]
    out = {}
    for key in parts[0]:
        out[key] = None if parts[0][key] is None else np.stack([p[key] for p in parts])
    return out


def forward_raw_batch_element(cfg, b):
    """Raw (unconstrained) inputs of batch element b: q, k_raw [T,H,d_k], v [T,H,d_v], a_raw, b_raw [T,H,m],
    c_raw [T,H], S0 or None.  q, k_raw, v hold values exactly representable in cfg.dtype."""
    rng = np.random.default_rng([cfg.seed, 7 * 10 ** 6 + b])
    T, H = cfg.T, cfg.H
    q = _store(cfg, rng.standard_normal((T, H, cfg.d_k), dtype=np.float32))
    k_raw = rng.standard_normal((T, H, cfg.d_k), dtype=np.float32)
    scale = np.exp(0.5 * rng.standard_normal((T, H, 1), dtype=np.float32))
    k_raw = _store(cfg, k_raw * scale)
    v = _store(cfg, rng.standard_normal((T, H, cfg.d_v), dtype=np.float32))
    a_raw = (3.0 + rng.standard_normal((T, H, cfg.m), dtype=np.float32)).astype(np.float32)
    b_raw = (1.5 * rng.standard_normal((T, H, cfg.m), dtype=np.float32)).astype(np.float32)
    c_raw = rng.standard_normal((T, H), dtype=np.float32)
    S0 = None
    if cfg.s0_std > 0:
        S0 = (cfg.s0_std * rng.standard_normal((H, cfg.d_k, cfg.d_v), dtype=np.float32)).astype(np.float32)
    return dict(q=q, k_raw=k_raw, v=v, a_raw=a_raw, b_raw=b_raw, c_raw=c_raw, S0=S0)


def forward_raw_inputs(cfg, batch=None):
    """Stack raw batch elements (all of them by default) into [B, T, H, ...] arrays."""
    bs = list(range(cfg.B) if batch is None else batch)
    if len(bs) > 1 and cfg.T * cfg.H >= 1 << 16:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=min(len(bs), os.cpu_count() or 1)) as pool:
            parts = list(pool.map(lambda b: forward_raw_batch_element(cfg, b), bs))
    else:
        parts = [forward_raw_batch_element(cfg, b) for b in bs]
    out = {}
    for key in parts[0]:
        out[key] = None if parts[0][key] is None else np.stack([p[key] for p in parts])
    return out


def decode_initial_state(cfg):
    rng = np.random.default_rng([cfg.seed, 2 ** 20])
    return (cfg.s0_std * rng.standard_normal((cfg.B, cfg.H, cfg.d_k, cfg.d_v), dtype=np.float32)).astype(np.float32)


def decode_step_inputs(cfg, step):
    """Inputs of decode step `step`: q,k [B,H,d_k], v [B,H,d_v], beta [B,H], alpha, theta [B,H,m]."""
    rng = np.random.default_rng([cfg.seed, step])
    B, H = cfg.B, cfg.H
    q = _store(cfg, rng.standard_normal((B, H, cfg.d_k), dtype=np.float32))
    k = _store(cfg, _unit_keys(rng.standard_normal((B, H, cfg.d_k), dtype=np.float32)))
    v = _store(cfg, rng.standard_normal((B, H, cfg.d_v), dtype=np.float32))
    beta = _draw_beta(cfg, rng, (B, H))
    alpha = _draw_alpha(cfg, rng, (B, H, cfg.m))
    theta = _draw_theta(cfg, rng, (B, H, cfg.m))
    return dict(q=q, k=k, v=v, beta=beta, alpha=alpha, theta=theta)


def sequences(inputs, pairs):
    """Pick (b, h) pairs out of [B,T,H,...] inputs -> [N,T,...] float64 arrays for the oracle."""
    sel = {}
    for key in ("q", "k", "v", "alpha", "theta"):
        sel[key] = np.stack([inputs[key][b, :, h] for b, h in pairs]).astype(np.float64)
    sel["beta"] = np.stack([inputs["beta"][b, :, h] for b, h in pairs]).astype(np.float64)
    sel["S0"] = None if inputs["S0"] is None else \
        np.stack([inputs["S0"][b, h] for b, h in pairs]).astype(np.float64)
    return sel
