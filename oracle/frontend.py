"""Stable parameterisation of the recurrence's per-token quantities (test infrastructure only).

From raw, unconstrained inputs a, b, c and an unnormalised key, the paragraph "Stable parameterization" of
Section 3 (Eqs. "param-alpha", "param-theta", "param-beta", "param-key") builds

    alpha = alpha_min + (alpha_max - alpha_min) * sigmoid(a),      0 <= alpha_min <= alpha_max <= 1
    theta = theta_max * tanh(b)
    beta  = sigmoid(c)
    k     = k_raw / (||k_raw||_2 + eps)

so that ||Lambda|| <= 1, 0 <= beta <= 1 and ||k|| <= 1.  Plain float64 numpy, one line per equation; the norm of
the key runs over its d_k real channels, which is the norm of the complex key.
"""
import numpy as np


def sigmoid(x):
    x = np.asarray(x, dtype=np.float64)
    return 1.0 / (1.0 + np.exp(-x))


def stable_parameterisation(a, b, c, k_raw, alpha_min, alpha_max, theta_max, eps):
    """a, b: [..., m]; c: [...]; k_raw: [..., d_k].  Returns alpha, theta, beta, k in float64."""
    if not (0.0 <= alpha_min <= alpha_max <= 1.0):
        raise ValueError("need 0 <= alpha_min <= alpha_max <= 1")
    alpha = alpha_min + (alpha_max - alpha_min) * sigmoid(a)                      # Eq. "param-alpha"
    theta = theta_max * np.tanh(np.asarray(b, dtype=np.float64))                   # Eq. "param-theta"
    beta = sigmoid(c)                                                              # Eq. "param-beta"
    k_raw = np.asarray(k_raw, dtype=np.float64)
    k = k_raw / (np.linalg.norm(k_raw, axis=-1, keepdims=True) + eps)              # Eq. "param-key"
    return alpha, theta, beta, k
