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


def stable_parameterisation_backward(a, b, c, k_raw, alpha_min, alpha_max, theta_max, eps, dalpha, dtheta, dbeta, dk):
    """Gradients of a loss with respect to the raw inputs, given its gradients with respect to alpha, theta, beta, k:

        da = dalpha (alpha_max - alpha_min) sigmoid(a) (1 - sigmoid(a))         db = dtheta theta_max (1 - tanh(b)^2)
        dc = dbeta sigmoid(c) (1 - sigmoid(c))
        dk_raw = s dk - s^2 (dk . k_raw) k_raw / n,    n = ||k_raw||_2,  s = 1 / (n + eps)

    (the derivative of k = s k_raw, with ds/dk_raw = -s^2 k_raw / n; a zero key, where the norm is not
    differentiable, takes the one-sided value s dk).  float64 numpy, one line per equation."""
    sa, sc = sigmoid(a), sigmoid(c)
    da = np.asarray(dalpha, dtype=np.float64) * (alpha_max - alpha_min) * sa * (1.0 - sa)
    db = np.asarray(dtheta, dtype=np.float64) * theta_max * (1.0 - np.tanh(np.asarray(b, dtype=np.float64)) ** 2)
    dc = np.asarray(dbeta, dtype=np.float64) * sc * (1.0 - sc)
    k_raw, dk = np.asarray(k_raw, dtype=np.float64), np.asarray(dk, dtype=np.float64)
    n = np.linalg.norm(k_raw, axis=-1, keepdims=True)
    s = 1.0 / (n + eps)
    dot = np.sum(dk * k_raw, axis=-1, keepdims=True)
    unit = np.divide(k_raw, n, out=np.zeros_like(k_raw), where=n > 0)
    dk_raw = s * dk - s * s * dot * unit
    return da, db, dc, dk_raw
