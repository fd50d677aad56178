"""CPU oracle of the throughput-model fit (test infrastructure only).

Sec. 4.1: theta_sys is fitted by minimising the root mean squared logarithmic error between
Eq. 11 and the observed (a, m, s, T_iter) tuples with L-BFGS-B, alpha and beta non-negative,
gamma in [1, 10].  Here: the objective in plain numpy (fp64) and scipy's L-BFGS-B as the
minimiser.  RMSLE is read in its textbook form sqrt(mean((ln(1 + pred) - ln(1 + obs))^2)).
"""
from __future__ import annotations

import numpy as np
import scipy.optimize as so

NUM_PARAMS = 7  # alpha_grad, beta_grad, alpha_local, beta_local, alpha_node, beta_node, gamma


def t_iter(theta, K, N, m, s):
    """Eq. 8-11 for arrays of observations."""
    a_g, b_g, a_l, b_l, a_n, b_n, gamma = (float(x) for x in theta)
    K = np.asarray(K, dtype=np.float64); N = np.asarray(N); m = np.asarray(m, dtype=np.float64)
    s = np.asarray(s, dtype=np.float64)
    tg = a_g + b_g * m                                                        # Eq. 8
    ts = np.where(K <= 1, 0.0, np.where(N == 1, a_l + b_l * (K - 2), a_n + b_n * (K - 2)))   # Eq. 9
    with np.errstate(divide="ignore", invalid="ignore"):
        both = (tg > 0) & (ts > 0)
        ov = np.where(both, (np.where(both, tg, 1.0) ** gamma + np.where(both, ts, 1.0) ** gamma) ** (1.0 / gamma),
                      np.maximum(tg, ts))                                     # Eq. 10
    return s * tg + ov                                                        # Eq. 11


def rmsle(theta, K, N, m, s, T):
    p = t_iter(theta, K, N, m, s)
    r = np.log1p(p) - np.log1p(np.asarray(T, dtype=np.float64))
    return float(np.sqrt(np.mean(r * r))) if r.size else 0.0


def fit(K, N, m, s, T, theta0, frozen: int = 0, maxiter: int = 500):
    """L-BFGS-B from theta0 (clamped into the bounds); bit i of `frozen` pins parameter i."""
    lb = np.array([0.0] * 6 + [1.0]); ub = np.array([np.inf] * 6 + [10.0])
    x0 = np.clip(np.asarray(theta0, dtype=np.float64), lb, ub)
    bounds = []
    for i in range(NUM_PARAMS):
        if (frozen >> i) & 1:
            x0[i] = float(theta0[i])
            bounds.append((x0[i], x0[i]))
        else:
            bounds.append((lb[i], None if np.isinf(ub[i]) else ub[i]))
    if len(T) == 0:
        return x0, 0.0
    res = so.minimize(lambda th: rmsle(th, K, N, m, s, T), x0, method="L-BFGS-B", bounds=bounds,
                      options={"maxiter": maxiter, "ftol": 1e-15, "gtol": 1e-10})
    return res.x, float(res.fun)
