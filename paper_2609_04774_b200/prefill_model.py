"""Cache-aware prefill-time model of the paper (Section 3.2, Eq. 2) fitted to this library's measured
prefill-time table, and the request placement cost that consumes it (Section 5.3).  Host-side
arithmetic only (numpy); the measurements come from ``bench.py --mode table``.

    E_C(R, P) = d + a R + b P + (c R + alpha W(R, P)) / C,     W(R, P) = R P + R (R + 1) / 2   (Eq. 1)

For an attention-only measurement ``a`` (communication, synchronisation) and ``c`` (token-local
projection / feed-forward) have nothing to describe; the fit is non-negative least squares, so they
come out at or near zero instead of absorbing noise with a negative sign.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def remaining_workload(R, P):
    """Eq. (1): visible (query, key) pairs left after a prefix hit."""
    R = np.asarray(R, dtype=np.float64)
    P = np.asarray(P, dtype=np.float64)
    return R * P + R * (R + 1.0) / 2.0


@dataclass
class PrefillModel:
    d: float      # fixed start-up overhead
    a: float      # per uncached token, not divided by C
    b: float      # per cached token (prefix access and replay)
    c: float      # per uncached token, divided by C
    alpha: float  # per visible (query, key) pair, divided by C

    def predict(self, R, P, C):
        """Eq. (2)."""
        R = np.asarray(R, dtype=np.float64)
        P = np.asarray(P, dtype=np.float64)
        C = np.asarray(C, dtype=np.float64)
        return self.d + self.a * R + self.b * P + (self.c * R + self.alpha * remaining_workload(R, P)) / C


def _nnls(A: np.ndarray, y: np.ndarray, iters: int = 20000) -> np.ndarray:
    """Non-negative least squares by projected gradient on column-scaled A (small problems only)."""
    scale = np.maximum(np.abs(A).max(axis=0), 1e-300)
    As = A / scale
    x = np.zeros(A.shape[1])
    L = np.linalg.norm(As, 2) ** 2
    for _ in range(iters):
        g = As.T @ (As @ x - y)
        x_new = np.maximum(x - g / L, 0.0)
        if np.abs(x_new - x).max() <= 1e-15 * max(1.0, np.abs(x).max()):
            x = x_new
            break
        x = x_new
    return x / scale


def fit(R, P, C, t, relative: bool = True) -> PrefillModel:
    """Fit (d, a, b, c, alpha) >= 0 of Eq. (2) to measured times t(R, P, C).  With ``relative`` every
    sample is weighted by 1/t, so that microsecond and second scale measurements count alike."""
    R = np.asarray(R, dtype=np.float64)
    P = np.asarray(P, dtype=np.float64)
    C = np.asarray(C, dtype=np.float64)
    t = np.asarray(t, dtype=np.float64)
    A = np.stack([np.ones_like(R), R, P, R / C, remaining_workload(R, P) / C], axis=1)
    if relative:
        A = A / t[:, None]
        t = np.ones_like(t)
    try:
        from scipy.optimize import nnls
        coef, _ = nnls(A / np.abs(A).max(axis=0), t)
        coef = coef / np.abs(A).max(axis=0)
    except Exception:
        coef = _nnls(A, t)
    return PrefillModel(*[float(x) for x in coef])


def placement_cost(queue_delay, service, C_w, service_at_cmin, C_min, beta=1.0, lam=0.0):
    """Section 5.3:  J = q_w + beta * s + lambda * (C_w * s - C_min * E_{C_min}), with s the predicted
    service time at the worker's degree and E_{C_min} the prediction at the smallest eligible degree
    under the same prefix reuse."""
    return queue_delay + beta * service + lam * (C_w * service - C_min * service_at_cmin)


def choose_worker(model: PrefillModel, workers, beta=1.0, lam=0.0):
    """workers: iterable of dicts {C, R, P, queue_delay}; returns (index of the minimum-cost worker, costs)."""
    workers = list(workers)
    c_min = min(w["C"] for w in workers)
    costs = []
    for w in workers:
        s = float(model.predict(w["R"], w["P"], w["C"]))
        s_min = float(model.predict(w["R"], w["P"], c_min))
        costs.append(placement_cost(w.get("queue_delay", 0.0), s, w["C"], s_min, c_min, beta, lam))
    return int(np.argmin(costs)), costs
