"""The entropy law of draftability (Section 4, Eq. 2), fitted on a round log.  Host-side analysis, numpy only.

    logit p_m(H) = b0 - b1 * H,        E[a | H] = sum_{l=1..L} p_m^l = p_m (1 - p_m^L) / (1 - p_m)

A round log is a list of (H, a): the target's root entropy in nats (written by the verify pass when
`glance_log_root_entropy` is set) and the accepted length.  The paper says the two constants are fitted on each
task's round log without naming the estimator; the reading here is the maximum-likelihood fit of the survival model
the law is derived from: given H the accepted run is a geometric run of matches with per-step probability p_m(H),
cut at the horizon L, so a round contributes `a` matches and one miss unless it reached L,

    log-likelihood = sum_rounds [ a * log p_m(H) + 1[a < L] * log(1 - p_m(H)) ].

This is a weighted logistic regression; it is concave and solved by Newton's method.
"""
from typing import Sequence, Tuple

import numpy as np


def match_probability(H, b0: float, b1: float):
    """p_m(H) = sigmoid(b0 - b1 H)."""
    return 1.0 / (1.0 + np.exp(-(b0 - b1 * np.asarray(H, dtype=np.float64))))


def expected_accept(H, b0: float, b1: float, L: int):
    """Eq. 2: E[a | H] = sum_{l=1..L} p_m(H)^l."""
    p = match_probability(H, b0, b1)
    return sum(p ** l for l in range(1, L + 1))


def fit_law(H: Sequence[float], a: Sequence[int], L: int, iters: int = 50) -> Tuple[float, float]:
    """Maximum-likelihood (b0, b1) of the truncated-geometric survival model on a round log."""
    H = np.asarray(H, dtype=np.float64)
    a = np.asarray(a, dtype=np.float64)
    assert H.shape == a.shape and H.size >= 2
    succ = a                                  # matches in the round
    fail = (a < L).astype(np.float64)         # the miss that ended it, unless the horizon did
    X = np.stack([np.ones_like(H), -H], axis=1)          # logit = X @ (b0, b1)
    beta = np.zeros(2)
    for _ in range(iters):
        p = 1.0 / (1.0 + np.exp(-(X @ beta)))
        grad = X.T @ (succ * (1.0 - p) - fail * p)
        w = (succ + fail) * p * (1.0 - p)
        hess = (X * w[:, None]).T @ X + 1e-12 * np.eye(2)
        step = np.linalg.solve(hess, grad)
        beta = beta + step
        if float(np.abs(step).max()) < 1e-10:
            break
    return float(beta[0]), float(beta[1])
