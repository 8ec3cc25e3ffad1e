"""Host-side entropy-law fit (Section 4, Eq. 2): closed forms, printed values, parameter recovery."""
import math
import os

import numpy as np

from paper_2609_00355_b200 import entropy_law as E


def test_expected_accept_is_the_truncated_geometric_sum():
    for b0, b1, H, L in ((1.226, 0.63, 0.0, 15), (0.96, 0.63, 1.3, 15), (0.2, 0.4, 2.0, 7)):
        p = 1.0 / (1.0 + math.exp(-(b0 - b1 * H)))
        closed = p * (1.0 - p ** L) / (1.0 - p)
        assert abs(float(E.expected_accept(H, b0, b1, L)) - closed) < 1e-12
    # strictly decreasing in H for b1 > 0
    vals = [float(E.expected_accept(h, 0.96, 0.63, 15)) for h in np.linspace(0, 6, 13)]
    assert all(x > y for x, y in zip(vals, vals[1:]))


def test_printed_values_of_the_law():
    """Values the paper prints for the law at b0 = 1.226 (zero entropy): the truncated mean and the cap e^{b0}."""
    path = os.path.join(os.path.dirname(__file__), "golden", "eq2_printed_values.txt")
    seen = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        kind, arg, L, val, dec = line.split()
        arg, L, val, dec = float(arg), int(L), float(val), int(dec)
        if kind == "sup_mean":
            assert round(float(E.expected_accept(0.0, arg, 0.63, L)), dec) == val
            seen += 1
        elif kind == "geo_cap":
            p = float(E.match_probability(0.0, arg, 0.63))
            assert round(p / (1.0 - p), dec) == val and round(math.exp(arg), dec) == val
            seen += 1
    assert seen == 2


def test_fit_recovers_the_parameters_of_a_synthetic_round_log():
    rng = np.random.default_rng(0)
    b0, b1, L, n = 0.96, 0.63, 15, 40000
    H = rng.uniform(0.0, 5.0, size=n)
    p = E.match_probability(H, b0, b1)
    a = np.zeros(n, dtype=np.int64)
    alive = np.ones(n, dtype=bool)
    for _ in range(L):
        alive &= rng.random(n) < p
        a += alive
    f0, f1 = E.fit_law(H, a, L)
    assert abs(f0 - b0) < 0.05 and abs(f1 - b1) < 0.03
    # the fitted law reproduces the mean accepted length of the log, bin by bin
    for lo in (0.0, 2.0, 4.0):
        m = (H >= lo) & (H < lo + 1.0)
        assert abs(float(E.expected_accept(H[m], f0, f1, L).mean()) - a[m].mean()) < 0.05
