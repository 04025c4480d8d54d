"""Pins for the closed-form proposal depths (Thm 2), the envelope fit (Sec. 4.1) and the branch bound (Sec. 4.3)."""
import json
import os

import numpy as np
from scipy import optimize

from oracle import depths as dp

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def test_closed_form_reproduces_printed_values():
    for row in GOLD["closed_form_depths"]:
        d1, d2 = dp.optimal_depths(row["alpha"], row["beta"], row["R"])
        assert round(d1, 2) == row["d1"] and round(d2, 2) == row["d2"]
        assert row["R"] > dp.validity_bound(row["alpha"], row["beta"])
        # the paper gives no rounding rule; the admissible pair minimising the bound brackets the real
        # optimum and shares d2 with the pair the paper measured as best
        s1, s2 = dp.snap_depths(row["alpha"], row["beta"], row["R"])
        assert s1 in (int(d1), int(d1) + 1) and s2 == row["measured_best"][1]


def test_closed_form_is_the_minimiser_of_the_bound():
    rng = np.random.default_rng(0)
    for _ in range(20):
        a, b, R = rng.uniform(0.5, 2.0), rng.uniform(0.05, 0.5), int(rng.integers(8, 64))
        d1, d2 = dp.optimal_depths(a, b, R)
        f = lambda x: dp.expected_steps_bound(x[0], x[1], a, b, R)
        # both partial derivatives vanish (proof of Thm 2)
        assert abs(1 - a * b * d1 ** (-a - 1) * d2) < 1e-9
        assert abs(b * d1 ** (-a) - 2 * a * b * R * d2 ** (-a - 1)) < 1e-9
        res = optimize.minimize(f, [d1 * 1.3, d2 * 0.8], method="Nelder-Mead",
                                options=dict(xatol=1e-10, fatol=1e-14, maxiter=4000))
        np.testing.assert_allclose(res.x, [d1, d2], rtol=1e-5)


def test_closed_form_special_case():
    # alpha = 1, beta = 1/2, R = 16: D = 3, alpha*beta = 1/2, 2*alpha*R = 32 -> d1 = 2^(-2/3) 2^(5/3) = 2, d2 = 2^(-1/3) 2^(10/3) = 8
    d1, d2 = dp.optimal_depths(1.0, 0.5, 16)
    np.testing.assert_allclose([d1, d2], [2.0, 8.0], rtol=1e-14)


def test_validity_condition_brackets_the_solution():
    # just above the bound the solution obeys 1 <= d1* < d2* < R
    for a, b in [(1.03, 0.175), (1.08, 0.207), (0.7, 0.3), (1.5, 0.4)]:
        R = dp.validity_bound(a, b) * 1.001
        d1, d2 = dp.optimal_depths(a, b, R)
        assert 1 <= d1 < d2 < R
    # for R = 4 with the paper's Raven-like envelope the condition fails and d1* < 1
    assert 4 < dp.validity_bound(1.03, 0.175)
    assert dp.optimal_depths(1.03, 0.175, 4)[0] < 1
    assert dp.snap_depths(1.03, 0.175, 4) in [(1, 2), (1, 3)]


def test_admissible_pairs():
    assert dp.admissible_pairs(4) == [(1, 2), (1, 3)]
    assert (2, 8) in dp.admissible_pairs(32) and (2, 10) in dp.admissible_pairs(32)
    assert (3, 6) not in dp.admissible_pairs(32) and (2, 5) not in dp.admissible_pairs(32)


def test_branch_bound():
    for row in GOLD["branch_bound"]:
        assert dp.max_branches(row["R"], row["d1"], row["d2"]) == row["B"]
    assert dp.max_branches(4, 1, 2) == 7           # s = 1, 1, 2, 3
    assert dp.max_branches(4, 1, 0) == 4
    assert dp.max_branches(16, 2, 8) == 18


def test_envelope_fit_recovers_a_power_law_and_bounds_from_above():
    r = np.arange(1, 11)
    a, b = dp.fit_envelope(0.2 * r ** -1.1)
    np.testing.assert_allclose([a, b], [1.1, 0.2], rtol=1e-9)
    rng = np.random.default_rng(1)
    tv = 0.2 * r ** -1.1 * rng.uniform(0.7, 1.0, len(r))
    a, b = dp.fit_envelope(tv)
    phi = b * r ** -a
    assert (phi >= tv * (1 - 1e-12)).all()
    worst = (phi / tv).max()
    # no other (alpha, beta) on a fine grid has a smaller maximum ratio while staying above
    for aa in np.linspace(0.5, 2.0, 151):
        bb = (tv * r ** aa).max()
        assert (bb * r ** -aa / tv).max() >= worst - 1e-9
