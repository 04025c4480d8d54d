"""Proposal-depth selection (Sec. 5, Theorem 2) and the branch bound (Sec. 4.3)."""
import itertools

import numpy as np


def optimal_depths(alpha, beta, R):
    """Closed-form (d1*, d2*) of Theorem 2 / Eq. 8."""
    D = alpha * alpha + alpha + 1.0
    ab, tar = alpha * beta, 2.0 * alpha * R
    d1 = ab ** ((alpha + 1.0) / D) * tar ** (1.0 / D)
    d2 = ab ** (alpha / D) * tar ** ((alpha + 1.0) / D)
    return d1, d2


def expected_steps_bound(d1, d2, alpha, beta, R):
    """f(d1,d2) = d1 + beta d1^-alpha d2 + 2 beta d2^-alpha R, the bound on E[C] in the proof of Thm 2."""
    return d1 + beta * d1 ** (-alpha) * d2 + 2.0 * beta * d2 ** (-alpha) * R


def validity_bound(alpha, beta):
    """Right-hand side of Theorem 2's condition on R (the solution satisfies 1 <= d1* < d2* < R above it)."""
    ab = alpha * beta
    D = alpha * alpha + alpha + 1.0
    return max(ab ** (1 / alpha), ab ** (-alpha - 1), ab ** (1 / alpha) * (2 * alpha) ** (D / alpha ** 2)) / (2 * alpha)


def admissible_pairs(R):
    """Integer pairs allowed by App. B "Depth Configuration": 1 <= d1 < d2 < R, d1 | d2, d1 | R."""
    return [(a, b) for a, b in itertools.product(range(1, R), repeat=2)
            if a < b < R and b % a == 0 and R % a == 0]


def snap_depths(alpha, beta, R):
    """Reading (the paper gives no rounding rule): the admissible integer pair minimising f."""
    pairs = admissible_pairs(R)
    return min(pairs, key=lambda p: (expected_steps_bound(p[0], p[1], alpha, beta, R), p))


def max_branches(R, d1, d2):
    """B = sum_{k < R/d1} s_k with s_k = s_{k-1} + s_{k - d2/d1}, s_k = 1 for k < d2/d1 (Sec. 4.3).

    d2 = 0 means a single proposal: one new branch per interval, B = R/d1.
    """
    n = R // d1
    if d2 == 0:
        return n
    lag = d2 // d1
    s = []
    for k in range(n):
        s.append(1 if k < lag else s[k - 1] + s[k - lag])
    return sum(s)


def fit_envelope(tv):
    """Power-law envelope phi(r) = beta r^-alpha over empirical TV at r = 1..len(tv) (Sec. 4.1).

    Reading: minimise max_r phi(r)/TV(r) subject to phi(r) >= TV(r) for every r -- an LP in
    (log beta, alpha) on log TV, solved by enumerating vertex candidates (pairs of depths).
    """
    tv = np.asarray(tv, dtype=np.float64)
    r = np.arange(1, len(tv) + 1, dtype=np.float64)
    lr, lt = np.log(r), np.log(tv)
    best = None
    alphas = set()
    for i in range(len(tv)):
        for j in range(i + 1, len(tv)):
            alphas.add(-(lt[j] - lt[i]) / (lr[j] - lr[i]))
    for a in sorted(x for x in alphas if x > 0):
        # for a fixed slope the tightest feasible envelope touches the largest residual
        logb = np.max(lt + a * lr)
        worst = np.max(logb - a * lr - lt)
        if best is None or worst < best[0] - 1e-15:
            best = (worst, a, float(np.exp(logb)))
    if best is None:
        raise ValueError("TV must decrease somewhere for a positive exponent")
    return best[1], best[2]
