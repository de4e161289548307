"""Analytic order statistics of iid normal run-times (Section 3.1.1 of the paper).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  These are the paper's closed-form
companions of the Monte-Carlo estimate; the tests use them to pin the oracle's
sort / mean / argmax tail, and they are the "order" baseline of Section 4.3.
"""
from __future__ import annotations

import math

import numpy as np
from scipy import integrate, special, stats


def expected_order_statistic(n: int, j: int, mu: float = 0.0, sigma: float = 1.0) -> float:
    """E[x~_(j)] of n iid N(mu, sigma^2) draws, j = 1 (smallest) .. n (largest).

    The integral printed in Section 3.1.1: Z(n, j) * integral of
    x Phi(x)^(j-1) (1 - Phi(x))^(n-j) p(x) dx with Z(n, j) = n! / ((j-1)! (n-j)!).
    (The paper labels it p(x~_(j)); the integrand x * density makes it the mean.)
    Evaluated for the standard normal in log space, then shifted and scaled.
    """
    log_z = special.gammaln(n + 1) - special.gammaln(j) - special.gammaln(n - j + 1)

    def integrand(x):
        log_term = (j - 1) * stats.norm.logcdf(x) + (n - j) * stats.norm.logsf(x) + stats.norm.logpdf(x)
        return x * math.exp(log_z + log_term)

    value, _ = integrate.quad(integrand, -12.0, 12.0, epsabs=1e-13, epsrel=1e-12, limit=400)
    return mu + sigma * value


def elfving(n: int, j: int, mu: float = 0.0, sigma: float = 1.0) -> float:
    """Elfving's approximation, Eq. (elfving) of the paper, in its standard form.

    The printed fraction (n - pi/8) / (j - pi/4 + 1) exceeds 1 for most j, where
    the normal quantile does not exist; the standard form (Royston 1982) is
    (j - pi/8) / (n - pi/4 + 1).  For j = n -- the only case the paper evaluates
    -- both give the same number.
    """
    return mu + sigma * float(stats.norm.ppf((j - math.pi / 8.0) / (n - math.pi / 4.0 + 1.0)))


def mean_idle_time(n: int, mu: float, sigma: float) -> float:
    """Left side of Eq. (3): (1/n) sum_j E[x~_(n) - x~_(j)]."""
    e = np.array([expected_order_statistic(n, j, mu, sigma) for j in range(1, n + 1)])
    return float(np.mean(e[-1] - e))
