"""Evaluation of cutoff rules on observed run-times (Sections 3, 3.1.1 and 4.1 of the paper).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  Plain, slow, double-precision statements of the
quantities Fig. 2 plots for every SGD iteration of a recorded trace:

  * the throughput a cutoff c achieves on the run-times that were actually observed,
    Omega(c) = c / x~_(c) with x~ the observed run-times in ascending order (Section 3);
  * the ground-truth maximum max_c Omega(c) and the cutoff that attains it ("oracle" in
    Fig. 2: known only in hindsight);
  * the throughput of waiting for all workers, N / x~_(N) (fully synchronous SGD);
  * a static cutoff, the same c at every iteration (Chen et al. 2016, cited in Section 1);
  * the "order" baseline of Fig. 4: the cutoff that maximises c / E[x~_(c)] when the expected
    order statistics come from Elfving's formula (Section 3.1.1) with the mean and standard
    deviation of all run-times observed so far.

Pins (tests/test_oracle_evaluation.py): brute force over every c on small vectors, the worked
example of Section 4.1 (158 workers, mean 1.057 s, deviation 0.393 s: expected maximum
2.1063 s), equal run-times, hand-made vectors with stragglers, and the running moments against
numpy on the concatenated history.
"""
from __future__ import annotations

import math

import numpy as np
from scipy import stats


def achieved_throughput(observed: np.ndarray, c: int) -> float:
    """Omega(c) = c / x~_(c): c gradients arrive after the c-th smallest observed run-time."""
    ordered = np.sort(np.asarray(observed, dtype=np.float64), kind="stable")
    return float(c) / float(ordered[c - 1])


def hindsight_best(observed: np.ndarray):
    """(c*, Omega(c*)): the cutoff that would have maximised the throughput of this step; ties -> larger c."""
    ordered = np.sort(np.asarray(observed, dtype=np.float64), kind="stable")
    best, arg = -math.inf, ordered.shape[0]
    for c in range(1, ordered.shape[0] + 1):
        omega = c / ordered[c - 1]
        if omega >= best:
            best, arg = omega, c
    return arg, best


def wait_for_all(observed: np.ndarray) -> float:
    """N / x~_(N): every worker's gradient is used, the step lasts as long as the slowest worker."""
    x = np.asarray(observed, dtype=np.float64)
    return float(x.shape[0]) / float(x.max())


def elfving_expected(n: int, mu: float, sigma: float) -> np.ndarray:
    """E[x~_(j)], j = 1..n, of n iid N(mu, sigma^2) run-times by Elfving's formula (Section 3.1.1).

    The fraction is taken in its standard form (j - pi/8) / (n - pi/4 + 1); the printed one exceeds 1
    for most j, where the normal quantile does not exist, and agrees with this one for j = n.
    """
    j = np.arange(1, n + 1, dtype=np.float64)
    return mu + sigma * stats.norm.ppf((j - math.pi / 8.0) / (n - math.pi / 4.0 + 1.0))


def cutoff_from_expected(expected: np.ndarray) -> int:
    """argmax_c c / E[x~_(c)] over c = 1..N with E > 0; ties -> larger c; c = N if no c is admissible."""
    best, arg = -math.inf, expected.shape[0]
    for c in range(1, expected.shape[0] + 1):
        if expected[c - 1] > 0.0:
            omega = c / expected[c - 1]
            if omega >= best:
                best, arg = omega, c
    return arg


def order_cutoffs(trace: np.ndarray) -> np.ndarray:
    """The "order" baseline for every step t of a trace [T, N].

    The cutoff of step t is set before its run-times are known, from the mean and the (population)
    standard deviation of every run-time observed in steps 0 .. t-1; step 0 has nothing to go on and
    waits for all workers.
    """
    x = np.asarray(trace, dtype=np.float64)
    T, N = x.shape
    out = np.empty(T, dtype=np.int64)
    out[0] = N
    for t in range(1, T):
        seen = x[:t].reshape(-1)
        mu = float(seen.mean())
        sigma = math.sqrt(max(float((seen * seen).mean()) - mu * mu, 0.0))
        out[t] = cutoff_from_expected(elfving_expected(N, mu, sigma))
    return out


def best_static_cutoff(trace: np.ndarray) -> int:
    """The single c that maximises the total throughput sum_t c / x~_(c)(t) of a trace; ties -> larger c."""
    ordered = np.sort(np.asarray(trace, dtype=np.float64), axis=1, kind="stable")
    T, N = ordered.shape
    best, arg = -math.inf, N
    for c in range(1, N + 1):
        total = float((c / ordered[:, c - 1]).sum())
        if total >= best:
            best, arg = total, c
    return arg


def evaluate(trace: np.ndarray, cutoffs: dict) -> dict:
    """Per-step scores of cutoff rules on a trace [T, N] (the quantities of Fig. 2).

    cutoffs maps a rule's name to its cutoffs, one per step (or a single integer: a static cutoff).
    Returns a dictionary of arrays of length T: "best_c", "best" (hindsight), "all" (wait for all), and for
    every rule "<name>" (achieved throughput) and "<name>_time" (seconds the step lasts, x~_(c)).
    """
    x = np.asarray(trace, dtype=np.float64)
    T, N = x.shape
    out = {"best_c": np.empty(T, dtype=np.int64), "best": np.empty(T), "all": np.empty(T)}
    for t in range(T):
        out["best_c"][t], out["best"][t] = hindsight_best(x[t])
        out["all"][t] = wait_for_all(x[t])
    for name, cs in cutoffs.items():
        cs = np.broadcast_to(np.asarray(cs, dtype=np.int64), (T,))
        out[name] = np.array([achieved_throughput(x[t], int(cs[t])) for t in range(T)])
        out[name + "_time"] = np.array([np.sort(x[t], kind="stable")[int(cs[t]) - 1] for t in range(T)])
    return out
