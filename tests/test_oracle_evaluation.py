"""Pins for the oracle's evaluation of cutoff rules (Sections 3, 3.1.1 and 4.1; Fig. 2 and Fig. 4).

Nothing here calls the functions under test to produce its expected values: they come from the paper's
text, from hand-worked vectors, from brute force written a second time with Python's own sort, from the
order-statistic integral, and from numpy on the concatenated history.
"""
import math
import os

import numpy as np

from oracle import evaluation as E
from oracle import iid_normal as A
from paper_1803_04209_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    vals = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    return vals


def test_the_straggler_example_of_section_3():
    # "if the slowest straggler takes 10 seconds to finish, but the second slowest takes 8, then there is
    # already a 20% reduction in the wall-clock time simply by setting the cutoff to n - 1"
    x = np.array([3.0, 8.0, 5.0, 10.0, 4.0])
    r = E.evaluate(x[None, :], {"all_but_one": 4, "everyone": 5})
    assert r["everyone_time"][0] == 10.0 and r["all_but_one_time"][0] == 8.0
    assert math.isclose(1.0 - r["all_but_one_time"][0] / r["everyone_time"][0], 0.20)
    assert math.isclose(r["everyone"][0], 5 / 10.0) and math.isclose(r["all"][0], 5 / 10.0)
    assert math.isclose(r["all_but_one"][0], 4 / 8.0)


def test_hand_worked_vectors():
    # three fast workers and one ten times slower: drop the straggler
    assert E.hindsight_best(np.array([1.0, 10.0, 1.0, 1.0])) == (3, 3.0)
    assert E.wait_for_all(np.array([1.0, 10.0, 1.0, 1.0])) == 0.4
    assert E.achieved_throughput(np.array([1.0, 10.0, 1.0, 1.0]), 1) == 1.0
    # run-times proportional to their rank: every c gives the same throughput, the tie goes to the largest c
    assert E.hindsight_best(np.array([0.5, 1.0, 1.5, 2.0])) == (4, 2.0)
    # equal run-times: waiting for everyone is optimal
    c, om = E.hindsight_best(np.full(7, 0.25))
    assert (c, om) == (7, 28.0)
    assert E.wait_for_all(np.full(7, 0.25)) == 28.0


def test_hindsight_best_against_brute_force_with_pythons_sort():
    rng = np.random.default_rng(0)
    for n in (1, 2, 3, 8, 33, 158):
        for _ in range(10):
            x = rng.lognormal(0.0, 0.6, size=n)
            ordered = sorted(float(v) for v in x)
            omegas = [(c + 1) / ordered[c] for c in range(n)]
            top = max(omegas)
            want_c = max(c + 1 for c in range(n) if omegas[c] == top)
            c, om = E.hindsight_best(x)
            assert c == want_c and om == top
            assert E.wait_for_all(x) == n / ordered[-1]
            for cc in (1, (n + 1) // 2, n):
                assert E.achieved_throughput(x, cc) == cc / ordered[cc - 1]
            assert om >= E.wait_for_all(x)


def test_elfving_reproduces_the_worked_example_of_section_4_1():
    g = _golden("paper_worked_example.txt")
    n = int(g["n_workers"])
    e = E.elfving_expected(n, g["mean_sec"], g["std_sec"])
    assert abs(e[-1] - g["expected_max_sec"]) < 2e-3           # 2.1063 s (printed inputs are rounded)
    assert abs((e[-1] - g["mean_sec"]) - g["mean_idle_sec"]) < 2e-3   # Eq. 3: idle = E[max] - middle = 1.049 s
    assert np.all(np.diff(e) > 0)                              # E[x~_(1)] <= ... <= E[x~_(n)]
    assert np.allclose(e + e[::-1], 2 * g["mean_sec"], atol=1e-12)    # symmetric around the mean


def test_elfving_follows_the_order_statistic_integral():
    for n in (2, 16, 158):
        e = E.elfving_expected(n, 0.0, 1.0)
        for j in sorted({1, 2, n // 2, n - 1, n} - {0}):
            exact = A.expected_order_statistic(n, j)
            assert abs(e[j - 1] - exact) < (0.04 if n == 2 else 0.02)   # the approximation's accuracy (worst for tiny n and at the ends)
    e = E.elfving_expected(16, 3.0, 0.5)
    assert np.allclose(e, 3.0 + 0.5 * E.elfving_expected(16, 0.0, 1.0))


def test_cutoff_from_expected_against_brute_force():
    rng = np.random.default_rng(1)
    cases = [np.array([1.0, 2.0, 3.0]), np.array([-1.0, 0.0, 0.5]), np.array([-2.0, -1.0]), np.array([0.3])]
    cases += [np.sort(rng.normal(0.4, 0.5, size=n)) for n in (2, 5, 17, 64) for _ in range(10)]
    for e in cases:
        ok = [c for c in range(1, len(e) + 1) if e[c - 1] > 0]
        if not ok:
            assert E.cutoff_from_expected(e) == len(e)
            continue
        top = max(c / e[c - 1] for c in ok)
        assert E.cutoff_from_expected(e) == max(c for c in ok if c / e[c - 1] == top)


def test_order_baseline_uses_the_running_moments_of_what_was_seen_before():
    trace = inputs.make_trace(24, 12, seed=3, sigma=0.3, groups=4, stay=0.8, slowdown=2.0)
    cs = E.order_cutoffs(trace)
    assert cs[0] == 24                                          # nothing observed yet: wait for all
    for t in (1, 2, 7, 11):
        seen = np.concatenate([trace[s].astype(np.float64) for s in range(t)])
        e = E.elfving_expected(24, float(np.mean(seen)), float(np.std(seen)))
        assert cs[t] == E.cutoff_from_expected(e)
    # the rule is blind to who is slow: permuting workers within steps changes nothing
    rng = np.random.default_rng(0)
    shuffled = np.stack([rng.permutation(row) for row in trace])
    assert np.array_equal(E.order_cutoffs(shuffled), cs)
    # no spread at all: every expected order statistic equals the mean, so c = N
    assert np.all(E.order_cutoffs(np.full((5, 9), 0.7)) == 9)
    # iid normal-looking data with a wide spread: the expected maximum is far out, so some workers are dropped
    wide = np.abs(np.random.default_rng(5).normal(1.0, 0.4, size=(6, 158))) + 0.05
    assert np.all(E.order_cutoffs(wide)[1:] < 158)


def test_best_static_cutoff_brute_force():
    trace = inputs.make_trace(16, 30, seed=9, sigma=0.3, straggler_p=0.1, straggler_scale=2.0)
    ordered = np.sort(trace.astype(np.float64), axis=1)
    totals = [sum(c / ordered[t][c - 1] for t in range(30)) for c in range(1, 17)]
    want = max(c for c in range(1, 17) if totals[c - 1] == max(totals))
    assert E.best_static_cutoff(trace) == want
    r = E.evaluate(trace, {"static": want, "hind": [E.hindsight_best(row)[0] for row in trace]})
    assert np.allclose(r["hind"], r["best"])
    assert np.all(r["static"] <= r["best"] + 1e-15) and np.all(r["all"] <= r["best"] + 1e-15)
    assert math.isclose(r["static"].sum(), max(totals))
