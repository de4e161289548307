"""Pins for the CPU oracle: what the paper and the mathematics fix, not the oracle itself.

Every test here runs on the CPU.  A plausible mistake in the oracle -- a
dropped term, a wrong sign or index, a transposed operand, a wrong noise
stream -- should fail at least one of them.
"""
import math
import os

import numpy as np
import pytest
from scipy import stats

from oracle import cutoff_oracle as O
from oracle import iid_normal as A
from paper_1803_04209_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------
# Philox4x32-10
# ----------------------------------------------------------------------------
def _kat_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append([int(tok, 16) for tok in line.split()])
    return rows


def test_philox_known_answer_vectors():
    rows = _kat_rows()
    assert len(rows) == 3
    for row in rows:
        out = O.philox4x32_10(*row[:6])
        assert [int(v) for v in out] == row[6:]


def _philox_bigint(ctr, key):
    """Second implementation from the published definition, on Python integers."""
    c = list(ctr)
    k = list(key)
    for r in range(10):
        prod_a = 0xD2511F53 * c[0]
        prod_b = 0xCD9E8D57 * c[2]
        c = [((prod_b >> 32) ^ c[1] ^ k[0]) & 0xFFFFFFFF, prod_b & 0xFFFFFFFF,
             ((prod_a >> 32) ^ c[3] ^ k[1]) & 0xFFFFFFFF, prod_a & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) % 2 ** 32, (k[1] + 0xBB67AE85) % 2 ** 32]
    return c


def _philox_inverse(out, key):
    """Run the ten rounds backwards: multiplication by an odd constant is invertible mod 2^32."""
    inv_a = pow(0xD2511F53, -1, 2 ** 32)
    inv_b = pow(0xCD9E8D57, -1, 2 ** 32)
    keys = [((key[0] + r * 0x9E3779B9) % 2 ** 32, (key[1] + r * 0xBB67AE85) % 2 ** 32) for r in range(10)]
    c = list(out)
    for r in range(9, -1, -1):
        c2 = (c[1] * inv_b) % 2 ** 32          # lo(M1*c2) -> c2
        c0 = (c[3] * inv_a) % 2 ** 32          # lo(M0*c0) -> c0
        c1 = c[0] ^ ((0xCD9E8D57 * c2) >> 32) ^ keys[r][0]
        c3 = c[2] ^ ((0xD2511F53 * c0) >> 32) ^ keys[r][1]
        c = [c0, c1, c2, c3]
    return c


def test_philox_against_bigint_and_inverse():
    rng = np.random.default_rng(11)
    words = rng.integers(0, 2 ** 32, size=(20000, 6), dtype=np.uint64)
    out = np.stack(O.philox4x32_10(*[words[:, i] for i in range(6)]), axis=1)
    for i in range(0, 20000, 7):
        ctr = [int(v) for v in words[i, :4]]
        key = [int(v) for v in words[i, 4:]]
        assert [int(v) for v in out[i]] == _philox_bigint(ctr, key)
        assert _philox_inverse([int(v) for v in out[i]], key) == ctr


def test_philox_is_a_bijection_on_a_slice():
    # distinct counters under one key give distinct outputs
    q = np.arange(1 << 16, dtype=np.uint64)
    out = np.stack(O.philox4x32_10(q, 5, 6, 7, 8, 9), axis=1)
    assert len({tuple(r) for r in out.tolist()}) == 1 << 16


# ----------------------------------------------------------------------------
# Box-Muller and the stream layout
# ----------------------------------------------------------------------------
def test_box_muller_moments_and_ks():
    eps = O.normals(seed=2024, step=3, stream=O.STREAM_EMISSION, k=np.arange(4096), n_elems=1024).ravel()
    n = eps.size                                         # 4.2e6 draws
    assert abs(eps.mean()) < 5.0 / math.sqrt(n)
    assert abs(eps.var() - 1.0) < 5.0 * math.sqrt(2.0 / n)
    assert abs(stats.skew(eps)) < 5.0 * math.sqrt(6.0 / n)
    assert abs(stats.kurtosis(eps)) < 5.0 * math.sqrt(24.0 / n)
    assert stats.kstest(eps[:: 4], "norm").pvalue > 1e-3
    assert np.abs(eps).max() <= math.sqrt(2.0 * 24.0 * math.log(2.0)) + 1e-12   # u1 >= 2^-24


def test_box_muller_uses_the_documented_bits():
    # radius^2 = -2 ln u1 with u1 from word 0 (resp. 2); the angle comes from word 1 (resp. 3)
    r = O.philox4x32_10(3, 17, 5, 9, 123, 456)
    eps = O.normals(seed=123 | (456 << 32), step=9, stream=5, k=[17], n_elems=16)[0]
    for pair, (wa, wb) in enumerate(((0, 1), (2, 3))):
        u1 = ((int(r[wa]) >> 8) + 1) / 2 ** 24
        u2 = (int(r[wb]) >> 8) / 2 ** 24
        e_cos, e_sin = eps[12 + 2 * pair], eps[13 + 2 * pair]      # counter word 0 = 3 -> elements 12..15
        assert math.isclose(e_cos ** 2 + e_sin ** 2, -2.0 * math.log(u1), rel_tol=1e-12)
        assert math.isclose(math.atan2(e_sin, e_cos) % (2 * math.pi), 2 * math.pi * u2, rel_tol=1e-9, abs_tol=1e-12)


def test_streams_steps_samples_are_independent_draws():
    base = O.normals(1, 0, 0, np.arange(64), 8)
    for other in (O.normals(2, 0, 0, np.arange(64), 8), O.normals(1, 1, 0, np.arange(64), 8),
                  O.normals(1, 0, 1, np.arange(64), 8), O.normals(1, 0, 0, np.arange(64, 128), 8)):
        assert not np.any(base == other)
        assert abs(np.corrcoef(base.ravel(), other.ravel())[0, 1]) < 0.2
    # a sample's draws do not depend on which other samples are asked for
    assert np.array_equal(O.normals(1, 0, 0, [40], 8)[0], base[40])
    # element count only truncates
    assert np.array_equal(O.normals(1, 0, 0, np.arange(64), 6), base[:, :6])


# ----------------------------------------------------------------------------
# The analytic iid-normal model (Section 3.1.1) and the paper's worked example
# ----------------------------------------------------------------------------
def test_order_statistic_integral_textbook_values():
    # n = 2: E[max] = 1/sqrt(pi); n = 3: E[max] = 3/(2 sqrt(pi)), E[median] = 0 (David & Nagaraja)
    assert math.isclose(A.expected_order_statistic(2, 2), 1.0 / math.sqrt(math.pi), rel_tol=1e-9)
    assert math.isclose(A.expected_order_statistic(2, 1), -1.0 / math.sqrt(math.pi), rel_tol=1e-9)
    assert math.isclose(A.expected_order_statistic(3, 3), 1.5 / math.sqrt(math.pi), rel_tol=1e-9)
    assert abs(A.expected_order_statistic(3, 2)) < 1e-10
    # the expectations of all order statistics sum to n * mu
    total = sum(A.expected_order_statistic(16, j, 1.5, 0.3) for j in range(1, 17))
    assert math.isclose(total, 16 * 1.5, rel_tol=1e-9)
    # symmetry about the mean, and monotone in j (Section 3.1.1)
    e = [A.expected_order_statistic(16, j) for j in range(1, 17)]
    assert all(math.isclose(e[j], -e[15 - j], abs_tol=1e-9) for j in range(16))
    assert all(e[j] < e[j + 1] for j in range(15))


def _paper_example():
    vals = {}
    for line in open(os.path.join(GOLDEN, "paper_worked_example.txt")):
        if line.strip() and not line.startswith("#"):
            key, v = line.split()
            vals[key] = float(v)
    return vals


def test_paper_worked_example_elfving_and_idle_time():
    ex = _paper_example()
    n = int(ex["n_workers"])
    approx = A.elfving(n, n, ex["mean_sec"], ex["std_sec"])
    exact = A.expected_order_statistic(n, n, ex["mean_sec"], ex["std_sec"])
    assert abs(approx - ex["expected_max_sec"]) < 2e-3
    assert abs(exact - ex["expected_max_sec"]) < 2e-3
    # Eq. (3): mean idle time; exactly E[max] - mu, approximated in the paper by the middle order statistic
    idle = A.mean_idle_time(n, ex["mean_sec"], ex["std_sec"])
    assert abs(idle - ex["mean_idle_sec"]) < 2e-3
    assert abs(idle - (exact - A.expected_order_statistic(n, n // 2, ex["mean_sec"], ex["std_sec"]))) < 5e-3


def test_elfving_close_to_integral():
    for n, j in ((16, 1), (16, 9), (158, 158), (158, 40)):
        assert abs(A.elfving(n, j) - A.expected_order_statistic(n, j)) < 2e-2   # an approximation


# ----------------------------------------------------------------------------
# Sort / mean / throughput / argmax tail against the analytic model
# ----------------------------------------------------------------------------
def _constant_emission_weights(N, D=2, H=4, mu=0.0, sigma=1.0):
    w = inputs.make_weights(N, D, H, seed=5, offsets=False)
    w["W4"][:] = 0.0
    w["b4"][:N] = mu
    w["b4"][N:] = 2.0 * math.log(sigma)
    return w


def _predictive_samples(w, S, window=2, seed=99, step=0):
    N = w["b4"].shape[0] // 2
    xhat = np.full((window, N), 0.5)
    return O.sample_runtimes(w, xhat, seed, step, np.arange(S))


def test_monte_carlo_order_statistics_match_integral_n2():
    mu, sigma, S = 1.25, 0.5, 1 << 19
    x = _predictive_samples(_constant_emission_weights(2, mu=mu, sigma=sigma), S)
    e = O.expected_order_statistics(x)
    tol = 4.5 * sigma / math.sqrt(S)
    assert abs(e[1] - (mu + sigma / math.sqrt(math.pi))) < tol
    assert abs(e[0] - (mu - sigma / math.sqrt(math.pi))) < tol


def test_monte_carlo_order_statistics_match_integral_n16():
    mu, sigma, S = 0.5, 0.1, 1 << 17
    x = _predictive_samples(_constant_emission_weights(16, mu=mu, sigma=sigma), S)
    e = O.expected_order_statistics(x)
    for j in range(1, 17):
        assert abs(e[j - 1] - A.expected_order_statistic(16, j, mu, sigma)) < 4.5 * sigma / math.sqrt(S)


def test_monte_carlo_max_of_158_matches_paper_example():
    ex = _paper_example()
    n, S = int(ex["n_workers"]), 1 << 15
    x = _predictive_samples(_constant_emission_weights(n, mu=ex["mean_sec"], sigma=ex["std_sec"]), S)
    e = O.expected_order_statistics(x)
    assert abs(e[-1] - ex["expected_max_sec"]) < 2e-3 + 4.5 * ex["std_sec"] * 0.45 / math.sqrt(S)
    assert abs(e[-1] - A.expected_order_statistic(n, n, ex["mean_sec"], ex["std_sec"])) < 4.5 * 0.2 / math.sqrt(S)


def test_invariants_of_expected_order_statistics():
    wl = inputs.WORKLOADS["n128"]
    w = inputs.workload_weights(wl)
    x = _predictive_samples(w, 4096, window=wl.window)
    e = O.expected_order_statistics(x)
    assert np.all(np.diff(e) >= 0)                                   # Section 3.1.1 monotonicity
    assert math.isclose(e.sum(), x.sum(axis=1).mean(), rel_tol=1e-12)  # sorting permutes each row
    assert x.min() <= e[0] and e[-1] <= x.max()
    # each row is a permutation: brute-force the sort on a few rows
    for row in x[:5]:
        assert sorted(row.tolist()) == np.sort(row, kind="stable").tolist()


def test_equal_deterministic_times_give_full_cutoff():
    # all workers take exactly the same time -> Omega(c) = c / t grows with c -> wait for all N
    w = _constant_emission_weights(12, mu=0.75, sigma=1e-30)
    x = _predictive_samples(w, 64)
    assert np.all(x == 0.75)
    omega = O.throughput(O.expected_order_statistics(x))
    assert O.argmax_cutoff(omega) == (12, False)


def _brute_force_cutoff(e):
    best, arg = None, None
    for c in range(1, len(e) + 1):
        if e[c - 1] > 0:
            val = c / e[c - 1]
            if best is None or val >= best:
                best, arg = val, c
    return (len(e), True) if arg is None else (arg, False)


def test_throughput_and_argmax_brute_force():
    rng = np.random.default_rng(3)
    cases = [
        np.array([1.0, 2.0, 3.0, 4.0]),            # Omega constant -> tie -> largest c
        np.array([1.0, 1.1, 1.2, 10.0]),           # drop the straggler
        np.array([-1.0, -0.5, 0.0, 0.0]),          # nothing admissible
        np.array([-1.0, 0.5, 0.6, 0.7]),           # non-positive entry excluded
        np.array([0.5]),
        np.array([2.0, 2.0, 2.0]),
    ]
    cases += [np.sort(rng.normal(0.5, 0.4, size=n)) for n in (2, 3, 7, 16, 33) for _ in range(20)]
    for e in cases:
        omega = O.throughput(e)
        for c in range(1, len(e) + 1):
            if e[c - 1] > 0:
                assert omega[c - 1] == c / e[c - 1]
            else:
                assert omega[c - 1] == -np.inf
        assert O.argmax_cutoff(omega) == _brute_force_cutoff(e)
    assert O.argmax_cutoff(O.throughput(cases[0])) == (4, False)
    assert O.argmax_cutoff(O.throughput(cases[1])) == (3, False)
    assert O.argmax_cutoff(O.throughput(cases[2])) == (4, True)


# ----------------------------------------------------------------------------
# Networks: special cases with closed forms
# ----------------------------------------------------------------------------
def test_encoder_reduces_to_geometric_sums_and_respects_direction():
    N, H, W = 6, 4, 5
    rng = np.random.default_rng(8)
    xhat = rng.uniform(0.2, 1.0, size=(W, N))
    w = inputs.make_weights(N, 3, H, seed=1, offsets=False)
    for name in ("Wxf", "Wxb", "Whf", "Whb", "bf", "bb"):
        w[name][:] = 0.0
    w["Wxf"][np.arange(H), np.arange(H)] = 1.0        # forward reads workers 0..3
    w["Wxb"][np.arange(H), np.arange(H) + 2] = 1.0    # backward reads workers 2..5
    w["Whf"][np.arange(H), np.arange(H)] = 0.5
    w["Whb"][np.arange(H), np.arange(H)] = 0.25
    w["a0"][:] = 0.8
    w["b0"][:] = 0.4
    a, b = O.encoder(xhat, w)
    for t in range(W):
        want_a = 0.8 * 0.5 ** (t + 1) + sum(0.5 ** (t - s) * xhat[s, :H] for s in range(t + 1))
        want_b = 0.4 * 0.25 ** (W - t) + sum(0.25 ** (s - t) * xhat[s, 2:2 + H] for s in range(t, W))
        assert np.allclose(a[t], want_a, rtol=1e-12)
        assert np.allclose(b[t], want_b, rtol=1e-12)
    # ReLU: a negative drive is clipped to zero
    w["bf"][:] = -100.0
    a, _ = O.encoder(xhat, w)
    assert np.all(a == 0.0)


def test_encoder_general_matrices_one_step():
    # one window position, zero initial state: a = relu(Wxf x + bf) is a plain matrix-vector product
    N, H = 5, 3
    w = inputs.make_weights(N, 2, H, seed=2, offsets=False)
    x = np.array([[0.3, 0.1, 0.9, 0.5, 0.7]])
    a, b = O.encoder(x, w)
    for i in range(H):
        drive_a = sum(float(w["Wxf"][i, j]) * x[0, j] for j in range(N)) + float(w["bf"][i])
        drive_b = sum(float(w["Wxb"][i, j]) * x[0, j] for j in range(N)) + float(w["bb"][i])
        assert math.isclose(a[0, i], max(drive_a, 0.0), rel_tol=1e-12, abs_tol=1e-15)
        assert math.isclose(b[0, i], max(drive_b, 0.0), rel_tol=1e-12, abs_tol=1e-15)


def test_guide_chain_zero_weights_gives_fixed_gaussian():
    D, H, W, S = 3, 4, 3, 1 << 16
    w = inputs.make_weights(5, D, H, seed=3, offsets=False)
    w["Wz"][:] = 0.0
    w["Wmu"][:] = 0.0
    a = np.zeros((W, H))
    eps = np.stack([O.normals(7, 0, t, np.arange(S), D) for t in range(W)], axis=1)
    z = O.guide_chain(a, a, w, eps)
    mu = w["bmu"].astype(np.float64)
    sd = np.log1p(np.exp(w["Wsig"].astype(np.float64) @ mu + w["bsig"]))
    assert np.all(np.abs(z.mean(axis=0) - mu) < 4.5 * sd / math.sqrt(S))
    assert np.all(np.abs(z.std(axis=0) / sd - 1.0) < 4.5 / math.sqrt(2 * S))
    # the draw of the LAST window step is the one that survives
    assert np.allclose(z, mu + sd * eps[:, W - 1, :], rtol=1e-12)


def test_guide_chain_noise_free_scalar_recursion():
    # D = H = 1, sigma -> 0: z_t = wmu * (tanh(wz z_{t-1} + bz) + a_t + b_t) / 3 + bmu
    w = inputs.make_weights(1, 1, 1, seed=4, offsets=False)
    w["Wz"][:] = 0.7; w["bz"][:] = -0.2; w["Wmu"][:] = 1.3; w["bmu"][:] = 0.1
    w["Wsig"][:] = 0.0; w["bsig"][:] = -800.0; w["z0"][:] = 0.4
    a = np.array([[0.5], [0.25], [2.0]])
    b = np.array([[1.0], [0.75], [0.125]])
    z = O.guide_chain(a, b, w, np.ones((2, 3, 1)))
    wz, bz, wmu, bmu = (float(w[k].ravel()[0]) for k in ("Wz", "bz", "Wmu", "bmu"))
    want = 0.4
    for t in range(3):
        want = wmu * (math.tanh(wz * want + bz) + a[t, 0] + b[t, 0]) / 3.0 + bmu
    assert np.allclose(z, want, rtol=1e-13)


def test_encoder_against_scalar_loops_dense_nonsymmetric_recurrence():
    # h_left(t) = relu(Wxf x_t + Whf h_left(t-1) + bf) from a0, h_right(t) likewise backwards from b0
    # (Section 3.1.3, guide): written out element by element, with dense non-symmetric recurrent matrices,
    # non-zero initial states and several window positions, so that a transposed Whf / Whb, a swapped
    # direction or a dropped initial state shows.
    N, H, W = 5, 4, 4
    rng = np.random.default_rng(21)
    w = inputs.make_weights(N, 3, H, seed=12, std=0.6, offsets=False)
    w["a0"] = rng.uniform(0.2, 1.0, size=H).astype(np.float32)
    w["b0"] = rng.uniform(0.2, 1.0, size=H).astype(np.float32)
    assert not np.allclose(w["Whf"], w["Whf"].T) and not np.allclose(w["Whb"], w["Whb"].T)
    xhat = rng.uniform(0.1, 1.2, size=(W, N))
    a, b = O.encoder(xhat, w)
    f = {k: v.astype(np.float64) for k, v in w.items()}
    state = [float(v) for v in f["a0"]]
    active = 0
    for t in range(W):
        new = []
        for i in range(H):
            pre = f["bf"][i]
            for j in range(N):
                pre += f["Wxf"][i][j] * xhat[t][j]
            for j in range(H):
                pre += f["Whf"][i][j] * state[j]
            new.append(max(pre, 0.0))
        state = new
        active += sum(v > 0 for v in new)
        for i in range(H):
            assert abs(a[t][i] - state[i]) < 1e-12
    state = [float(v) for v in f["b0"]]
    for t in range(W - 1, -1, -1):
        new = []
        for i in range(H):
            pre = f["bb"][i]
            for j in range(N):
                pre += f["Wxb"][i][j] * xhat[t][j]
            for j in range(H):
                pre += f["Whb"][i][j] * state[j]
            new.append(max(pre, 0.0))
        state = new
        active += sum(v > 0 for v in new)
        for i in range(H):
            assert abs(b[t][i] - state[i]) < 1e-12
    assert active >= W * H // 2          # the case is not vacuous: most units carry state forward
    # the pin has teeth: the same loops against a transposed recurrence disagree
    wt = dict(w); wt["Whf"] = w["Whf"].T.copy()
    assert np.max(np.abs(O.encoder(xhat, wt)[0] - a)) > 1e-3


def test_guide_chain_against_scalar_loops_dense_weights_with_noise():
    # z_t = mu + sigma * eps,  h_out = (tanh(Wz z_{t-1} + bz) + h_left(t) + h_right(t)) / 3,
    # mu = Wmu h_out + bmu,  sigma = softplus(Wsig mu + bsig)   (Section 3.1.3, guide), element by element:
    # dense Wz feeding dense Wmu feeding dense Wsig over three steps, non-zero z0, noise on.
    D, H, W, S = 3, 5, 3, 4
    rng = np.random.default_rng(22)
    w = inputs.make_weights(4, D, H, seed=13, std=0.8, offsets=False)
    w["z0"] = rng.normal(size=D).astype(np.float32)
    a = np.abs(rng.normal(size=(W, H)))
    b = np.abs(rng.normal(size=(W, H)))
    eps = rng.standard_normal((S, W, D))
    got = O.guide_chain(a, b, w, eps)
    f = {k: v.astype(np.float64) for k, v in w.items()}
    for k in range(S):
        z = [float(v) for v in f["z0"]]
        for t in range(W):
            h_out = []
            for i in range(H):
                pre = f["bz"][i]
                for d in range(D):
                    pre += f["Wz"][i][d] * z[d]
                h_out.append((math.tanh(pre) + a[t][i] + b[t][i]) / 3.0)
            mu = []
            for d in range(D):
                acc = f["bmu"][d]
                for i in range(H):
                    acc += f["Wmu"][d][i] * h_out[i]
                mu.append(acc)
            z = []
            for d in range(D):
                pre = f["bsig"][d]
                for e in range(D):
                    pre += f["Wsig"][d][e] * mu[e]
                z.append(mu[d] + math.log1p(math.exp(pre)) * eps[k][t][d])
        for d in range(D):
            assert abs(got[k][d] - z[d]) < 1e-12
    # teeth: a transposed Wsig, or the window's encodings taken in reverse order, change the result
    wt = dict(w); wt["Wsig"] = w["Wsig"].T.copy()
    assert np.max(np.abs(O.guide_chain(a, b, wt, eps) - got)) > 1e-3
    assert np.max(np.abs(O.guide_chain(a[::-1], b[::-1], w, eps) - got)) > 1e-3


def test_guide_head_orientation():
    # Wz = 0: h_out is the same for every sample, so mu = Wmu h + bmu and sigma = softplus(Wsig mu + bsig)
    D, H, S = 3, 5, 1 << 15
    w = inputs.make_weights(4, D, H, seed=6, offsets=False)
    w["Wz"][:] = 0.0
    a = np.abs(np.random.default_rng(0).normal(size=(1, H)))
    b = np.abs(np.random.default_rng(1).normal(size=(1, H)))
    eps = O.normals(5, 0, 0, np.arange(S), D)[:, None, :]
    z = O.guide_chain(a, b, w, eps)
    h = (np.tanh(w["bz"].astype(np.float64)) + a[0] + b[0]) / 3.0
    mu = np.array([sum(float(w["Wmu"][d, i]) * h[i] for i in range(H)) + float(w["bmu"][d]) for d in range(D)])
    pre = np.array([sum(float(w["Wsig"][d, e]) * mu[e] for e in range(D)) + float(w["bsig"][d]) for d in range(D)])
    sd = np.log1p(np.exp(pre))
    assert np.all(np.abs(z.mean(axis=0) - mu) < 4.5 * sd / math.sqrt(S))
    assert np.all(np.abs(z.std(axis=0) / sd - 1.0) < 4.5 / math.sqrt(2 * S))


def test_linear_gaussian_special_case_of_transition_and_emission():
    # Large positive hidden biases keep every ReLU in its linear part and constant log-variance heads
    # make the model linear-Gaussian: x = A z_T + c + noise with a closed-form mean and covariance.
    N, D, H, S = 5, 3, 4, 1 << 17
    w = inputs.make_weights(N, D, H, seed=9, offsets=False)
    w["b1"][:] = 50.0
    w["b3"][:] = 50.0
    w["W2"][D:] = 0.0
    w["W4"][N:] = 0.0
    rng = np.random.default_rng(4)
    z_T = rng.normal(size=(1, D)).repeat(S, axis=0)
    f = {k: v.astype(np.float64) for k, v in w.items()}
    eps_t = O.normals(21, 2, O.STREAM_TRANSITION, np.arange(S), D)
    eps_e = O.normals(21, 2, O.STREAM_EMISSION, np.arange(S), N)
    z_next = O.transition(z_T, w, eps_t)
    x = O.emission(z_next, w, eps_e)
    A_t = f["W2"][:D] @ f["W1"]
    mean_z = A_t @ z_T[0] + f["W2"][:D] @ f["b1"] + f["b2"][:D]
    cov_z = np.diag(np.exp(f["b2"][D:]))
    A_e = f["W4"][:N] @ f["W3"]
    mean_x = A_e @ mean_z + f["W4"][:N] @ f["b3"] + f["b4"][:N]
    cov_x = A_e @ cov_z @ A_e.T + np.diag(np.exp(f["b4"][N:]))
    sd_x = np.sqrt(np.diag(cov_x))
    assert np.all(np.abs(z_next.mean(axis=0) - mean_z) < 4.5 * np.sqrt(np.diag(cov_z) / S))
    assert np.all(np.abs(x.mean(axis=0) - mean_x) < 4.5 * sd_x / math.sqrt(S))
    emp = np.cov(x, rowvar=False)
    assert np.all(np.abs(emp - cov_x) < 6.0 * np.outer(sd_x, sd_x) * math.sqrt(2.0 / S))
    # ReLU does clip: with large negative hidden bias the heads reduce to their biases
    w["b3"][:] = -50.0
    x0 = O.emission(z_next, w, np.zeros((S, N)))
    assert np.allclose(x0, f["b4"][:N], rtol=1e-12)


def test_log_variance_head_is_a_variance_not_a_deviation():
    w = _constant_emission_weights(4, mu=0.0, sigma=0.3)
    x = _predictive_samples(w, 1 << 16)
    assert np.all(np.abs(x.std(axis=0) / 0.3 - 1.0) < 4.5 / math.sqrt(2 * (1 << 16)))


# ----------------------------------------------------------------------------
# Observation handling and the whole decision
# ----------------------------------------------------------------------------
def test_normaliser_is_twice_the_mean_of_the_first_window():
    hist = np.arange(1, 25, dtype=np.float32).reshape(6, 4)
    assert O.normaliser(hist, 2) == 2.0 * np.mean(np.arange(1, 9))
    assert O.normaliser(hist, 6) == 2.0 * 12.5


def _driven_oracle(name, S, scale=1.0, steps=None, offsets=True):
    wl = inputs.WORKLOADS[name]
    w = inputs.workload_weights(wl, offsets=offsets)
    trace = inputs.workload_trace(wl, steps)
    orc = O.CutoffOracle(w, wl.lag, S, seed=77)
    for x in trace:
        orc.push(x * np.float32(scale))
    return orc


def test_warmup_waits_for_everyone():
    wl = inputs.WORKLOADS["tiny"]
    orc = O.CutoffOracle(inputs.workload_weights(wl), wl.lag, 64, seed=1)
    assert orc.predict()[:2] == (O.WARMUP, wl.N)
    orc.push(np.ones(wl.N, dtype=np.float32))
    assert orc.predict()[:2] == (O.WARMUP, wl.N)
    orc.push(np.ones(wl.N, dtype=np.float32))
    assert orc.predict()[0] == O.OK


def test_scale_invariance_of_the_decision():
    # times measured in other units (x4, exact in binary): same c, E scales linearly
    base = _driven_oracle("tiny", 512).predict()
    scaled = _driven_oracle("tiny", 512, scale=4.0).predict()
    assert base[1] == scaled[1]
    assert np.allclose(scaled[2], 4.0 * base[2], rtol=1e-12)
    assert np.allclose(scaled[3], base[3] / 4.0, rtol=1e-12)


def test_decision_matches_its_parts_and_steps_advance_the_noise():
    orc = _driven_oracle("n128", 256, steps=12)
    x = orc.samples(np.arange(256))
    code, c, e, omega = orc.predict()
    assert code == O.OK
    assert np.allclose(e, orc.scale() * np.sort(x, axis=1).mean(axis=0), rtol=1e-13)
    assert c == _brute_force_cutoff(e)[0]
    x_next = orc.samples(np.arange(256))          # same window, next decision: fresh noise
    assert not np.any(x_next == x)


def test_raw_weights_exercise_the_non_positive_rule():
    orc = _driven_oracle("n128", 256, steps=12, offsets=False)
    code, c, e, omega = orc.predict()
    assert e[0] <= 0 and omega[0] == -np.inf and e[c - 1] > 0


def test_window_uses_only_the_last_pushes_but_the_first_window_fixes_the_scale():
    wl = inputs.WORKLOADS["tiny"]
    trace = inputs.workload_trace(wl)
    orc = _driven_oracle("tiny", 64)
    assert np.allclose(orc.xhat(), trace[-wl.window:].astype(np.float64) / (2.0 * trace[: wl.window].mean(dtype=np.float64)))


def test_trace_generators_are_seeded_and_positive():
    for name, wl in inputs.WORKLOADS.items():
        t1 = inputs.workload_trace(wl, 30)
        t2 = inputs.workload_trace(wl, 30)
        assert t1.dtype == np.float32 and t1.shape == (30, wl.N)
        assert np.array_equal(t1, t2) and np.all(np.isfinite(t1)) and np.all(t1 > 0)
    w = inputs.workload_weights(inputs.WORKLOADS["n4096"])
    assert all(np.array_equal(v, inputs.round_to_bf16(v)) for v in w.values())


def test_noise_streams_feed_the_documented_stages():
    # Identity-like weights make x = b_mu + sigma_q * eps_q[last step] + 0.5 * eps_transition + 0.25 * eps_emission,
    # so each stage's noise stream (guide step t -> t, transition -> 0x100, emission -> 0x200) shows in the output.
    n, W, seed, step = 4, 3, 31337, 6
    w = inputs.make_weights(n, n, n, seed=12, offsets=False)
    eye = np.eye(n, dtype=np.float32)
    for name in ("Wz", "Wmu", "Wsig"):
        w[name][:] = 0.0
    w["W1"][:] = eye; w["b1"][:] = 50.0
    w["W2"][:n] = eye; w["W2"][n:] = 0.0; w["b2"][:n] = -50.0; w["b2"][n:] = 2.0 * math.log(0.5)
    w["W3"][:] = eye; w["b3"][:] = 50.0
    w["W4"][:n] = eye; w["W4"][n:] = 0.0; w["b4"][:n] = -50.0; w["b4"][n:] = 2.0 * math.log(0.25)
    k = np.arange(100, 164)
    x = O.sample_runtimes(w, np.full((W, n), 0.5), seed, step, k)
    sd_q = np.log1p(np.exp(w["bsig"].astype(np.float64)))
    want = (w["bmu"].astype(np.float64) + sd_q * O.normals(seed, step, W - 1, k, n)
            + math.exp(0.5 * float(w["b2"][n])) * O.normals(seed, step, O.STREAM_TRANSITION, k, n)
            + math.exp(0.5 * float(w["b4"][n])) * O.normals(seed, step, O.STREAM_EMISSION, k, n))
    assert O.STREAM_TRANSITION == 0x100 and O.STREAM_EMISSION == 0x200
    assert np.allclose(x, want, rtol=0, atol=1e-12)


# ----------------------------------------------------------------------------
# Censored run-times (Section 4.2)
# ----------------------------------------------------------------------------
def test_imputation_draws_from_the_left_truncated_predictive():
    # every worker's predictive distribution is N(1.0, 0.2^2); censoring at 1.1 s
    rng = np.random.default_rng(5)
    S, N = 4000, 600
    draws = rng.normal(1.0, 0.2, size=(S, N))
    observed = np.full(N, 0.9)
    observed[0] = 1.1                                  # the slowest worker that finished
    censored = np.zeros(N, dtype=bool)
    censored[100:] = True
    x, threshold = O.impute_censored(observed, censored, draws, seed=77, step=3)
    assert threshold == 1.1
    assert np.array_equal(x[:100], observed[:100])     # what was observed is kept
    assert np.all(x[100:] > threshold)
    a = (threshold - 1.0) / 0.2
    assert stats.kstest(x[100:], stats.truncnorm(a, np.inf, loc=1.0, scale=0.2).cdf).pvalue > 1e-3
    assert abs(x[100:].mean() - stats.truncnorm(a, np.inf, loc=1.0, scale=0.2).mean()) < 4.5 * 0.12 / math.sqrt(500)
    # each replacement is one of that worker's own predictive draws
    assert all(x[j] in draws[:, j] for j in range(100, 130))
    # same inputs, same result; another step number starts the scans elsewhere
    x2, _ = O.impute_censored(observed, censored, draws, seed=77, step=3)
    x3, _ = O.impute_censored(observed, censored, draws, seed=77, step=4)
    assert np.array_equal(x, x2) and not np.array_equal(x, x3)


def test_imputation_scan_order_and_fallback():
    draws = np.array([[1.0, 5.0], [3.0, 5.0], [2.0, 5.0], [4.0, 0.5]])      # 4 draws, 2 workers
    start = int(O.philox4x32_10(0, 0, O.STREAM_IMPUTE, 9, 21, 0)[0]) % 4
    x, thr = O.impute_censored([0.0, 1.5], [True, False], draws, seed=21, step=9)
    want = [v for v in np.roll(draws[:, 0], -start) if v > 1.5][0]          # first draw above 1.5 s from the start
    assert thr == 1.5 and x[0] == want and x[1] == 1.5
    # nothing above the threshold: the threshold itself
    x, thr = O.impute_censored([0.0, 9.0], [True, False], draws, seed=21, step=9)
    assert x[0] == 9.0
    # no censoring: untouched
    x, thr = O.impute_censored([0.7, 0.8], [False, False], draws, seed=21, step=9)
    assert thr is None and list(x) == [0.7, 0.8]


def test_oracle_push_with_censoring_uses_the_last_decision():
    orc = _driven_oracle("tiny", 256)
    code, c, e, omega = orc.predict()
    wl = inputs.WORKLOADS["tiny"]
    observed = inputs.workload_trace(wl, 21)[20]
    order = np.argsort(observed)
    censored = np.zeros(wl.N, dtype=bool)
    censored[order[c:]] = True                         # the workers beyond the cutoff were killed
    if c == wl.N:
        censored[order[-2:]] = True
    orc.push(observed, censored)
    pushed = orc.history[-1]
    assert np.array_equal(pushed[~censored], observed[~censored])
    assert np.all(pushed[censored] >= observed[~censored].max())
    assert orc.predict()[0] == O.OK


def test_order_statistic_spread_matches_closed_forms():
    # two iid N(mu, sigma^2) times: Var(max) = Var(min) = sigma^2 (1 - 1/pi); one time: sigma itself
    mu, sigma, S = 0.8, 0.25, 1 << 18
    x = _predictive_samples(_constant_emission_weights(2, mu=mu, sigma=sigma), S)
    sd = O.order_statistic_std(x)
    want = sigma * math.sqrt(1.0 - 1.0 / math.pi)
    assert np.all(np.abs(sd / want - 1.0) < 5.0 / math.sqrt(2 * S) * 1.5)
    x1 = _predictive_samples(_constant_emission_weights(1, mu=mu, sigma=sigma), S)
    assert abs(O.order_statistic_std(x1)[0] / sigma - 1.0) < 5.0 / math.sqrt(2 * S)
    # the spread is about the position's own mean: shifting all times changes nothing
    assert np.allclose(O.order_statistic_std(x + 3.0), sd, rtol=1e-9)
    orc = _driven_oracle("tiny", 256)
    orc.predict()
    assert np.allclose(orc.last_std_sec, np.sort(orc.last_draws_sec, axis=1).std(axis=0), rtol=1e-12)
