"""Pins for the oracle's ELBO, its gradient and the optimiser (Section 3.1.3, Section 4.1).

The expected values come from outside the functions under test: central finite differences, the log marginal
likelihood of a linear-Gaussian model computed from its textbook formula, the closed-form Gaussian KL divergence,
and an Adam run worked by hand.
"""
import math

import numpy as np

from oracle import cutoff_oracle as O
from oracle import elbo as L
from paper_1803_04209_b200 import inputs


def _model(N=5, D=3, H=4, seed=3, std=0.5):
    w = inputs.make_weights(N, D, H, seed=seed, std=std, offsets=False)
    rng = np.random.default_rng(seed)
    for k in ("a0", "b0", "z0"):
        w[k] = (rng.standard_normal(w[k].shape) * 0.3).astype(np.float32)
    return {k: v.astype(np.float64) for k, v in w.items()}


def test_gradient_of_every_tensor_against_central_differences():
    N, D, H, W, B = 5, 3, 4, 3, 2
    w = _model(N, D, H)
    rng = np.random.default_rng(0)
    x = rng.uniform(0.2, 1.0, size=(B, W, N))
    eps = rng.standard_normal((B, W, D))
    elbo, g = L.elbo_and_grad(w, x, eps)
    assert elbo.shape == (B,) and set(g) == set(L.PARAMS)
    worst = 0.0
    for name in L.PARAMS:
        flat = w[name].reshape(-1)
        picks = rng.choice(flat.size, size=min(flat.size, 6), replace=False)
        for i in picks:
            keep = flat[i]
            step = 1e-6
            flat[i] = keep + step
            up = L.elbo_and_grad(w, x, eps, want_grad=False)[0].sum()
            flat[i] = keep - step
            down = L.elbo_and_grad(w, x, eps, want_grad=False)[0].sum()
            flat[i] = keep
            fd = (up - down) / (2 * step)
            got = g[name].reshape(-1)[i]
            worst = max(worst, abs(fd - got) / max(1.0, abs(fd)))
    assert worst < 2e-6, worst


def test_elbo_equals_the_log_evidence_when_the_guide_is_the_exact_posterior():
    # one step, one latent, one worker, everything linear-Gaussian:
    #   z ~ N(m0, s0^2),  x | z ~ N(a z + c, r^2)   =>   x ~ N(a m0 + c, a^2 s0^2 + r^2),
    #   z | x ~ N(m0 + k (x - a m0 - c), s0^2 (1 - k a)),  k = a s0^2 / (a^2 s0^2 + r^2).
    # With q set to that posterior the one-sample ELBO is the log evidence for EVERY eps.
    m0, s0, a, c, r, x = 0.3, 0.8, 1.7, -0.2, 0.5, 1.1
    var_x = a * a * s0 * s0 + r * r
    k = a * s0 * s0 / var_x
    post_m, post_s = m0 + k * (x - a * m0 - c), math.sqrt(s0 * s0 * (1 - k * a))
    log_evidence = -0.5 * (math.log(2 * math.pi) + math.log(var_x) + (x - a * m0 - c) ** 2 / var_x)
    big = 50.0                                         # keeps the single ReLU of each MLP in its linear part
    w = {k_: np.zeros(s_) for k_, s_ in inputs.tensor_shapes(1, 1, 1).items()}
    w["bmu"][:] = post_m
    w["bsig"][:] = math.log(math.expm1(post_s))        # softplus^-1
    w["b1"][:] = big; w["W2"][:] = 0.0; w["b2"][:] = [m0, 2 * math.log(s0)]
    w["W3"][:] = 1.0; w["b3"][:] = big; w["W4"][0, 0] = a; w["b4"][:] = [c - a * big, 2 * math.log(r)]
    for e in (-2.0, -0.3, 0.0, 0.9, 2.5):
        elbo, _ = L.elbo_and_grad(w, np.array([[[x]]]), np.array([[[e]]]), want_grad=False)
        assert abs(elbo[0] - log_evidence) < 1e-10
    # a wrong guide gives, on average, the evidence minus KL(q || posterior)
    w["bmu"][:] = post_m + 0.4
    w["bsig"][:] = math.log(math.expm1(0.7 * post_s))
    eps = O.normals(11, 0, 0, np.arange(1 << 16), 1)
    vals, _ = L.elbo_and_grad(w, np.full((eps.shape[0], 1, 1), x), eps[:, None, :], want_grad=False)
    kl = L.gaussian_kl([post_m + 0.4], [0.7 * post_s], [post_m], [post_s])
    assert abs(vals.mean() - (log_evidence - kl)) < 5 * vals.std() / math.sqrt(vals.size)
    assert kl > 0.05


def test_gaussian_kl_closed_form_cases():
    assert L.gaussian_kl([0.3, -1.0], [0.5, 2.0], [0.3, -1.0], [0.5, 2.0]) == 0.0
    assert math.isclose(L.gaussian_kl([1.0], [1.0], [0.0], [1.0]), 0.5)                 # shifted unit Gaussians
    assert math.isclose(L.gaussian_kl([0.0], [2.0], [0.0], [1.0]), 1.5 - math.log(2.0))
    # against the defining integral, numerically
    mq, sq, mp, sp = 0.2, 0.6, -0.1, 0.9
    z = np.linspace(-8, 8, 400001)
    q = np.exp(-0.5 * ((z - mq) / sq) ** 2) / (sq * math.sqrt(2 * math.pi))
    logq = -0.5 * ((z - mq) / sq) ** 2 - math.log(sq * math.sqrt(2 * math.pi))
    logp = -0.5 * ((z - mp) / sp) ** 2 - math.log(sp * math.sqrt(2 * math.pi))
    assert abs(np.trapezoid(q * (logq - logp), z) - L.gaussian_kl([mq], [sq], [mp], [sp])) < 1e-8


def test_the_elbo_uses_the_same_networks_as_the_decision_path():
    # the sampled path z_0 .. z_{W-1} inside the ELBO is the guide chain the decision draws from
    N, D, H, W, B = 4, 3, 5, 3, 6
    w = _model(N, D, H, seed=5)
    rng = np.random.default_rng(1)
    x = rng.uniform(0.2, 1.0, size=(1, W, N))
    eps = rng.standard_normal((B, W, D))
    a, b = O.encoder(x[0], w)
    z_T = O.guide_chain(a, b, w, eps)
    # raise the emission's weight on z_T only: d ELBO / d (last-step x mean bias) = sum_b (x - m_x) / var, which needs z_T
    elbo, g = L.elbo_and_grad(w, np.repeat(x, B, axis=0), eps)
    v = np.maximum(z_T @ w["W3"].T + w["b3"], 0.0)
    head = v @ w["W4"].T + w["b4"]
    m_x, lv_x = head[:, :N], head[:, N:]
    last = ((x[0, W - 1] - m_x) * np.exp(-lv_x)).sum(axis=0)
    # remove the earlier steps' share by differencing against a window whose last observation moved
    x2 = x.copy(); x2[0, W - 1] += 0.25
    _, g2 = L.elbo_and_grad(w, np.repeat(x2, B, axis=0), eps)
    a2, b2 = O.encoder(x2[0], w)
    z_T2 = O.guide_chain(a2, b2, w, eps)
    v2 = np.maximum(z_T2 @ w["W3"].T + w["b3"], 0.0)
    head2 = v2 @ w["W4"].T + w["b4"]
    last2 = ((x2[0, W - 1] - head2[:, :N]) * np.exp(-head2[:, N:])).sum(axis=0)
    # d/d b4[mean] sums the same expression over all steps; the steps before the last see the change of x_T only
    # through the backward RNN, so compare totals built from the oracle's own decision-path functions step by step
    def total_mean_bias_grad(xw):
        aa, bb = O.encoder(xw[0], w)
        out = np.zeros(N)
        for t in range(W):
            z_t = O.guide_chain(aa[: t + 1], bb[: t + 1], w, eps[:, : t + 1])
            vv = np.maximum(z_t @ w["W3"].T + w["b3"], 0.0)
            hh = vv @ w["W4"].T + w["b4"]
            out += ((xw[0, t] - hh[:, :N]) * np.exp(-hh[:, N:])).sum(axis=0)
        return out
    assert np.allclose(g["b4"][:N], total_mean_bias_grad(x), rtol=1e-10, atol=1e-12)
    assert np.allclose(g2["b4"][:N], total_mean_bias_grad(x2), rtol=1e-10, atol=1e-12)
    assert not np.allclose(last, last2)


def test_adam_two_steps_by_hand():
    # one scalar, gradients 0.5 then -1.0, lr 0.1, beta1 0.9, beta2 0.999, eps 1e-8
    p = {"w": np.array([1.0])}
    opt = L.Adam(lr=0.1)
    opt.step(p, {"w": np.array([0.5])})
    # m = 0.05, v = 0.00025; m_hat = 0.5, v_hat = 0.25 -> step = 0.1 * 0.5 / (0.5 + 1e-8)
    w1 = 1.0 - 0.1 * 0.5 / (0.5 + 1e-8)
    assert math.isclose(p["w"][0], w1, rel_tol=1e-14)
    opt.step(p, {"w": np.array([-1.0])})
    m = 0.9 * 0.05 + 0.1 * -1.0                      # -0.055
    v = 0.999 * 0.00025 + 0.001 * 1.0                # 0.00124975
    m_hat, v_hat = m / (1 - 0.9 ** 2), v / (1 - 0.999 ** 2)
    w2 = w1 - 0.1 * m_hat / (math.sqrt(v_hat) + 1e-8)
    assert math.isclose(p["w"][0], w2, rel_tol=1e-14)
    assert w2 > w1                                    # the second gradient pushed the other way and won


def test_clipping_scales_by_the_global_norm():
    g = {"a": np.array([3.0, 0.0]), "b": np.array([[0.0, 4.0]])}
    out, norm = L.clip_by_global_norm(g, 10.0)
    assert norm == 5.0 and out is g
    out, norm = L.clip_by_global_norm(g, 1.0)
    assert norm == 5.0
    assert np.allclose(out["a"], [0.6, 0.0]) and np.allclose(out["b"], [[0.0, 0.8]])


def test_fitting_raises_the_elbo_and_learns_the_level_of_the_data():
    # a small cluster with two groups, one persistently slow: after a few hundred steps the emission mean must
    # sit on the data (normalised run-times average 0.5) and the ELBO must have risen by a wide margin
    N, D, H, lag = 12, 4, 16, 1
    trace = inputs.make_trace(N, 160, seed=4, sigma=0.15, groups=2, stay=0.97, slowdown=2.0)
    w0 = inputs.make_weights(N, D, H, seed=1, offsets=False)
    scale = 2.0 * float(trace[: lag + 1].astype(np.float64).mean())
    data = L.windows_of(trace.astype(np.float64) / scale, lag + 1)
    eps = np.random.default_rng(0).standard_normal((data.shape[0], lag + 1, D))
    before = L.elbo_and_grad(w0, data, eps, want_grad=False)[0].mean()
    fitted, hist = L.fit(w0, trace, lag, steps=400, batch=32, lr=5e-3, seed=2, log_every=100)
    after = L.elbo_and_grad(fitted, data, eps, want_grad=False)[0].mean()
    assert after > before + 10.0 * N * (lag + 1) * 0.05
    assert hist[-1][1] > hist[0][1]
    # predictive mean of the fitted model against the data's level
    orc = O.CutoffOracle(fitted, lag, 512, seed=3)
    for row in trace[:40]:
        orc.push(row)
    draws = orc.samples(np.arange(512)) * orc.scale()
    assert abs(draws.mean() / trace[40:60].mean() - 1.0) < 0.25
