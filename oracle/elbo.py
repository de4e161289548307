"""Learning the model: the variational lower bound of Section 3.1.3, its gradient, and Adam with clipping.

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  Plain numpy in double precision, written for reading.

Section 3.1.3 ("Model Learning and Amortized Inference") fits the generative model p_theta and the guide
q_phi together by stochastic gradient ascent on

    ELBO = E_q [ log p_theta(x_{T-l:T}, z_{T-l:T}) - log q_phi(z_{T-l:T} | x_{T-l:T}) ],

with the factorisations printed there: p = prod_t p(z_t | z_{t-1}) p(x_t | z_t) (the hidden Markov model of
Section 3.1.2) and q = prod_t q(z_t | z_{t-1}, x_{T-l:T}) (the left-right guide).  Section 4.1 names the
optimiser: Adam with gradient clipping.

This module evaluates a one-sample, reparameterised estimate of the ELBO for a batch of windows -- z_t = mu_t +
sigma_t * eps_t with eps supplied by the caller -- for the "compact" networks (transition and emission are
one-hidden-layer ReLU MLPs with mean and log-variance heads), and its gradient with respect to every weight
tensor by reverse-mode differentiation written out layer by layer.  The latent before the window, z_{T-l-1},
is the learned vector z0; the RNNs start from the learned states a0, b0.

    log N(y; m, exp(lv))  = -1/2 [ log 2 pi + lv + (y - m)^2 exp(-lv) ]             (mean / log-variance heads)
    log q(z_t)            = sum_d -1/2 log 2 pi - log sigma_d - 1/2 eps_d^2         (z = mu + sigma eps)

Pins (tests/test_oracle_elbo.py): central finite differences of every tensor's gradient; a linear-Gaussian
model whose exact posterior the guide is set to, where the one-sample ELBO equals the log marginal likelihood for
every eps; the closed-form Gaussian KL divergence; a two-step Adam run worked by hand; the clipping rule.
"""
from __future__ import annotations

import math

import numpy as np

LOG_2PI = math.log(2.0 * math.pi)

# tensors that are learned (every tensor of the compact weight dictionary)
PARAMS = ("Wxf", "Whf", "bf", "a0", "Wxb", "Whb", "bb", "b0", "Wz", "bz", "Wmu", "bmu", "Wsig", "bsig", "z0",
          "W1", "b1", "W2", "b2", "W3", "b3", "W4", "b4")


def _softplus(v):
    return np.logaddexp(0.0, v)


def _sigmoid(v):
    return 0.5 * (1.0 + np.tanh(0.5 * v))


def elbo_and_grad(w: dict, xhat: np.ndarray, eps: np.ndarray, want_grad: bool = True):
    """One-sample ELBO of every window and (optionally) the gradient of their sum.

    w     weight dictionary (the compact variant's tensors), any float dtype; used in double
    xhat  [B, W, N] normalised run-times, oldest first
    eps   [B, W, D] standard-normal draws of the guide
    Returns (elbo [B], grads) with grads[name] = d sum_b elbo_b / d w[name] (None if want_grad is False).
    """
    p = {k: np.asarray(v, dtype=np.float64) for k, v in w.items()}
    x = np.asarray(xhat, dtype=np.float64)
    eps = np.asarray(eps, dtype=np.float64)
    B, W, N = x.shape
    D = p["z0"].shape[0]
    H = p["bf"].shape[0]

    # ---- forward: encoder RNNs over the window (h_left, h_right) -----------------------------------------
    a = np.zeros((W, B, H))
    b = np.zeros((W, B, H))
    state = np.broadcast_to(p["a0"], (B, H))
    for t in range(W):
        state = np.maximum(x[:, t] @ p["Wxf"].T + state @ p["Whf"].T + p["bf"], 0.0)
        a[t] = state
    state = np.broadcast_to(p["b0"], (B, H))
    for t in range(W - 1, -1, -1):
        state = np.maximum(x[:, t] @ p["Wxb"].T + state @ p["Whb"].T + p["bb"], 0.0)
        b[t] = state

    # ---- forward: guide chain, transition and emission densities along the sampled path ------------------
    z_prev = np.broadcast_to(p["z0"], (B, D))
    steps = []
    elbo = np.zeros(B)
    for t in range(W):
        comb = np.tanh(z_prev @ p["Wz"].T + p["bz"])
        h_out = (comb + a[t] + b[t]) / 3.0
        mu = h_out @ p["Wmu"].T + p["bmu"]
        pre_sig = mu @ p["Wsig"].T + p["bsig"]
        sigma = _softplus(pre_sig)
        z = mu + sigma * eps[:, t]
        log_q = np.sum(-0.5 * LOG_2PI - np.log(sigma) - 0.5 * eps[:, t] ** 2, axis=1)
        u = np.maximum(z_prev @ p["W1"].T + p["b1"], 0.0)
        head_z = u @ p["W2"].T + p["b2"]
        m_z, lv_z = head_z[:, :D], head_z[:, D:]
        log_pz = np.sum(-0.5 * (LOG_2PI + lv_z + (z - m_z) ** 2 * np.exp(-lv_z)), axis=1)
        v = np.maximum(z @ p["W3"].T + p["b3"], 0.0)
        head_x = v @ p["W4"].T + p["b4"]
        m_x, lv_x = head_x[:, :N], head_x[:, N:]
        log_px = np.sum(-0.5 * (LOG_2PI + lv_x + (x[:, t] - m_x) ** 2 * np.exp(-lv_x)), axis=1)
        elbo += log_px + log_pz - log_q
        steps.append(dict(z_prev=z_prev, comb=comb, h_out=h_out, mu=mu, pre_sig=pre_sig, sigma=sigma, z=z, u=u,
                          m_z=m_z, lv_z=lv_z, v=v, m_x=m_x, lv_x=lv_x))
        z_prev = z
    if not want_grad:
        return elbo, None

    # ---- backward ----------------------------------------------------------------------------------------
    g = {k: np.zeros_like(val) for k, val in p.items()}
    g_a = np.zeros((W, B, H))
    g_b = np.zeros((W, B, H))
    g_z_next = np.zeros((B, D))              # d ELBO / d z_t flowing back from step t+1
    for t in range(W - 1, -1, -1):
        s = steps[t]
        g_z = g_z_next.copy()
        # emission density log p(x_t | z_t)
        r = x[:, t] - s["m_x"]
        inv = np.exp(-s["lv_x"])
        d_head = np.concatenate([r * inv, -0.5 + 0.5 * r * r * inv], axis=1)
        g["W4"] += d_head.T @ s["v"]
        g["b4"] += d_head.sum(axis=0)
        d_pre = (d_head @ p["W4"]) * (s["v"] > 0.0)
        g["W3"] += d_pre.T @ s["z"]
        g["b3"] += d_pre.sum(axis=0)
        g_z += d_pre @ p["W3"]
        # transition density log p(z_t | z_{t-1})
        r = s["z"] - s["m_z"]
        inv = np.exp(-s["lv_z"])
        g_z += -r * inv
        d_head = np.concatenate([r * inv, -0.5 + 0.5 * r * r * inv], axis=1)
        g["W2"] += d_head.T @ s["u"]
        g["b2"] += d_head.sum(axis=0)
        d_pre = (d_head @ p["W2"]) * (s["u"] > 0.0)
        g["W1"] += d_pre.T @ s["z_prev"]
        g["b1"] += d_pre.sum(axis=0)
        g_z_prev = d_pre @ p["W1"]
        # guide: z = mu + sigma eps, and - log q contributes + log sigma
        d_mu = g_z.copy()
        d_sigma = g_z * eps[:, t] + 1.0 / s["sigma"]
        d_pre_sig = d_sigma * _sigmoid(s["pre_sig"])
        g["Wsig"] += d_pre_sig.T @ s["mu"]
        g["bsig"] += d_pre_sig.sum(axis=0)
        d_mu += d_pre_sig @ p["Wsig"]
        g["Wmu"] += d_mu.T @ s["h_out"]
        g["bmu"] += d_mu.sum(axis=0)
        d_h = (d_mu @ p["Wmu"]) / 3.0
        g_a[t] += d_h
        g_b[t] += d_h
        d_pre_c = d_h * (1.0 - s["comb"] ** 2)
        g["Wz"] += d_pre_c.T @ s["z_prev"]
        g["bz"] += d_pre_c.sum(axis=0)
        g_z_prev += d_pre_c @ p["Wz"]
        g_z_next = g_z_prev
    g["z0"] += g_z_next.sum(axis=0)
    # encoder RNNs
    carry = np.zeros((B, H))
    for t in range(W - 1, -1, -1):           # forward RNN, unrolled backwards
        d_pre = (g_a[t] + carry) * (a[t] > 0.0)
        prev = a[t - 1] if t > 0 else np.broadcast_to(p["a0"], (B, H))
        g["Wxf"] += d_pre.T @ x[:, t]
        g["Whf"] += d_pre.T @ prev
        g["bf"] += d_pre.sum(axis=0)
        carry = d_pre @ p["Whf"]
    g["a0"] += carry.sum(axis=0)
    carry = np.zeros((B, H))
    for t in range(W):                       # backward RNN: b_t depends on b_{t+1}
        d_pre = (g_b[t] + carry) * (b[t] > 0.0)
        prev = b[t + 1] if t + 1 < W else np.broadcast_to(p["b0"], (B, H))
        g["Wxb"] += d_pre.T @ x[:, t]
        g["Whb"] += d_pre.T @ prev
        g["bb"] += d_pre.sum(axis=0)
        carry = d_pre @ p["Whb"]
    g["b0"] += carry.sum(axis=0)
    return elbo, g


def gaussian_kl(mu_q, sigma_q, mu_p, sigma_p):
    """KL( N(mu_q, sigma_q^2) || N(mu_p, sigma_p^2) ), summed over dimensions (diagonal Gaussians)."""
    mu_q, sigma_q, mu_p, sigma_p = (np.asarray(v, dtype=np.float64) for v in (mu_q, sigma_q, mu_p, sigma_p))
    return float(np.sum(np.log(sigma_p / sigma_q) + (sigma_q ** 2 + (mu_q - mu_p) ** 2) / (2.0 * sigma_p ** 2) - 0.5))


def clip_by_global_norm(grads: dict, max_norm: float):
    """Scale all gradients by max_norm / ||g|| if their joint Euclidean norm exceeds max_norm.  Returns (grads, norm)."""
    norm = math.sqrt(sum(float(np.sum(g * g)) for g in grads.values()))
    if norm > max_norm:
        grads = {k: g * (max_norm / norm) for k, g in grads.items()}
    return grads, norm


class Adam:
    """Adam (Kingma & Ba 2015): bias-corrected first and second moment estimates, one state per tensor."""

    def __init__(self, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8):
        self.lr, self.beta1, self.beta2, self.eps = lr, beta1, beta2, eps
        self.t = 0
        self.m = {}
        self.v = {}

    def step(self, params: dict, grads: dict):
        """In place: params <- params - lr * m_hat / (sqrt(v_hat) + eps) for the gradient of a loss to minimise."""
        self.t += 1
        for k, g in grads.items():
            m = self.m.get(k, np.zeros_like(g))
            v = self.v.get(k, np.zeros_like(g))
            m = self.beta1 * m + (1.0 - self.beta1) * g
            v = self.beta2 * v + (1.0 - self.beta2) * g * g
            self.m[k], self.v[k] = m, v
            m_hat = m / (1.0 - self.beta1 ** self.t)
            v_hat = v / (1.0 - self.beta2 ** self.t)
            params[k] = params[k] - self.lr * m_hat / (np.sqrt(v_hat) + self.eps)


def windows_of(trace_normalised: np.ndarray, window: int) -> np.ndarray:
    """Every run of `window` consecutive vectors of a normalised trace [T, N] -> [T - window + 1, window, N]."""
    T = trace_normalised.shape[0]
    return np.stack([trace_normalised[t:t + window] for t in range(T - window + 1)])


def fit(weights: dict, trace_sec: np.ndarray, lag: int, steps: int, batch: int = 64, lr: float = 2e-3,
        clip: float = 10.0, seed: int = 0, log_every: int = 0):
    """Maximise the ELBO over all windows of a recorded trace by Adam with gradient clipping (Section 4.1).

    The trace is normalised as at run time: divided by twice the mean of its first window (Section 3.1.3, last
    paragraph).  Returns (fitted weights as float32 arrays, list of (step, mean ELBO per window of the batch)).
    """
    window = lag + 1
    scale = 2.0 * float(np.asarray(trace_sec[:window], dtype=np.float64).mean())
    data = windows_of(np.asarray(trace_sec, dtype=np.float64) / scale, window)
    params = {k: np.asarray(weights[k], dtype=np.float64).copy() for k in PARAMS}
    D = params["z0"].shape[0]
    rng = np.random.Generator(np.random.Philox(seed))
    opt = Adam(lr=lr)
    history = []
    for it in range(steps):
        idx = rng.integers(0, data.shape[0], size=batch)
        eps = rng.standard_normal((batch, window, D))
        elbo, grads = elbo_and_grad(params, data[idx], eps)
        loss_grads = {k: -g / batch for k, g in grads.items()}         # minimise the negative mean ELBO
        loss_grads, _ = clip_by_global_norm(loss_grads, clip)
        opt.step(params, loss_grads)
        if log_every and (it % log_every == 0 or it == steps - 1):
            history.append((it, float(elbo.mean())))
    return {k: v.astype(np.float32) for k, v in params.items()}, history
