"""CPU oracle for the run-time cutoff decision of Cutoff SGD (Teng & Wood, 2018).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  This file is the plain, slow,
double-precision statement of what the library computes.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it.  It shares no
code with the CUDA path and imports nothing from it.

What it computes, in the paper's order and notation:

  Algorithm 1, parameter-server branch: ``c <- predict_cutoff(q_phi, obs)``
  once per SGD step; ``obs`` grows by the run-times r_w that arrive.

  Section 3 ("Methodology"): throughput Omega(c) = c / x~_(c) over the
  *ordered* run-times, decision argmax_c Omega(c).

  Section 3.1.1 ("Order Statistics"), last paragraph: Monte-Carlo order
  statistics -- sample the joint run-times, sort, record, repeat.

  Section 3.1.3 ("Model Learning and Amortized Inference"): the guide q_phi
  (forward / backward ReLU RNNs over the lagged window, a tanh combiner,
  Gaussian heads), the transition z_t ~ N(G(z_{t-1}), H(z_{t-1})), the emission
  x_t ~ N(I(z_t), J(z_t)), and the K-sample approximation of the posterior
  predictive (the display after Eq. 4): z_T^(k) is the last-step marginal of
  the k-th draw from q_phi.

  Section 3.1.3, last paragraph: observations are divided by twice the mean of
  the first fixed-lag window.

The method is a Monte-Carlo approximation, so the oracle follows the algorithm
step by step and draws its noise from the same counter-based generator as the
library: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) feeding the basic
Box-Muller transform.  Both are written here from their published definitions.

Pins (see tests/test_oracle_*.py): Philox against the published known-answer
vectors, against a second big-integer implementation and against its own
inverse; Box-Muller against N(0,1) moments and a KS test; the sort/mean/argmax
tail against the iid-normal order-statistic integral of Section 3.1.1, the
worked example of Section 4.1 and brute force; the networks against
linear-Gaussian closed forms and special cases; ``encoder`` and ``guide_chain``
with dense, non-symmetric weights, non-zero initial states and noise against
scalar loops written element by element from the guide equations.

Model variants.  "compact": transition and emission are one-hidden-layer ReLU
MLPs with a (mean, log-variance) head (``transition`` / ``emission``).
"literal": the networks as Section 3.1.3 prints them -- the gated transition
G, H and the emission I = MLP_2(z, Identity, Identity), J = MLP_2(I, ReLU,
Softplus) (``transition_gated`` / ``emission_literal``); there the second
argument of N(.,.) is taken as a standard deviation, like the guide's sigma.
A weight dictionary that holds "Wg1" selects the literal variant.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------
# Philox4x32-10 (Salmon et al., SC'11, Section 3.3 and Table 2 constants)
# ----------------------------------------------------------------------------
_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)     # golden ratio
_W1 = np.uint64(0xBB67AE85)     # sqrt(3) - 1
_MASK = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)

STREAM_TRANSITION = 0x100       # guide step t uses stream t (0 .. lag)
STREAM_EMISSION = 0x200
STREAM_IMPUTE = 0x300           # where the scan for a censored worker's replacement starts


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds of the Philox-4x32 bijection.

    All arguments are arrays (or scalars) of 32-bit values and broadcast
    against each other.  Returns the four 32-bit output words as uint64 arrays
    holding values < 2**32.
    """
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK
    k0 = np.asarray(k0, dtype=np.uint64) & _MASK
    k1 = np.asarray(k1, dtype=np.uint64) & _MASK
    for rnd in range(10):
        if rnd > 0:                       # key schedule: a Weyl sequence per key word
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0                     # 32x32 -> 64 bit products
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _SH32, p0 & _MASK
        hi1, lo1 = p1 >> _SH32, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return c0, c1, c2, c3


def box_muller(r_a, r_b):
    """Two standard normals from two 32-bit words (Box & Muller 1958, basic form).

    u1 = (top 24 bits of r_a + 1) / 2**24 lies in (0, 1]; u2 = (top 24 bits of
    r_b) / 2**24 lies in [0, 1).  Both are exact in single precision.
    """
    u1 = ((np.asarray(r_a, dtype=np.uint64) >> np.uint64(8)).astype(np.float64) + 1.0) * 2.0 ** -24
    u2 = (np.asarray(r_b, dtype=np.uint64) >> np.uint64(8)).astype(np.float64) * 2.0 ** -24
    radius = np.sqrt(-2.0 * np.log(u1))
    angle = 2.0 * np.pi * u2
    return radius * np.cos(angle), radius * np.sin(angle)


def normals(seed: int, step: int, stream: int, k, n_elems: int) -> np.ndarray:
    """Standard normals eps[k, e] for sample indices ``k`` and elements e < n_elems.

    One Philox call serves elements 4q .. 4q+3 of one (sample, stream, step):
    counter = (q, k, stream, step), key = (seed low word, seed high word);
    output words (r0, r1) give elements 4q, 4q+1 and (r2, r3) give 4q+2, 4q+3.
    """
    k = np.asarray(k, dtype=np.uint64).reshape(-1, 1)
    nq = (n_elems + 3) // 4
    q = np.arange(nq, dtype=np.uint64).reshape(1, -1)
    r0, r1, r2, r3 = philox4x32_10(q, k, stream, step, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    e0, e1 = box_muller(r0, r1)
    e2, e3 = box_muller(r2, r3)
    eps = np.stack([e0, e1, e2, e3], axis=-1).reshape(k.shape[0], 4 * nq)
    return eps[:, :n_elems]


# ----------------------------------------------------------------------------
# Observations: window and normaliser (Section 3.1.3, last paragraph)
# ----------------------------------------------------------------------------
def normaliser(history: np.ndarray, window: int) -> float:
    """s = 2 x mean over every entry of the first ``window`` pushed vectors."""
    first = np.asarray(history[:window], dtype=np.float64)
    return 2.0 * float(first.mean())


# ----------------------------------------------------------------------------
# Guide q_phi (Section 3.1.3: h_left, h_right, h_out, mu_q, sigma_q)
# ----------------------------------------------------------------------------
def _f64(w: dict) -> dict:
    return {name: np.asarray(v, dtype=np.float64) for name, v in w.items()}


def relu(v):
    return np.maximum(v, 0.0)


def softplus(v):
    return np.logaddexp(0.0, v)


def encoder(xhat: np.ndarray, w: dict):
    """h_left and h_right for every window position.

    xhat is the normalised window [W, N], oldest first.  a[t] summarises
    xhat[0..t] (forward ReLU RNN from the learned state a0); b[t] summarises
    xhat[t..W-1] (backward ReLU RNN from b0).  Both include position t, so
    that the last latent sees the newest observation.
    """
    w = _f64(w)
    W = xhat.shape[0]
    H = w["bf"].shape[0]
    a = np.zeros((W, H))
    b = np.zeros((W, H))
    state = w["a0"]
    for t in range(W):
        state = relu(w["Wxf"] @ xhat[t] + w["Whf"] @ state + w["bf"])
        a[t] = state
    state = w["b0"]
    for t in range(W - 1, -1, -1):
        state = relu(w["Wxb"] @ xhat[t] + w["Whb"] @ state + w["bb"])
        b[t] = state
    return a, b


def guide_chain(a: np.ndarray, b: np.ndarray, w: dict, eps: np.ndarray) -> np.ndarray:
    """Draw z_T^(k) for every sample k by ancestral sampling through q_phi.

    eps[k, t, :] is the standard-normal draw of sample k at window step t.
    h_out = (tanh-layer(z_{t-1}) + h_left + h_right) / 3; mu = linear(h_out);
    sigma = softplus(linear(mu)); z_t = mu + sigma * eps.  sigma is a standard
    deviation.
    """
    w = _f64(w)
    S, W, D = eps.shape
    z = np.broadcast_to(w["z0"], (S, D))
    for t in range(W):
        comb = np.tanh(z @ w["Wz"].T + w["bz"])
        h_out = (comb + a[t] + b[t]) / 3.0
        mu = h_out @ w["Wmu"].T + w["bmu"]
        sigma = softplus(mu @ w["Wsig"].T + w["bsig"])
        z = mu + sigma * eps[:, t, :]
    return z


# ----------------------------------------------------------------------------
# Generative model p_theta (Section 3.1.3: transition and emission)
# ----------------------------------------------------------------------------
def transition(z: np.ndarray, w: dict, eps: np.ndarray) -> np.ndarray:
    """z_{T+1} ~ N(G(z_T), H(z_T)): hidden ReLU layer, then mean and log-variance heads."""
    w = _f64(w)
    D = z.shape[1]
    u = relu(z @ w["W1"].T + w["b1"])
    head = u @ w["W2"].T + w["b2"]
    mean, logvar = head[:, :D], head[:, D:]
    return mean + np.exp(0.5 * logvar) * eps


def emission(z: np.ndarray, w: dict, eps: np.ndarray) -> np.ndarray:
    """x_{T+1} ~ N(I(z_{T+1}), J(z_{T+1})): one run-time per worker, in normalised units."""
    w = _f64(w)
    N = eps.shape[1]
    v = relu(z @ w["W3"].T + w["b3"])
    head = v @ w["W4"].T + w["b4"]
    mean, logvar = head[:, :N], head[:, N:]
    return mean + np.exp(0.5 * logvar) * eps


def sigmoid(v):
    return 1.0 / (1.0 + np.exp(-v))


def transition_gated(z: np.ndarray, w: dict, eps: np.ndarray) -> np.ndarray:
    """The gated transition of Section 3.1.3, z_{T+1} = G + H * eps with

        g = MLP_2(z, ReLU, Sigmoid)          h = MLP_2(z, ReLU, Identity)
        G = (1 - g) * MLP_1(z, Identity) + g * h
        H = MLP_1(ReLU(G), Softplus)         (a standard deviation)
    """
    w = _f64(w)
    g = sigmoid(relu(z @ w["Wg1"].T + w["bg1"]) @ w["Wg2"].T + w["bg2"])
    h = relu(z @ w["Wh1"].T + w["bh1"]) @ w["Wh2"].T + w["bh2"]
    G = (1.0 - g) * (z @ w["Wl"].T + w["bl"]) + g * h
    H = softplus(relu(G) @ w["Ws"].T + w["bs"])
    return G + H * eps


def emission_literal(z: np.ndarray, w: dict, eps: np.ndarray) -> np.ndarray:
    """The emission of Section 3.1.3, x_{T+1} = I + J * eps with

        I = MLP_2(z, Identity, Identity)     (two affine layers: the mean of every worker)
        J = MLP_2(I, ReLU, Softplus)         (a standard deviation, computed from the mean)
    """
    w = _f64(w)
    I = (z @ w["Wi1"].T + w["bi1"]) @ w["Wi2"].T + w["bi2"]
    J = softplus(relu(I @ w["Wj1"].T + w["bj1"]) @ w["Wj2"].T + w["bj2"])
    return I + J * eps


def is_literal(w: dict) -> bool:
    return "Wg1" in w


def n_workers(w: dict) -> int:
    return w["bi2"].shape[0] if is_literal(w) else w["b4"].shape[0] // 2


def sample_runtimes(w: dict, xhat: np.ndarray, seed: int, step: int, k) -> np.ndarray:
    """Posterior-predictive draws x^(k)_{T+1} (normalised units), one row per sample index."""
    k = np.asarray(k, dtype=np.int64).reshape(-1)
    W = xhat.shape[0]
    D = w["z0"].shape[0]
    N = n_workers(w)
    a, b = encoder(xhat, w)
    eps_q = np.stack([normals(seed, step, t, k, D) for t in range(W)], axis=1)
    z_T = guide_chain(a, b, w, eps_q)
    eps_tr = normals(seed, step, STREAM_TRANSITION, k, D)
    eps_em = normals(seed, step, STREAM_EMISSION, k, N)
    if is_literal(w):
        return emission_literal(transition_gated(z_T, w, eps_tr), w, eps_em)
    return emission(transition(z_T, w, eps_tr), w, eps_em)


# ----------------------------------------------------------------------------
# Order statistics, throughput, decision (Sections 3 and 3.1.1)
# ----------------------------------------------------------------------------
def expected_order_statistics(x: np.ndarray) -> np.ndarray:
    """Sort every sampled vector ascending, then average position by position."""
    return np.sort(x, axis=1, kind="stable").mean(axis=0)


def order_statistic_std(x: np.ndarray) -> np.ndarray:
    """Standard deviation over the samples of each sorted position (the +-2 sigma bands of Fig. 3)."""
    return np.sort(x, axis=1, kind="stable").std(axis=0)


def throughput(expected_sorted: np.ndarray) -> np.ndarray:
    """Omega(c) = c / E[x~_(c)] for c = 1..N; minus infinity where the expectation is not positive."""
    e = np.asarray(expected_sorted, dtype=np.float64)
    c = np.arange(1, e.shape[0] + 1, dtype=np.float64)
    omega = np.full(e.shape, -np.inf)
    ok = e > 0.0
    omega[ok] = c[ok] / e[ok]
    return omega


def argmax_cutoff(omega: np.ndarray):
    """(c*, degenerate): the largest c attaining the maximum; c = N if no c is admissible."""
    n = omega.shape[0]
    best = -np.inf
    c_star = n
    for c in range(1, n + 1):          # c in {1..N}, ties go to the larger c
        if omega[c - 1] >= best and omega[c - 1] > -np.inf:
            best = omega[c - 1]
            c_star = c
    return c_star, bool(best == -np.inf)


def impute_censored(runtimes_sec, censored, predictive_sec, seed: int, step: int):
    """Replace censored run-times by draws from the predictive distribution, left-truncated at the cutoff time.

    Section 4.2 ("Handling Censored Run-times"): stragglers are killed once c gradients have arrived,
    so their run-times are only known to exceed the cutoff time -- the largest run-time that was
    observed in this step.  Each censored worker gets a draw from its own predictive distribution for
    this step, p(x; x > cutoff time) = p(x) / P(x > cutoff time).  The predictive distribution is the
    Monte-Carlo one: predictive_sec[k, j] is the k-th predictive draw of worker j (seconds).  The draws
    are iid, so taking the first one above the threshold, scanning cyclically from a start index that
    does not depend on their values, is an exact draw from the truncated distribution.  The start is
    Philox word 0 of counter (worker, 0, STREAM_IMPUTE, step) modulo the number of draws.  If no draw of
    a worker exceeds the threshold, the threshold itself is used (all that is known).
    """
    x = np.array(runtimes_sec, dtype=np.float64)
    censored = np.asarray(censored).astype(bool)
    if not censored.any():
        return x, None
    assert not censored.all(), "at least one worker must have finished"
    threshold = float(x[~censored].max())
    S = predictive_sec.shape[0]
    for j in np.flatnonzero(censored):
        word0 = int(philox4x32_10(int(j), 0, STREAM_IMPUTE, step, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)[0])
        start = word0 % S
        column = np.roll(predictive_sec[:, j], -start)          # scan order: start, start+1, ..., wrapping
        above = np.flatnonzero(column > threshold)
        x[j] = column[above[0]] if above.size else threshold
    return x, threshold


OK, WARMUP, DEGENERATE = 0, 1, 2


class CutoffOracle:
    """The parameter server's view: push observed run-times, ask for the cutoff.

    Mirrors the call order of Algorithm 1: ``predict`` before the step's
    run-times arrive, ``push`` once they have.
    """

    def __init__(self, weights: dict, lag: int, n_samples: int, seed: int, chunk: int = 2048):
        self.w = weights
        self.window = lag + 1
        self.S = n_samples
        self.seed = seed
        self.chunk = chunk
        self.N = n_workers(weights)
        self.reset()

    def reset(self):
        self.history = []
        self.step = 0
        self.last_draws_sec = None       # predictive draws of the last decision, seconds, [S, N]

    def push(self, runtimes_sec, censored=None):
        """obs <- obs U r_w.  `censored` marks workers whose run-time was not observed (Section 4.2)."""
        x = np.asarray(runtimes_sec, dtype=np.float32)
        assert x.shape == (self.N,)
        if censored is not None and np.any(censored):
            assert self.last_draws_sec is not None, "imputation needs the predictive draws of this step"
            x64, _ = impute_censored(np.where(np.asarray(censored).astype(bool), 0.0, x), censored,
                                     self.last_draws_sec, self.seed, self.step)
            x = x64.astype(np.float32)
        assert np.all(np.isfinite(x)) and np.all(x > 0)
        self.history.append(x.copy())

    def scale(self) -> float:
        return normaliser(np.stack(self.history[: self.window]), self.window)

    def xhat(self) -> np.ndarray:
        return np.stack(self.history[-self.window:]).astype(np.float64) / self.scale()

    def samples(self, k) -> np.ndarray:
        """Unsorted predictive draws in normalised units for the coming decision."""
        return sample_runtimes(self.w, self.xhat(), self.seed, self.step, k)

    def predict(self):
        """Returns (code, c, E[x~_(j)] in seconds, Omega(c) per second)."""
        if len(self.history) < self.window:      # obs too short: wait for everyone
            return WARMUP, self.N, None, None
        s = self.scale()
        rows = [self.samples(np.arange(k0, min(k0 + self.chunk, self.S)))   # rows are independent:
                for k0 in range(0, self.S, self.chunk)]                     # chunking only bounds memory
        draws = np.concatenate(rows, axis=0)
        ordered = np.sort(draws, axis=1, kind="stable")      # sorted once, used for the mean and for the spread
        self.last_draws_sec = s * draws
        self.last_std_sec = s * ordered.std(axis=0)
        expected = s * ordered.mean(axis=0)
        omega = throughput(expected)
        c, degenerate = argmax_cutoff(omega)
        self.step += 1
        return (DEGENERATE if degenerate else OK), c, expected, omega
