"""Seeded synthetic inputs: model weights and worker run-time traces.

This module holds no arithmetic of the cutoff method itself.  It only draws
random weights and random run-time traces, so that the CUDA library and the
CPU oracle can be fed the very same arrays.  It imports neither of them.

The recorded cluster traces and trained networks of the paper were never
released, so the traces below stand in for them.  They are shaped on what the
paper says about its clusters: iterations of about one second with a spread
of a few tenths of a second (Section 4.1), groups of co-located workers that
slow down together for long stretches and then recover (Section 2.1 and the
two "dynamical modes" of Section 4.1), and a thin tail of stragglers
(Section 1).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# Order and shapes of the model tensors.  N workers, D latent size, H hidden
# width.  Every matrix is row-major [outputs x inputs].
#   encoder RNNs (guide, h_left / h_right):  Wxf Whf bf a0 | Wxb Whb bb b0
#   guide combiner and heads:                Wz bz Wmu bmu Wsig bsig z0
#   transition MLP (mean | log-variance):    W1 b1 W2 b2
#   emission MLP   (mean | log-variance):    W3 b3 W4 b4
TENSOR_ORDER = (
    "Wxf", "Whf", "bf", "a0", "Wxb", "Whb", "bb", "b0",
    "Wz", "bz", "Wmu", "bmu", "Wsig", "bsig", "z0",
    "W1", "b1", "W2", "b2", "W3", "b3", "W4", "b4",
)


def tensor_shapes(N: int, D: int, H: int) -> dict:
    return {
        "Wxf": (H, N), "Whf": (H, H), "bf": (H,), "a0": (H,),
        "Wxb": (H, N), "Whb": (H, H), "bb": (H,), "b0": (H,),
        "Wz": (H, D), "bz": (H,), "Wmu": (D, H), "bmu": (D,),
        "Wsig": (D, D), "bsig": (D,), "z0": (D,),
        "W1": (H, D), "b1": (H,), "W2": (2 * D, H), "b2": (2 * D,),
        "W3": (H, D), "b3": (H,), "W4": (2 * N, H), "b4": (2 * N,),
    }


# The networks as Section 3.1.3 prints them ("literal" variant): the guide tensors
# are the same; the generative model has
#   gated transition:  gate Wg1 bg1 Wg2 bg2 | proposal Wh1 bh1 Wh2 bh2 | linear Wl bl | scale Ws bs
#   emission:          mean Wi1 bi1 Wi2 bi2 (two affine layers) | scale Wj1 bj1 Wj2 bj2 (input: the mean)
GUIDE_TENSORS = TENSOR_ORDER[:15]
TENSOR_ORDER_LITERAL = GUIDE_TENSORS + (
    "Wg1", "bg1", "Wg2", "bg2", "Wh1", "bh1", "Wh2", "bh2", "Wl", "bl", "Ws", "bs",
    "Wi1", "bi1", "Wi2", "bi2", "Wj1", "bj1", "Wj2", "bj2",
)


def tensor_shapes_literal(N: int, D: int, H: int) -> dict:
    base = tensor_shapes(N, D, H)
    shapes = {k: base[k] for k in GUIDE_TENSORS}
    shapes.update({
        "Wg1": (H, D), "bg1": (H,), "Wg2": (D, H), "bg2": (D,),
        "Wh1": (H, D), "bh1": (H,), "Wh2": (D, H), "bh2": (D,),
        "Wl": (D, D), "bl": (D,), "Ws": (D, D), "bs": (D,),
        "Wi1": (H, D), "bi1": (H,), "Wi2": (N, H), "bi2": (N,),
        "Wj1": (H, N), "bj1": (H,), "Wj2": (N, H), "bj2": (N,),
    })
    return shapes


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16-representable fp32 (ties to even)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def make_weights(N: int, D: int, H: int, seed: int = 0, std: float = 0.1,
                 fan_in_ref: int | None = None, offsets: bool = True,
                 bf16: bool = False) -> dict:
    """Random-initialised weights.

    Every tensor, biases included, is drawn from a zero-mean Gaussian.  With
    ``fan_in_ref=None`` the standard deviation is ``std`` for every tensor.
    With ``fan_in_ref=r`` a matrix with more than ``r`` inputs uses
    ``std*sqrt(r/inputs)`` so that pre-activations keep the scale they have
    in the smallest configuration instead of growing with the layer width.
    The initial latent and RNN states are zero.

    ``offsets=True`` then moves the untrained model into the regime a fitted
    one works in, where predicted times are positive and of the right order
    for normalised data (observations are divided by twice their mean, so
    they average 0.5):
      emission mean head      weights and bias halved, then bias += 0.5
      emission log-variance   bias += 2 ln 0.05   (noise of about 0.05)
      transition log-variance bias += 2 ln 0.1    (a slowly moving latent)
    ``offsets=False`` leaves the raw draw, whose predicted times are often
    negative; it exercises the rule for non-positive expectations.
    """
    rng = np.random.Generator(np.random.Philox(seed))
    w = {}
    for name, shape in tensor_shapes(N, D, H).items():
        if name in ("a0", "b0", "z0"):
            w[name] = np.zeros(shape, dtype=np.float32)
            continue
        sd = std
        if fan_in_ref is not None and len(shape) == 2 and shape[1] > fan_in_ref:
            sd = std * math.sqrt(fan_in_ref / shape[1])
        w[name] = (rng.standard_normal(shape) * sd).astype(np.float32)
    if offsets:
        w["W4"][:N] *= np.float32(0.5)
        w["b4"][:N] = w["b4"][:N] * np.float32(0.5) + np.float32(0.5)
        w["b4"][N:] += np.float32(2.0 * math.log(0.05))
        w["b2"][D:] += np.float32(2.0 * math.log(0.1))
    if bf16:
        w = {k: round_to_bf16(v) for k, v in w.items()}
    return w


def make_weights_literal(N: int, D: int, H: int, seed: int = 0, std: float = 0.1,
                         fan_in_ref: int | None = None, offsets: bool = True, bf16: bool = False) -> dict:
    """Random-initialised weights of the literal variant, drawn like `make_weights`.

    ``offsets=True`` moves the untrained model into the regime of a fitted one:
      emission mean        last layer and bias halved, then bias += 0.5
      emission scale       bias += softplus^-1(0.05)   (noise of about 0.05)
      transition scale     bias += softplus^-1(0.1)    (a slowly moving latent)
    """
    rng = np.random.Generator(np.random.Philox(seed))
    w = {}
    for name, shape in tensor_shapes_literal(N, D, H).items():
        if name in ("a0", "b0", "z0"):
            w[name] = np.zeros(shape, dtype=np.float32)
            continue
        sd = std
        if fan_in_ref is not None and len(shape) == 2 and shape[1] > fan_in_ref:
            sd = std * math.sqrt(fan_in_ref / shape[1])
        w[name] = (rng.standard_normal(shape) * sd).astype(np.float32)
    if offsets:
        w["Wi2"] *= np.float32(0.5)
        w["bi2"] = w["bi2"] * np.float32(0.5) + np.float32(0.5)
        w["bj2"] += np.float32(math.log(math.expm1(0.05)))
        w["bs"] += np.float32(math.log(math.expm1(0.1)))
    if bf16:
        w = {k: round_to_bf16(v) for k, v in w.items()}
    return w


@dataclass(frozen=True)
class Workload:
    name: str
    N: int
    D: int
    H: int
    lag: int            # the paper's l; the window holds lag+1 vectors
    S: int              # Monte-Carlo samples (the paper's K)
    history: int        # run-time vectors pushed before the measured decision
    precision: int      # 0 fp32 FMA, 1 tf32 tensor cores, 2 bf16 weights + fp32 accumulate
    weight_seed: int = 0
    trace_seed: int = 0
    trace: dict = field(default_factory=dict)

    @property
    def window(self) -> int:
        return self.lag + 1


WORKLOADS = {
    "tiny": Workload("tiny", N=16, D=4, H=32, lag=1, S=1024, history=20, precision=0,
                     trace_seed=1, trace=dict(sigma=0.25)),
    "n128": Workload("n128", N=128, D=8, H=128, lag=2, S=16384, history=200, precision=0,
                     trace_seed=2, trace=dict(sigma=0.2, groups=4, stay=0.95, slowdown=2.0)),
    "n1024": Workload("n1024", N=1024, D=16, H=256, lag=4, S=65536, history=500, precision=1,
                      trace_seed=3, trace=dict(sigma=0.3, groups=16, stay=0.9, slowdown=2.0,
                                               straggler_p=0.02, straggler="exp", straggler_scale=1.5)),
    "n4096": Workload("n4096", N=4096, D=32, H=512, lag=4, S=32768, history=500, precision=2,
                      trace_seed=4, trace=dict(sigma=0.25, groups=64, stay=0.9, slowdown=2.0,
                                               straggler_p=0.01, straggler="pareto", straggler_scale=1.0,
                                               pareto_alpha=2.0)),
    "stream": Workload("stream", N=1024, D=16, H=256, lag=4, S=8192, history=1005, precision=1,
                       trace_seed=7, trace=dict(sigma=0.3, groups=16, stay=0.9, slowdown=2.0,
                                                straggler_p=0.02, straggler="exp", straggler_scale=1.5)),
    # shape-only cases: the worker counts of the paper's two clusters and its lag of 20
    "n158": Workload("n158", N=158, D=8, H=64, lag=20, S=2048, history=40, precision=0,
                     trace_seed=5, trace=dict(sigma=0.3, groups=4, stay=0.95, slowdown=2.0)),
    "n2175": Workload("n2175", N=2175, D=16, H=128, lag=20, S=1024, history=30, precision=1,
                      trace_seed=6, trace=dict(sigma=0.3, groups=32, stay=0.9, slowdown=2.0,
                                               straggler_p=0.01, straggler="exp", straggler_scale=1.5)),
}


def workload_weights_literal(wl: Workload, offsets: bool = True) -> dict:
    return make_weights_literal(wl.N, wl.D, wl.H, seed=wl.weight_seed, std=0.1, fan_in_ref=32, offsets=offsets,
                                bf16=(wl.precision == 2))


def workload_weights(wl: Workload, offsets: bool = True) -> dict:
    return make_weights(wl.N, wl.D, wl.H, seed=wl.weight_seed, std=0.1, fan_in_ref=32,
                        offsets=offsets, bf16=(wl.precision == 2))


def make_trace(N: int, steps: int, seed: int, sigma: float, groups: int = 0,
               stay: float = 1.0, slowdown: float = 1.0, straggler_p: float = 0.0,
               straggler: str = "exp", straggler_scale: float = 1.0,
               pareto_alpha: float = 2.0) -> np.ndarray:
    """Run-times in seconds, shape [steps, N], fp32, all finite and > 0.

    base      lognormal(0, sigma) per worker per step, independent
    groups    workers split into ``groups`` equal contiguous groups (the last
              takes the remainder); each group carries a two-state Markov
              chain (clear / contended) that keeps its state with probability
              ``stay``; a contended group's times are multiplied by
              ``slowdown``.  Group 0 starts contended, the others clear.
    straggler with probability ``straggler_p`` a worker's time gets an extra
              Exp(mean straggler_scale) or Pareto(alpha, scale) seconds.
    """
    rng = np.random.Generator(np.random.Philox(seed))
    x = np.exp(rng.standard_normal((steps, N)) * sigma)
    if groups > 0:
        gsize = max(1, N // groups)
        gid = np.minimum(np.arange(N) // gsize, groups - 1)
        state = np.zeros(groups, dtype=bool)
        state[0] = True
        for t in range(steps):
            x[t] *= np.where(state[gid], slowdown, 1.0)
            flip = rng.random(groups) >= stay
            state = np.where(flip, ~state, state)
    if straggler_p > 0.0:
        hit = rng.random((steps, N)) < straggler_p
        if straggler == "exp":
            extra = rng.exponential(straggler_scale, size=(steps, N))
        elif straggler == "pareto":
            extra = straggler_scale * (1.0 - rng.random((steps, N))) ** (-1.0 / pareto_alpha)
        else:
            raise ValueError(f"unknown straggler kind {straggler!r}")
        x += np.where(hit, extra, 0.0)
    return x.astype(np.float32)


def workload_trace(wl: Workload, steps: int | None = None) -> np.ndarray:
    return make_trace(wl.N, wl.history if steps is None else steps, wl.trace_seed, **wl.trace)
