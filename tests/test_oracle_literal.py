"""Pins for the oracle's literal networks (Section 3.1.3: gated transition, emission I / J).

Each test checks `transition_gated` or `emission_literal` against something that does not come from
the functions themselves: numbers worked out by hand, limits of the gate, the composition of two affine
maps, scalar loops written from the printed formulas, and the moments the Gaussian must have.
"""
import math

import numpy as np

from oracle import cutoff_oracle as co
from paper_1803_04209_b200 import inputs


def _w(**kw):
    return {k: np.asarray(v, dtype=np.float32) for k, v in kw.items()}


def test_gated_transition_hand_worked_scalar_case():
    # D = H = 1, z = 2.  gate: relu(1*2+0)=2 -> 0.5*2 + (ln 3 - 1) = ln 3 -> sigmoid = 3/4.
    # proposal: relu(-1*2+0)=0 -> h = 0*7 + 3 = 3.   linear: 0.25*2 + 1 = 1.5.
    # G = (1/4)*1.5 + (3/4)*3 = 2.625.   H = softplus(2*relu(2.625) - 5.25) = softplus(0) = ln 2.
    w = _w(Wg1=[[1.0]], bg1=[0.0], Wg2=[[0.5]], bg2=[math.log(3.0) - 1.0],
           Wh1=[[-1.0]], bh1=[0.0], Wh2=[[7.0]], bh2=[3.0],
           Wl=[[0.25]], bl=[1.0], Ws=[[2.0]], bs=[-5.25])
    z = np.array([[2.0]])
    for eps in (-1.5, 0.0, 2.0):
        out = co.transition_gated(z, w, np.array([[eps]]))
        assert abs(out[0, 0] - (2.625 + math.log(2.0) * eps)) < 1e-6     # bg2 is stored in fp32


def test_gate_limits_select_the_linear_map_or_the_proposal():
    rng = np.random.default_rng(0)
    D, H, K = 3, 5, 7
    w = inputs.make_weights_literal(4, D, H, seed=3, std=0.5, offsets=False)
    z = rng.standard_normal((K, D))
    zero = np.zeros((K, D))
    closed = dict(w); closed["Wg2"] = np.zeros_like(w["Wg2"]); closed["bg2"] = np.full(D, -60.0, np.float32)
    lin = z @ w["Wl"].astype(np.float64).T + w["bl"]
    assert np.allclose(co.transition_gated(z, closed, zero), lin, atol=1e-12)
    opened = dict(closed); opened["bg2"] = np.full(D, 60.0, np.float32)
    prop = np.maximum(z @ w["Wh1"].astype(np.float64).T + w["bh1"], 0) @ w["Wh2"].astype(np.float64).T + w["bh2"]
    assert np.allclose(co.transition_gated(z, opened, zero), prop, atol=1e-12)
    half = dict(closed); half["bg2"] = np.zeros(D, np.float32)
    assert np.allclose(co.transition_gated(z, half, zero), 0.5 * (lin + prop), atol=1e-12)


def test_gated_transition_against_scalar_loops():
    rng = np.random.default_rng(1)
    D, H, K = 4, 6, 3
    w = inputs.make_weights_literal(5, D, H, seed=9, std=0.7, offsets=False)
    z = rng.standard_normal((K, D)); eps = rng.standard_normal((K, D))
    got = co.transition_gated(z, w, eps)
    f = {k: v.astype(np.float64) for k, v in w.items()}
    for k in range(K):
        G = []
        for d in range(D):
            pre_g = f["bg2"][d]; pre_h = f["bh2"][d]
            for i in range(H):
                ug = max(f["bg1"][i] + sum(f["Wg1"][i][e] * z[k][e] for e in range(D)), 0.0)
                uh = max(f["bh1"][i] + sum(f["Wh1"][i][e] * z[k][e] for e in range(D)), 0.0)
                pre_g += f["Wg2"][d][i] * ug
                pre_h += f["Wh2"][d][i] * uh
            g = 1.0 / (1.0 + math.exp(-pre_g))
            lin = f["bl"][d] + sum(f["Wl"][d][e] * z[k][e] for e in range(D))
            G.append((1.0 - g) * lin + g * pre_h)
        for d in range(D):
            pre = f["bs"][d] + sum(f["Ws"][d][e] * max(G[e], 0.0) for e in range(D))
            want = G[d] + math.log1p(math.exp(pre)) * eps[k][d]
            assert abs(got[k][d] - want) < 1e-12


def test_literal_emission_mean_is_the_composed_affine_map_and_scale_reads_the_mean():
    rng = np.random.default_rng(2)
    N, D, H, K = 6, 3, 5, 4
    w = inputs.make_weights_literal(N, D, H, seed=5, std=0.6, offsets=False)
    f = {k: v.astype(np.float64) for k, v in w.items()}
    z = rng.standard_normal((K, D))
    A = f["Wi2"] @ f["Wi1"]; c = f["Wi2"] @ f["bi1"] + f["bi2"]
    mean = z @ A.T + c
    assert np.allclose(co.emission_literal(z, w, np.zeros((K, N))), mean, atol=1e-12)
    # the scale is a function of the mean alone: two latents with the same mean get the same scale
    one = np.ones((K, N))
    scale = co.emission_literal(z, w, one) - mean
    for k in range(K):
        for j in range(N):
            pre = f["bj2"][j]
            for i in range(H):
                pre += f["Wj2"][j][i] * max(f["bj1"][i] + sum(f["Wj1"][i][m] * mean[k][m] for m in range(N)), 0.0)
            assert abs(scale[k][j] - math.log1p(math.exp(pre))) < 1e-12
    assert np.all(scale > 0)


def test_literal_emission_hand_worked_scalar_case():
    # N = D = H = 1, z = 3:  I = 2*(0.5*3 + 1) - 4 = 1.   J = softplus(4*relu(-1*1 + 1.5) - 2) = softplus(0) = ln 2.
    w = _w(Wi1=[[0.5]], bi1=[1.0], Wi2=[[2.0]], bi2=[-4.0], Wj1=[[-1.0]], bj1=[1.5], Wj2=[[4.0]], bj2=[-2.0])
    out = co.emission_literal(np.array([[3.0]]), w, np.array([[-2.0]]))
    assert abs(out[0, 0] - (1.0 - 2.0 * math.log(2.0))) < 1e-12


def test_second_argument_is_a_standard_deviation():
    # with weights that make G = 0 and H = softplus(bs), the draws have standard deviation softplus(bs), not its root
    D, K = 2, 200000
    w = {k: np.zeros(s, np.float32) for k, s in inputs.tensor_shapes_literal(3, D, 4).items()}
    w["bs"] = np.full(D, 1.3, np.float32)
    eps = co.normals(5, 0, co.STREAM_TRANSITION, np.arange(K), D)
    out = co.transition_gated(np.zeros((K, D)), w, eps)
    sd = math.log1p(math.exp(float(np.float32(1.3))))
    assert abs(out.std() - sd) < 0.01 and abs(out.mean()) < 0.01
    w["bj2"] = np.full(3, -0.4, np.float32)
    x = co.emission_literal(np.zeros((K, D)), w, co.normals(5, 0, co.STREAM_EMISSION, np.arange(K), 3))
    assert abs(x.std() - math.log1p(math.exp(float(np.float32(-0.4))))) < 0.01


def test_literal_weights_select_the_literal_networks_in_the_decision():
    wl = inputs.WORKLOADS["tiny"]
    w = inputs.workload_weights_literal(wl)
    trace = inputs.workload_trace(wl, wl.window + 2)
    orc = co.CutoffOracle(w, wl.lag, 256, seed=4)
    for x in trace: orc.push(x)
    k = np.arange(8)
    xhat = orc.xhat()
    a, b = co.encoder(xhat, w)
    eps_q = np.stack([co.normals(4, 0, t, k, wl.D) for t in range(wl.window)], axis=1)
    z = co.guide_chain(a, b, w, eps_q)
    z = co.transition_gated(z, w, co.normals(4, 0, co.STREAM_TRANSITION, k, wl.D))
    want = co.emission_literal(z, w, co.normals(4, 0, co.STREAM_EMISSION, k, wl.N))
    assert np.array_equal(orc.samples(k), want)
    code, c, expected, omega = orc.predict()
    assert code == co.OK and 1 <= c <= wl.N and np.all(np.diff(expected) >= 0)
    # a fitted-regime model predicts times near the data's own scale (normalised mean 0.5)
    assert 0.2 * trace.mean() < expected.mean() < 3.0 * trace.mean()
