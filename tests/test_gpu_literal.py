"""Parity of the literal model variant (Section 3.1.3 as printed: gated transition, emission I / J) with
the CPU oracle, through the C ABI, on a real GPU.  Tolerances as in test_gpu_parity.py."""
import numpy as np
import pytest

from oracle import cutoff_oracle as O
from paper_1803_04209_b200 import binding, build, inputs
from test_gpu_parity import SEED, TOL_X, assert_decision_close, assert_samples_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    import torch
    assert torch.cuda.is_available(), "these tests need a GPU"
    build.build()
    return binding.load_library()


def make_pair(name, S=None, steps=None, offsets=True, precision=None, seed=SEED, flags=0, **kw):
    wl = inputs.WORKLOADS[name]
    S = S or wl.S
    w = inputs.workload_weights_literal(wl, offsets=offsets)
    trace = inputs.workload_trace(wl, steps)
    prec = wl.precision if precision is None else precision
    gpu = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=prec, seed=seed, flags=flags | binding.FLAG_LITERAL, **kw)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, wl.lag, S, seed=seed)
    assert O.is_literal(w)
    for x in trace:
        gpu.push(x)
        orc.push(x)
    return wl, gpu, orc, prec


@pytest.mark.parametrize("name,S,offsets", [("tiny", 1024, True), ("tiny", 1024, False), ("n128", 2048, True),
                                            ("n128", 777, False), ("n158", 512, True)])
def test_sampled_runtimes_fp32(name, S, offsets):
    wl, gpu, orc, prec = make_pair(name, S=S, offsets=offsets)
    x_gpu = gpu.debug_samples(0, S)
    assert_samples_close(x_gpu, orc.samples(np.arange(S)), TOL_X[prec])
    assert np.array_equal(gpu.debug_samples(100, 50), x_gpu[100:150])


@pytest.mark.parametrize("name,S,offsets", [("tiny", 1024, True), ("tiny", 1024, False), ("n128", 4096, True),
                                            ("n158", 1024, True)])
def test_decision_fp32(name, S, offsets):
    wl, gpu, orc, prec = make_pair(name, S=S, offsets=offsets)
    assert_decision_close(gpu, orc.predict(), wl.N)


def test_wide_models_fp32_arithmetic():
    for name, S in (("n1024", 300), ("n2175", 200), ("n4096", 130)):
        wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 3, precision=0)
        assert_samples_close(gpu.debug_samples(0, S), orc.samples(np.arange(S)), 1e-5)
        assert_decision_close(gpu, orc.predict(), wl.N)


@pytest.mark.parametrize("name,S", [("n1024", 1024), ("n1024", 130), ("n2175", 300), ("n4096", 384), ("stream", 256)])
def test_sampled_runtimes_tensor_cores(name, S):
    wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 3)
    assert prec in (1, 2)
    x_gpu = gpu.debug_samples(0, S)
    assert_samples_close(x_gpu, orc.samples(np.arange(S)), TOL_X[prec])
    assert np.array_equal(gpu.debug_samples(S // 2, 7), x_gpu[S // 2: S // 2 + 7])


@pytest.mark.parametrize("name,S,offsets", [("n1024", 4096, True), ("n1024", 1000, False), ("n2175", 512, True),
                                            ("n4096", 640, True)])
def test_decision_tensor_cores(name, S, offsets):
    wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 3, offsets=offsets)
    assert_decision_close(gpu, orc.predict(), wl.N)


def test_full_size_sampled_rows_and_invariants():
    wl, gpu, orc, prec = make_pair("n1024", steps=inputs.WORKLOADS["n1024"].window + 3)
    S = wl.S
    for k0 in (0, S // 2 - 17, S - 48):
        assert_samples_close(gpu.debug_samples(k0, 48), orc.samples(np.arange(k0, k0 + 48)), TOL_X[prec])
    x_all = gpu.debug_samples(0, S).astype(np.float64)
    code, c = gpu.predict()
    e, om = gpu.get_stats()
    s_norm = orc.scale()
    assert code == binding.OK
    want = s_norm * np.sort(x_all, axis=1).mean(axis=0)
    assert np.max(np.abs(e - want) / want[-1]) <= 1e-6
    assert c == int(np.flatnonzero(om == om[np.isfinite(om)].max()).max()) + 1


@pytest.mark.parametrize("N,D,H,lag,S,prec", [(1, 4, 32, 0, 300, 0), (3, 4, 32, 1, 257, 0), (5, 8, 64, 0, 129, 0),
                                               (130, 16, 64, 0, 200, 1), (257, 16, 192, 2, 130, 1), (1025, 32, 96, 1, 140, 2),
                                               (333, 8, 320, 1, 150, 1)])
def test_small_and_ragged_shapes(N, D, H, lag, S, prec):
    w = inputs.make_weights_literal(N, D, H, seed=3, fan_in_ref=32, bf16=(prec == 2))
    trace = inputs.make_trace(N, lag + 4, seed=9, sigma=0.2)
    gpu = binding.Cutoff(N, D, H, lag, S, precision=prec, seed=SEED, flags=binding.FLAG_LITERAL)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, lag, S, seed=SEED)
    for x in trace:
        gpu.push(x)
        orc.push(x)
    assert_samples_close(gpu.debug_samples(0, S), orc.samples(np.arange(S)), TOL_X[prec])
    c = assert_decision_close(gpu, orc.predict(), N)
    assert 1 <= c <= N


def test_variant_of_blob_and_context_must_agree():
    wl = inputs.WORKLOADS["tiny"]
    compact, literal = inputs.workload_weights(wl), inputs.workload_weights_literal(wl)
    for flags, wrong in ((0, literal), (binding.FLAG_LITERAL, compact)):
        gpu = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 64, flags=flags)
        with pytest.raises(binding.CutoffError) as e:
            gpu.load_weights(wrong)
        assert e.value.code == binding.ERR_BAD_BLOB


def test_graph_replay_and_censored_push():
    # the streaming call and the imputation of censored run-times do not depend on the model variant
    wl = inputs.WORKLOADS["n128"]
    S = 512
    w = inputs.workload_weights_literal(wl)
    trace = inputs.workload_trace(wl, wl.window + 8)
    plain = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, seed=SEED, flags=binding.FLAG_LITERAL)
    graph = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, seed=SEED, flags=binding.FLAG_LITERAL | binding.FLAG_GRAPH)
    orc = O.CutoffOracle(w, wl.lag, S, seed=SEED)
    plain.load_weights(w)
    graph.load_weights(w)
    for x in trace:
        orc.push(x)
        code_o, c_o, e_o, om_o = orc.predict()
        rp, rg = plain.step(x), graph.step(x)
        assert rp == rg and rp[0] == code_o
        if code_o == O.OK:
            assert np.array_equal(plain.get_stats()[0], graph.get_stats()[0])
            assert np.max(np.abs(graph.get_stats()[0] - e_o) / e_o[-1]) <= 1e-4
    observed = inputs.workload_trace(wl, wl.window + 9)[-1]
    censored = np.zeros(wl.N, dtype=bool)
    censored[np.argsort(observed)[-5:]] = True
    plain.push(observed, censored)
    orc.push(observed, censored)
    got, want = plain.debug_window()[-1], orc.history[-1]
    assert np.array_equal(got[~censored], want[~censored])
    assert np.max(np.abs(got[censored] - want[censored]) / want[censored]) <= 1e-5
