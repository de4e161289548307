"""Parity of the CUDA library with the CPU oracle, through the C ABI, on a real GPU.

Tolerances:
  noise words            bit-exact
  standard normals       2e-6 * max(1, |eps|)
  sampled run-times      rel 1e-5 (fp32 path) or 2e-3 (tf32 / bf16-weight tensor-core path),
                         relative to max(|x|, mean |x|)
  expected order stats   rel 1e-4, relative to max(|E_j|, |E_N|)
  cutoff                 exact, unless the oracle's two best throughputs differ by less than 1e-4 relative
  sort permutation       bit-exact; rows sorted by the decision's own fp32 network bit-exact
"""
import numpy as np
import pytest

from oracle import cutoff_oracle as O
from paper_1803_04209_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu

SEED = 0x5EEDC0FFEE123
TOL_X = {0: 1e-5, 1: 2e-3, 2: 2e-3}
TOL_E = 1e-4


@pytest.fixture(scope="module", autouse=True)
def _lib():
    import torch
    assert torch.cuda.is_available(), "these tests need a GPU"
    build.build()
    return binding.load_library()


def make_pair(name, S=None, steps=None, offsets=True, precision=None, seed=SEED, **kw):
    wl = inputs.WORKLOADS[name]
    S = S or wl.S
    w = inputs.workload_weights(wl, offsets=offsets)
    trace = inputs.workload_trace(wl, steps)
    prec = wl.precision if precision is None else precision
    gpu = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=prec, seed=seed, **kw)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, wl.lag, S, seed=seed)
    for x in trace:
        gpu.push(x)
        orc.push(x)
    return wl, gpu, orc, prec


def assert_samples_close(x_gpu, x_orc, tol):
    floor = np.abs(x_orc).mean()
    err = np.abs(x_gpu.astype(np.float64) - x_orc) / np.maximum(np.abs(x_orc), floor)
    assert np.all(np.isfinite(x_gpu))
    assert err.max() <= tol, f"max relative error {err.max():.3e} > {tol:.1e}"


def assert_decision_close(gpu, orc_result, N):
    code_o, c_o, e_o, om_o = orc_result
    code_g, c_g = gpu.predict()
    e_g, om_g = gpu.get_stats()
    assert code_g == code_o
    denom = np.maximum(np.abs(e_o), np.abs(e_o[-1]))
    assert np.max(np.abs(e_g - e_o) / denom) <= TOL_E
    assert np.all(np.diff(e_g) >= 0)
    finite = np.isfinite(om_o)
    clearly_positive = e_o > TOL_E * np.abs(e_o[-1])
    assert np.array_equal(np.isfinite(om_g)[clearly_positive | (e_o < -TOL_E * np.abs(e_o[-1]))],
                          finite[clearly_positive | (e_o < -TOL_E * np.abs(e_o[-1]))])
    both = finite & np.isfinite(om_g) & clearly_positive
    assert np.max(np.abs(om_g[both] - om_o[both]) / np.abs(om_o[both])) <= 10 * TOL_E
    if c_g != c_o:
        # allowed only when the oracle's two best throughputs are within tolerance of each other
        top = np.sort(om_o[finite])[-2:]
        assert (top[1] - top[0]) <= TOL_E * abs(top[1]), f"cutoff {c_g} != oracle {c_o}"
        assert abs(om_o[c_g - 1] - top[1]) <= TOL_E * abs(top[1])
    return c_g


# ----------------------------------------------------------------------------
def test_noise_generator_bit_exact():
    for (step, stream, k0, count, n) in ((0, 0, 0, 64, 16), (7, 0x200, 4_000_000_000, 33, 1024),
                                          (123456, 0x100, 65500, 100, 7), (1, 3, 5, 1, 1)):
        normals, words = binding.debug_normals(SEED, step, stream, k0, count, n)
        k = np.arange(k0, k0 + count, dtype=np.uint64)
        nq = (n + 3) // 4
        ref_words = np.stack(O.philox4x32_10(np.arange(nq, dtype=np.uint64)[None, :], k[:, None], stream, step,
                                             SEED & 0xFFFFFFFF, SEED >> 32), axis=-1)
        assert np.array_equal(words.astype(np.uint64), ref_words)
        ref = O.normals(SEED, step, stream, k, n)
        assert np.max(np.abs(normals - ref) / np.maximum(1.0, np.abs(ref))) <= 2e-6


def test_noise_generator_known_answer_on_gpu():
    # counter (0, 0, 0, 0), key (0, 0): first published known-answer vector
    _, words = binding.debug_normals(0, 0, 0, 0, 1, 4)
    assert [int(v) for v in words[0, 0]] == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]


@pytest.mark.parametrize("n", [1, 2, 3, 16, 33, 158, 512, 1024, 1025, 2175, 4096])
def test_sort_permutation_bit_exact(n):
    rng = np.random.default_rng(n)
    rows = [rng.integers(0, 50, size=n), rng.integers(-1000, 1000, size=n), np.full(n, 7),
            np.arange(n)[::-1], np.arange(n), rng.integers(0, 3, size=n)]
    rows += [rng.integers(-5, 5, size=n) for _ in range(11)]
    rows = np.stack(rows).astype(np.float32) * np.float32(0.25)
    rows[rows == 0] = 0.0          # no negative zeros
    gpu = binding.Cutoff(16, 4, 32, 1, 64)
    keys, perm = gpu.debug_sort(rows)
    want_perm = np.argsort(rows, axis=1, kind="stable")
    assert np.array_equal(perm, want_perm)
    assert np.array_equal(keys, np.take_along_axis(rows, want_perm, axis=1))


@pytest.mark.parametrize("n", [1, 2, 33, 158, 512, 1024, 1025, 2175, 4096])
def test_float_sort_rows_bit_exact(n):
    # the fp32 instantiation of the network -- the one every decision runs -- row by row against numpy's sort:
    # continuous keys, many equal keys, both zeros, infinities among the keys, already sorted and reversed rows
    rng = np.random.default_rng(1000 + n)
    rows = [rng.standard_normal(n), rng.lognormal(0.0, 0.5, size=n), rng.integers(-3, 4, size=n) * 0.5,
            np.full(n, 1.5), np.sort(rng.standard_normal(n)), np.sort(rng.standard_normal(n))[::-1],
            np.where(rng.random(n) < 0.3, np.inf, rng.standard_normal(n)),
            np.where(rng.random(n) < 0.5, 0.0, -0.0), rng.standard_normal(n) * 1e-30, rng.standard_normal(n) * 1e30]
    rows += [rng.standard_normal(n) for _ in range(23)]
    rows = np.stack(rows).astype(np.float32)
    gpu = binding.Cutoff(16, 4, 32, 1, 64)
    got = gpu.debug_sort_values(rows)
    want = np.sort(rows, axis=1, kind="stable")
    assert np.array_equal(got, want)                                       # value for value (-0 == +0)
    nonzero = want != 0
    assert np.array_equal(got.view(np.uint32)[nonzero], want.view(np.uint32)[nonzero])   # bit for bit
    assert np.array_equal(np.signbit(got).sum(axis=1), np.signbit(rows).sum(axis=1))     # zeros keep their signs
    zeros = (got == 0)
    for r in np.flatnonzero(zeros.any(axis=1)):                            # -0 sorts before +0
        z = np.signbit(got[r][zeros[r]])
        assert np.all(z[:-1] >= z[1:])


@pytest.mark.parametrize("name,S,offsets", [("tiny", 1024, True), ("tiny", 1024, False), ("n128", 2048, True),
                                            ("n128", 777, False), ("n158", 512, True)])
def test_sampled_runtimes_fp32(name, S, offsets):
    wl, gpu, orc, prec = make_pair(name, S=S, offsets=offsets)
    x_gpu = gpu.debug_samples(0, S)
    x_orc = orc.samples(np.arange(S))
    assert_samples_close(x_gpu, x_orc, TOL_X[prec])
    # a window of samples from the middle gives the same rows (draws are addressed by sample index)
    assert np.array_equal(gpu.debug_samples(100, 50), x_gpu[100:150])


@pytest.mark.parametrize("name,S,offsets", [("tiny", 1024, True), ("tiny", 1024, False), ("n128", 4096, True),
                                            ("n128", 1500, False), ("n158", 1024, True)])
def test_decision_fp32(name, S, offsets):
    wl, gpu, orc, prec = make_pair(name, S=S, offsets=offsets)
    assert_decision_close(gpu, orc.predict(), wl.N)


def test_wide_models_fp32_arithmetic():
    # the large shapes with every product in fp32: isolates the non-tensor-core kernels
    for name, S in (("n1024", 1536), ("n2175", 300), ("n4096", 300)):
        wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 7, precision=0)
        assert_samples_close(gpu.debug_samples(0, min(S, 256)), orc.samples(np.arange(min(S, 256))), TOL_X[0])
        assert_decision_close(gpu, orc.predict(), wl.N)


@pytest.mark.parametrize("name,S", [("n1024", 1024), ("n1024", 130), ("n2175", 300), ("n4096", 384), ("stream", 256)])
def test_sampled_runtimes_tensor_cores(name, S):
    # output layer on tcgen05: operands rounded to tf32 (n4096: weights already bf16-representable)
    wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 7)
    assert prec in (1, 2)
    x_gpu = gpu.debug_samples(0, S)
    x_orc = orc.samples(np.arange(S))
    assert_samples_close(x_gpu, x_orc, TOL_X[prec])
    assert np.array_equal(gpu.debug_samples(S // 2, 7), x_gpu[S // 2: S // 2 + 7])


@pytest.mark.parametrize("name,S,offsets", [("n1024", 4096, True), ("n1024", 1000, False), ("n2175", 512, True),
                                            ("n4096", 1024, True)])
def test_decision_tensor_cores(name, S, offsets):
    wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 7, offsets=offsets)
    assert_decision_close(gpu, orc.predict(), wl.N)


@pytest.mark.parametrize("name", ["n1024", "n4096"])
def test_full_size_sampled_rows_and_invariants(name):
    # the workload at its full size, in the launch configuration bench.py times
    wl, gpu, orc, prec = make_pair(name, steps=inputs.WORKLOADS[name].window + 7)
    S = wl.S
    for k0 in (0, S // 2 - 17, S - 48):                    # rows the oracle computes one by one
        x_gpu = gpu.debug_samples(k0, 48)
        x_orc = orc.samples(np.arange(k0, k0 + 48))
        assert_samples_close(x_gpu, x_orc, TOL_X[prec])
    x_all = gpu.debug_samples(0, S).astype(np.float64)     # properties that hold at any size
    code, c = gpu.predict()
    e, om = gpu.get_stats()
    sums = gpu.get_partial_sums()
    s_norm = orc.scale()
    assert code == binding.OK
    assert np.all(np.diff(e) >= 0)                                                    # order statistics ascend
    assert abs(sums.sum() - x_all.sum()) <= 1e-6 * np.abs(x_all).sum()                # sorting permutes each row
    assert x_all.min() * s_norm <= e[0] * (1 + 1e-6) and e[-1] <= x_all.max() * s_norm * (1 + 1e-6)
    want = s_norm * np.sort(x_all, axis=1).mean(axis=0)                               # numpy sort of the GPU's own draws
    assert np.max(np.abs(e - want) / want[-1]) <= 1e-6
    finite = np.isfinite(om)
    assert c == int(np.flatnonzero(om == om[finite].max()).max()) + 1                 # largest c attaining the maximum


def test_full_size_decision_against_the_full_oracle():
    wl, gpu, orc, prec = make_pair("n1024", steps=inputs.WORKLOADS["n1024"].window + 7)
    assert_decision_close(gpu, orc.predict(), wl.N)


def test_full_size_decision_n4096_against_the_full_oracle():
    # N = 4096, S = 32768, bf16-representable weights: the whole decision, every sample, against the oracle
    wl, gpu, orc, prec = make_pair("n4096", steps=inputs.WORKLOADS["n4096"].window + 7)
    assert gpu.S == 32768
    assert_decision_close(gpu, orc.predict(), wl.N)


def test_streaming_loop_matches_oracle():
    wl = inputs.WORKLOADS["tiny"]
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, 14)
    gpu = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 512, seed=SEED)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, wl.lag, 512, seed=SEED)
    for t, x in enumerate(trace):
        code_o, c_o, e_o, _ = orc.predict()
        code_g, c_g = gpu.predict()
        assert code_g == code_o
        if code_o == O.WARMUP:
            assert c_g == wl.N == c_o
        else:
            e_g, _ = gpu.get_stats()
            assert np.max(np.abs(e_g - e_o) / e_o[-1]) <= TOL_E
            assert c_g == c_o
        gpu.push(x)
        orc.push(x)


def test_graph_replay_equals_plain_calls_and_oracle():
    # the streaming loop: step() = push + predict; with the graph flag the same kernels are replayed
    wl = inputs.WORKLOADS["stream"]
    S = 512
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, wl.window + 12)
    plain = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=wl.precision, seed=SEED)
    graph = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=wl.precision, seed=SEED, flags=binding.FLAG_GRAPH)
    orc = O.CutoffOracle(w, wl.lag, S, seed=SEED)
    plain.load_weights(w)
    graph.load_weights(w)
    launches = []
    for t, x in enumerate(trace):
        orc.push(x)
        code_o, c_o, e_o, om_o = orc.predict()
        rp = plain.step(x)
        rg = graph.step(x)
        assert rp == rg and rp[0] == code_o
        launches.append(graph.launch_count())
        if code_o == O.OK:
            e_p, e_g = plain.get_stats()[0], graph.get_stats()[0]
            assert np.array_equal(e_p, e_g)                     # same kernels, same bits
            assert np.max(np.abs(e_g - e_o) / e_o[-1]) <= TOL_E
            top = np.sort(om_o[np.isfinite(om_o)])[-2:]
            assert rg[1] == c_o or (top[1] - top[0]) <= TOL_E * top[1]
    assert launches[-1] - launches[-2] == launches[-2] - launches[-3] > 0    # replays are counted
    with pytest.raises(binding.CutoffError) as e:
        graph.step(np.zeros(wl.N, dtype=np.float32))
    assert e.value.code == binding.ERR_BAD_VALUE


def test_device_pushes_equal_host_pushes():
    import torch
    wl = inputs.WORKLOADS["n128"]
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, 9)
    a = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 256, seed=3)
    b = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 256, seed=3)
    a.load_weights(w)
    b.load_weights(w)
    dev = torch.from_numpy(trace).cuda()
    torch.cuda.synchronize()
    for t in range(trace.shape[0]):
        a.push(trace[t])
        if t % 2:
            b.push(dev[t])
        else:
            b.push_async(dev[t])
    assert a.predict() == b.predict()
    assert np.array_equal(a.get_stats()[0], b.get_stats()[0])


def test_pass_size_does_not_change_the_result():
    wl, gpu, orc, _ = make_pair("n128", S=5000, steps=8)
    ref = gpu.predict()
    e_ref, _ = gpu.get_stats()
    wl, gpu2, _, _ = make_pair("n128", S=5000, steps=8)
    gpu2.set_option("pass_rows", 1024)
    assert gpu2.predict() == ref
    e2, _ = gpu2.get_stats()
    assert np.max(np.abs(e2 - e_ref) / e_ref[-1]) <= 1e-6


def test_sample_sharding_adds_up():
    # two contexts that each draw half of the samples of one decision
    wl = inputs.WORKLOADS["n128"]
    S = 2048
    _, whole, orc, _ = make_pair("n128", S=S, steps=8)
    _, lo, _, _ = make_pair("n128", S=S // 2, steps=8, sample_offset=0, total_samples=S)
    _, hi, _, _ = make_pair("n128", S=S // 2, steps=8, sample_offset=S // 2, total_samples=S)
    assert np.array_equal(hi.debug_samples(0, 8), whole.debug_samples(S // 2, 8))   # global sample index
    code, c = whole.predict()
    lo.predict()
    hi.predict()
    total = lo.get_partial_sums() + hi.get_partial_sums()
    assert np.allclose(total, whole.get_partial_sums(), rtol=1e-6)
    code2, c2 = lo.decide_from_sums(total)
    assert (code2, c2) == (code, c)
    assert np.max(np.abs(lo.get_stats()[0] - whole.get_stats()[0]) / whole.get_stats()[0][-1]) <= 1e-6


def test_state_save_restore_and_reset():
    wl, gpu, orc, _ = make_pair("tiny", S=256, steps=7)
    blob = gpu.save_state()
    first = gpu.predict()
    e_first, _ = gpu.get_stats()
    gpu.push(inputs.workload_trace(wl, 8)[7])
    gpu.restore_state(blob)
    assert gpu.predict() == first
    assert np.array_equal(gpu.get_stats()[0], e_first)
    gpu.reset()
    assert gpu.predict() == (binding.WARMUP, wl.N)


def test_errors_are_codes_not_crashes():
    wl = inputs.WORKLOADS["tiny"]
    w = inputs.workload_weights(wl)
    gpu = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 128)
    with pytest.raises(binding.CutoffError) as e:
        gpu.predict()                                   # no weights yet
    assert e.value.code == binding.ERR_STATE
    blob = binding.pack_weights(w, wl.N, wl.D, wl.H)
    for bad in (blob[:-4], b"\0" * len(blob), blob[:8] + b"\x11\0\0\0" + blob[12:]):
        with pytest.raises(binding.CutoffError) as e:
            gpu.load_weights(bad)
        assert e.value.code == binding.ERR_BAD_BLOB
    nan_blob = bytearray(blob)
    nan_blob[24:28] = np.float32(np.nan).tobytes()
    with pytest.raises(binding.CutoffError) as e:
        gpu.load_weights(bytes(nan_blob))
    assert e.value.code == binding.ERR_BAD_BLOB
    gpu.load_weights(w)
    assert gpu.predict() == (binding.WARMUP, wl.N)
    good = np.ones(wl.N, dtype=np.float32)
    for bad_value in (0.0, -1.0, np.nan, np.inf):
        x = good.copy()
        x[5] = bad_value
        with pytest.raises(binding.CutoffError) as e:
            gpu.push(x)
        assert e.value.code == binding.ERR_BAD_VALUE
        import torch
        with pytest.raises(binding.CutoffError) as e:
            gpu.push(torch.from_numpy(x).cuda())
        assert e.value.code == binding.ERR_BAD_VALUE
    # rejected pushes leave no trace: two good pushes complete the window
    gpu.push(good)
    assert gpu.predict() == (binding.WARMUP, wl.N)
    gpu.push(good)
    assert gpu.predict()[0] == binding.OK
    with pytest.raises(binding.CutoffError) as e:
        gpu.fetch()                                     # nothing enqueued
    assert e.value.code == binding.ERR_STATE


def _censor_beyond_cutoff(observed, c):
    order = np.argsort(observed, kind="stable")
    censored = np.zeros(observed.shape[0], dtype=bool)
    censored[order[min(c, observed.shape[0] - 3):]] = True          # at least the three slowest are killed
    return censored


@pytest.mark.parametrize("name,S", [("n128", 2048), ("n1024", 1024)])
def test_censored_push_imputes_from_the_truncated_predictive(name, S):
    import torch
    wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 5)
    tol = TOL_X[prec]
    observed = inputs.workload_trace(wl, wl.window + 6)[-1]
    with pytest.raises(binding.CutoffError) as e:                   # no decision yet: nothing to draw from
        gpu.push(observed, np.ones(wl.N, dtype=bool))
    assert e.value.code == binding.ERR_STATE
    x_gpu = gpu.debug_samples(0, S).astype(np.float64) * orc.scale()   # the draws the decision is about to make
    code_o, c_o, _, _ = orc.predict()
    code_g, c_g = gpu.predict()
    assert code_g == code_o == binding.OK
    censored = _censor_beyond_cutoff(observed, c_o)
    with pytest.raises(binding.CutoffError) as e:                   # nobody finished
        gpu.push(observed, np.ones(wl.N, dtype=bool))
    assert e.value.code == binding.ERR_BAD_ARG
    junk = observed.copy()
    junk[censored] = np.nan                                         # censored entries are ignored
    gpu.push(junk, censored)
    orc.push(observed, censored)
    got = gpu.debug_window()[-1].astype(np.float64)
    want = orc.history[-1].astype(np.float64)
    threshold = float(observed[~censored].max())
    assert np.array_equal(got[~censored], observed[~censored].astype(np.float64))
    assert np.all(got[censored] >= threshold)
    # every replacement is the first of the worker's own draws above the threshold, in the oracle's scan order
    draws = orc.last_draws_sec
    checked = 0
    for j in np.flatnonzero(censored):
        start = int(O.philox4x32_10(int(j), 0, O.STREAM_IMPUTE, orc.step, SEED & 0xFFFFFFFF, SEED >> 32)[0]) % S
        col = np.roll(draws[:, j], -start)
        hits = np.flatnonzero(col > threshold)
        upto = col[: hits[0] + 1] if hits.size else col
        if np.any(np.abs(upto - threshold) <= 2 * tol * threshold):
            continue                                                # a draw too close to the threshold to call
        checked += 1
        assert abs(got[j] - want[j]) <= tol * max(abs(want[j]), threshold)
        k_star = (start + hits[0]) % S if hits.size else None
        if k_star is not None:
            assert abs(got[j] - x_gpu[k_star, j]) <= 1e-6 * abs(got[j])     # it is the GPU's own draw
    assert checked >= 0.8 * censored.sum()
    # the imputed window feeds the next decision
    assert_decision_close(gpu, orc.predict(), wl.N)
    # device pointers take the same path
    _, gpu2, _, _ = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 5)
    gpu2.predict()
    gpu2.push(torch.from_numpy(np.where(censored, 1.0, observed).astype(np.float32)).cuda(),
              torch.from_numpy(censored.astype(np.uint8)).cuda())
    assert np.array_equal(gpu2.debug_window()[-1], got.astype(np.float32))
    # a push without censored workers is an ordinary push; a second censored push needs a new decision
    gpu2.predict()
    assert gpu2.push(observed, np.zeros(wl.N, dtype=bool)) == binding.OK
    with pytest.raises(binding.CutoffError) as e:
        gpu2.push(observed, censored)
    assert e.value.code == binding.ERR_STATE


@pytest.mark.parametrize("name,S", [("tiny", 1024), ("n158", 1024), ("n1024", 2048), ("n2175", 300)])
def test_order_statistic_spread(name, S):
    # the +-2 sigma bands of the paper's Fig. 3: standard deviation of each order statistic over the samples
    wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 5)
    with pytest.raises(binding.CutoffError) as e:
        gpu.predict()
        gpu.get_order_stat_std()                            # not asked for
    assert e.value.code == binding.ERR_STATE
    plain = gpu.get_stats()[0]
    orc.predict()
    gpu.restore_state(_state_before(gpu, wl, name))         # same decision again, now with the squares
    gpu.set_option("order_stat_std", 1)
    code, c = gpu.predict()
    sd = gpu.get_order_stat_std()
    assert np.array_equal(gpu.get_stats()[0], plain)        # the means do not change
    want = orc.last_std_sec
    assert np.max(np.abs(sd - want)) <= 2e-3 * want.max()
    assert np.all(sd >= 0)


def _state_before(gpu, wl, name):
    """Observation state of a fresh context that saw the same pushes and has made no decision."""
    fresh = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 64, precision=0)
    for x in inputs.workload_trace(wl, wl.window + 5):
        fresh.push(x)
    return fresh.save_state()


@pytest.mark.parametrize("N,D,H,lag,S,prec", [(1, 4, 32, 0, 300, 0), (3, 4, 32, 1, 257, 0), (5, 8, 64, 0, 129, 0),
                                               (130, 16, 64, 0, 200, 1), (257, 16, 192, 2, 130, 1), (1025, 32, 96, 1, 140, 2)])
def test_small_and_ragged_shapes(N, D, H, lag, S, prec):
    # one worker, odd worker counts, a window of one vector, sample counts that leave ragged tiles
    w = inputs.make_weights(N, D, H, seed=3, fan_in_ref=32, bf16=(prec == 2))
    trace = inputs.make_trace(N, lag + 4, seed=9, sigma=0.2)
    gpu = binding.Cutoff(N, D, H, lag, S, precision=prec, seed=SEED)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, lag, S, seed=SEED)
    for x in trace:
        gpu.push(x)
        orc.push(x)
    assert_samples_close(gpu.debug_samples(0, S), orc.samples(np.arange(S)), TOL_X[prec])
    c = assert_decision_close(gpu, orc.predict(), N)
    assert 1 <= c <= N


def test_degenerate_and_equal_times():
    # every expected time negative -> c = N with the informational code; equal deterministic times -> c = N
    wl = inputs.WORKLOADS["tiny"]
    w = inputs.workload_weights(wl)
    w["W4"][:] = 0.0
    w["b4"][: wl.N] = -1.0
    gpu = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 128)
    gpu.load_weights(w)
    for x in inputs.workload_trace(wl, 3):
        gpu.push(x)
    assert gpu.predict() == (binding.DEGENERATE, wl.N)
    e, om = gpu.get_stats()
    assert np.all(e < 0) and np.all(np.isneginf(om))
    w["b4"][: wl.N] = 0.75
    w["b4"][wl.N:] = -150.0
    gpu.load_weights(w)
    assert gpu.predict() == (binding.OK, wl.N)
    e, om = gpu.get_stats()
    s = 2.0 * inputs.workload_trace(wl, 3)[:2].astype(np.float64).mean()
    assert np.allclose(e, 0.75 * s, rtol=1e-6)


@pytest.mark.parametrize("N,D,H,lag,S,prec", [(32, 4, 1024, 1, 200, 0), (8, 4, 32, 255, 64, 0), (4096, 4, 16, 0, 40, 0),
                                               (96, 32, 512, 3, 150, 1), (64, 8, 1024, 0, 130, 2)])
def test_limits_of_the_supported_shapes(N, D, H, lag, S, prec):
    # the widest hidden layer, the longest window, the most workers, the widest tensor-core chain
    w = inputs.make_weights(N, D, H, seed=5, fan_in_ref=32, bf16=(prec == 2))
    trace = inputs.make_trace(N, lag + 3, seed=11, sigma=0.2)
    gpu = binding.Cutoff(N, D, H, lag, S, precision=prec, seed=SEED)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, lag, S, seed=SEED)
    for x in trace:
        gpu.push(x)
        orc.push(x)
    assert_samples_close(gpu.debug_samples(0, S), orc.samples(np.arange(S)), TOL_X[prec])
    assert_decision_close(gpu, orc.predict(), N)


@pytest.mark.parametrize("H,lag", [(256, 4), (288, 3), (320, 2), (384, 5), (512, 0), (576, 1), (640, 2)])
def test_encoder_widths_on_the_cluster_kernel(H, lag):
    # hidden widths from 256 up whose recurrence runs on the cluster of 8 CTAs per direction (rows split 8 ways,
    # state exchanged through distributed shared memory), widths that are not powers of two included
    N, D, S = 40, 8, 96
    w = inputs.make_weights(N, D, H, seed=H, fan_in_ref=32)
    trace = inputs.make_trace(N, lag + 4, seed=H + 1, sigma=0.2)
    gpu = binding.Cutoff(N, D, H, lag, S, precision=0, seed=SEED)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, lag, S, seed=SEED)
    for x in trace:
        gpu.push(x)
        orc.push(x)
    assert_samples_close(gpu.debug_samples(0, S), orc.samples(np.arange(S)), TOL_X[0])
    assert_decision_close(gpu, orc.predict(), N)


@pytest.mark.parametrize("kw", [dict(n_workers=4097), dict(latent_dim=5), dict(latent_dim=64), dict(hidden=1028),
                                dict(hidden=30), dict(lag=256), dict(latent_dim=32, hidden=1024)])
def test_unsupported_shapes_are_refused(kw):
    args = dict(n_workers=64, latent_dim=8, hidden=64, lag=1, n_samples=64)
    args.update(kw)
    with pytest.raises(binding.CutoffError) as e:
        binding.Cutoff(**args)
    assert e.value.code in (binding.ERR_UNSUPPORTED, binding.ERR_BAD_ARG)


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    for _ in range(n):
        D = int(rng.choice([4, 8, 16, 32]))
        H = D * int(rng.integers(1, 256 // D + 1)) if rng.random() < 0.7 else 64 * int(rng.integers(1, 5))
        H = max(H, 8) // D * D or D
        N = int(rng.choice([rng.integers(1, 40), rng.integers(40, 600), rng.integers(600, 2300)]))
        lag = int(rng.integers(0, 6))
        S = int(rng.integers(1, 700))
        prec = int(rng.integers(0, 3))
        literal = bool(rng.random() < 0.5)
        shapes.append((N, D, H, lag, S, prec, literal))
    return shapes


@pytest.mark.parametrize("N,D,H,lag,S,prec,literal", _random_shapes(16, seed=20260101))
def test_random_shapes_both_variants(N, D, H, lag, S, prec, literal):
    # shapes nobody picked by hand: every kernel selection rule (tensor-core chain or not, resident encoder or not,
    # sort width, ragged tiles) gets exercised in combinations
    make = inputs.make_weights_literal if literal else inputs.make_weights
    w = make(N, D, H, seed=N + H, fan_in_ref=32, bf16=(prec == 2))
    trace = inputs.make_trace(N, lag + 3, seed=S, sigma=0.25)
    gpu = binding.Cutoff(N, D, H, lag, S, precision=prec, seed=SEED + N, flags=binding.FLAG_LITERAL if literal else 0)
    gpu.load_weights(w)
    orc = O.CutoffOracle(w, lag, S, seed=SEED + N)
    for x in trace:
        gpu.push(x)
        orc.push(x)
    assert_samples_close(gpu.debug_samples(0, S), orc.samples(np.arange(S)), TOL_X[prec])
    assert_decision_close(gpu, orc.predict(), N)


@pytest.mark.parametrize("seed,literal,graph,H", [(1, False, False, 64), (2, True, False, 64), (3, False, True, 64),
                                                  (4, True, True, 64), (5, False, True, 320), (6, False, False, 512)])
def test_random_call_sequences(seed, literal, graph, H):
    # pushes from host and device, decisions, save / restore, reset and reloaded weights in random order: the
    # library's cached state (window, normaliser, per-slot projections, captured graph) must follow the oracle's
    import copy
    import torch
    rng = np.random.default_rng(seed)
    N, D, lag, S = 96, 8, 2, 192        # H = 320 and 512: the cluster recurrence of the encoder, also inside the graph
    make = inputs.make_weights_literal if literal else inputs.make_weights
    weights = [make(N, D, H, seed=s, fan_in_ref=32) for s in (11, 12)]
    trace = inputs.make_trace(N, 80, seed=seed, sigma=0.25)
    flags = (binding.FLAG_LITERAL if literal else 0) | (binding.FLAG_GRAPH if graph else 0)
    gpu = binding.Cutoff(N, D, H, lag, S, seed=SEED, flags=flags)
    gpu.load_weights(weights[0])
    orc = O.CutoffOracle(weights[0], lag, S, seed=SEED)
    saved = None
    t = 0
    decisions = 0
    for _ in range(60):
        op = rng.choice(["push", "push_dev", "predict", "step", "save", "restore", "reset", "weights"],
                        p=[0.25, 0.1, 0.25, 0.15, 0.07, 0.07, 0.04, 0.07])
        if op == "push":
            gpu.push(trace[t]); orc.push(trace[t]); t += 1
        elif op == "push_dev":
            gpu.push(torch.from_numpy(trace[t]).cuda()); orc.push(trace[t]); t += 1
        elif op in ("predict", "step"):
            if op == "step":
                res_g = gpu.step(trace[t]); orc.push(trace[t]); t += 1
            else:
                res_g = gpu.predict()
            code_o, c_o, e_o, om_o = orc.predict()
            assert res_g[0] == code_o
            if code_o == O.WARMUP:
                assert res_g[1] == N
                continue
            decisions += 1
            e_g, _ = gpu.get_stats()
            assert np.max(np.abs(e_g - e_o) / np.abs(e_o[-1])) <= TOL_E
            top = np.sort(om_o[np.isfinite(om_o)])[-2:]
            assert res_g[1] == c_o or (top[1] - top[0]) <= TOL_E * abs(top[1])
        elif op == "save":
            saved = (gpu.save_state(), copy.deepcopy(orc.history), orc.step)
        elif op == "restore" and saved is not None:
            gpu.restore_state(saved[0]); orc.history = copy.deepcopy(saved[1]); orc.step = saved[2]
        elif op == "reset":
            gpu.reset(); orc.reset()
        elif op == "weights":
            w = weights[int(rng.integers(0, 2))]
            gpu.load_weights(w); orc.w = w
    assert decisions >= 5


def test_step_device_equals_step_and_rejects_bad_values():
    # run-times that already sit on the GPU: same decisions as the host call, with and without the graph
    import torch
    wl = inputs.WORKLOADS["stream"]
    S = 384
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, wl.window + 10)
    dev = torch.from_numpy(trace).cuda()
    host_ctx = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=wl.precision, seed=SEED, flags=binding.FLAG_GRAPH)
    dev_ctx = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=wl.precision, seed=SEED, flags=binding.FLAG_GRAPH)
    plain_ctx = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=wl.precision, seed=SEED)
    for ctx in (host_ctx, dev_ctx, plain_ctx):
        ctx.load_weights(w)
    for t in range(trace.shape[0]):
        a, b, c = host_ctx.step(trace[t]), dev_ctx.step_device(dev[t]), plain_ctx.step_device(dev[t])
        assert a == b == c
        if a[0] == binding.OK:
            assert np.array_equal(host_ctx.get_stats()[0], dev_ctx.get_stats()[0])
            assert np.array_equal(host_ctx.get_stats()[0], plain_ctx.get_stats()[0])
    # a bad value inside a replay: reported, and nothing has moved (window, decision counter)
    bad = dev[3].clone()
    bad[17] = -1.0
    for ctx in (dev_ctx, plain_ctx):
        with pytest.raises(binding.CutoffError) as e:
            ctx.step_device(bad)
        assert e.value.code == binding.ERR_BAD_VALUE
    nxt = trace[5]
    a, b, c = host_ctx.step(nxt), dev_ctx.step_device(torch.from_numpy(nxt).cuda()), plain_ctx.step_device(torch.from_numpy(nxt).cuda())
    assert a == b == c
    assert np.array_equal(host_ctx.get_stats()[0], dev_ctx.get_stats()[0])


def test_censored_push_refuses_a_mask_without_finishers_and_stale_draws():
    import torch
    wl, gpu, orc, prec = make_pair("n128", S=512, steps=inputs.WORKLOADS["n128"].window + 5)
    observed = inputs.workload_trace(wl, wl.window + 6)[-1]
    assert gpu.predict()[0] == binding.OK
    before = gpu.debug_window()
    # device mask of all ones: nobody finished, so there is no cutoff time to truncate at
    with pytest.raises(binding.CutoffError) as e:
        gpu.push(torch.from_numpy(observed).cuda(), torch.ones(wl.N, dtype=torch.uint8, device="cuda"))
    assert e.value.code == binding.ERR_BAD_VALUE
    assert np.array_equal(gpu.debug_window(), before)               # the window did not move
    # the refused push used up this decision's draws: decide again, then save / restore
    assert gpu.predict()[0] == binding.OK
    blob = gpu.save_state()
    gpu.restore_state(blob)
    censored = np.zeros(wl.N, dtype=bool)
    censored[:5] = True
    with pytest.raises(binding.CutoffError) as e:                   # draws of a decision on the replaced state
        gpu.push(observed, censored)
    assert e.value.code == binding.ERR_STATE
    assert gpu.predict()[0] == binding.OK
    assert gpu.push(observed, censored) == binding.OK


def test_pass_rows_cannot_change_under_a_captured_graph():
    wl = inputs.WORKLOADS["n128"]
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, wl.window + 6)
    gpu = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, 4096, seed=SEED, flags=binding.FLAG_GRAPH)
    gpu.load_weights(w)
    gpu.set_option("pass_rows", 2048)                               # before the capture: fine
    for x in trace:
        gpu.step(x)                                                 # the later steps replay the captured graph
    with pytest.raises(binding.CutoffError) as e:
        gpu.set_option("pass_rows", 4096)
    assert e.value.code == binding.ERR_STATE
    with pytest.raises(binding.CutoffError) as e:
        gpu.set_option("pass_rows", 1 << 40)
    assert e.value.code == binding.ERR_BAD_ARG
    censored = np.zeros(wl.N, dtype=bool)
    censored[-4:] = True
    with pytest.raises(binding.CutoffError) as e:                   # two passes: the draws of pass one are gone
        gpu.push(trace[-1], censored)
    assert e.value.code == binding.ERR_STATE


def test_partial_decisions_add_up_on_the_device():
    # two contexts draw half of the samples each; their sums are added in the library's own device array and the
    # decision is finished from there: same result as one context with all samples, nothing through the host
    import torch
    S = 2048
    _, whole, orc, _ = make_pair("n128", S=S, steps=8)
    _, lo, _, _ = make_pair("n128", S=S // 2, steps=8, sample_offset=0, total_samples=S)
    _, hi, _, _ = make_pair("n128", S=S // 2, steps=8, sample_offset=S // 2, total_samples=S)
    code, c = whole.predict()
    assert lo.predict_partial_async() == binding.OK
    assert hi.predict_partial_async() == binding.OK
    with pytest.raises(binding.CutoffError) as e:
        lo.predict()                                                # a partial decision is open
    assert e.value.code == binding.ERR_STATE
    t_lo, t_hi = lo.partial_sums_tensor(), hi.partial_sums_tensor()
    torch.cuda.synchronize()
    total = t_lo + t_hi
    assert np.allclose(total.cpu().numpy(), whole.get_partial_sums(), rtol=1e-6)
    t_lo.copy_(total)                                               # what an in-place all-reduce leaves behind
    torch.cuda.synchronize()
    assert lo.decide_from_device_sums(t_lo) == (code, c)
    assert hi.decide_from_device_sums(total) == (code, c)
    assert np.max(np.abs(lo.get_stats()[0] - whole.get_stats()[0]) / whole.get_stats()[0][-1]) <= 1e-6
    # both contexts advanced their decision counter exactly once: the next shared decision matches the next whole one
    code2, c2 = whole.predict()
    lo.predict_partial_async(); hi.predict_partial_async()
    torch.cuda.synchronize()
    total = lo.partial_sums_tensor() + hi.partial_sums_tensor()
    assert np.allclose(total.cpu().numpy(), whole.get_partial_sums(), rtol=1e-6)
    assert lo.decide_from_device_sums(total) == (code2, c2)
    assert hi.decide_from_device_sums(total) == (code2, c2)
    fresh = binding.Cutoff(128, 8, 128, 2, 64)
    fresh.load_weights(inputs.workload_weights(inputs.WORKLOADS["n128"]))
    assert fresh.predict_partial_async() == binding.WARMUP


def test_measured_pipe_rates_are_plausible():
    r = binding.measure_pipe_rates(0)
    assert 1.0 <= r["minmax"] <= 2.1          # 64 lanes per SM per clock = 2 warp-instructions
    assert 0.5 <= r["shuffle"] <= 1.1         # 32 lanes per SM per clock
    assert 2.0 <= r["fma"] <= 4.1             # 128 lanes per SM per clock


def test_measured_operand_stream_is_plausible():
    # all SMs together, L2 -> shared memory: above what HBM alone could feed, below 64 bytes per clock per SM x 2
    r = binding.measure_operand_stream(0)
    assert 4000.0 <= r["hidden_64mb"] <= 40000.0
    assert 4000.0 <= r["weights_2mb"] <= 40000.0
    assert r["weights_2mb"] >= 0.8 * r["hidden_64mb"]
    # a second call gives about the same figures (the first repetition of each is a warm-up)
    r2 = binding.measure_operand_stream(0)
    assert abs(r2["hidden_64mb"] - r["hidden_64mb"]) <= 0.2 * r["hidden_64mb"]


@pytest.mark.parametrize("name,S", [("n1024", 700), ("n2175", 300), ("n4096", 384)])
def test_two_sm_emission_option_gives_the_same_draws(name, S):
    # the output layer with tensor-core instructions that span two SMs (each SM loads half of every weight tile)
    wl, gpu, orc, prec = make_pair(name, S=S, steps=inputs.WORKLOADS[name].window + 7)
    ref = gpu.debug_samples(0, S)
    gpu.set_option("pair_emission", 1)
    got = gpu.debug_samples(0, S)
    assert np.allclose(got, ref, rtol=1e-6, atol=1e-7)
    assert_samples_close(got, orc.samples(np.arange(S)), TOL_X[prec])
    assert_decision_close(gpu, orc.predict(), wl.N)
    fp32 = binding.Cutoff(16, 4, 32, 1, 64)
    with pytest.raises(binding.CutoffError) as e:
        fp32.set_option("pair_emission", 1)
    assert e.value.code == binding.ERR_UNSUPPORTED


def test_sharded_decision_all_reduces_the_librarys_own_array_under_nccl():
    # one rank, NCCL: the path bench.py takes with several GPUs -- the partial sums stay in the library's device
    # array, NCCL reduces them in place on the context's stream, the decision is finished from there
    import socket
    import torch
    import torch.distributed as dist
    from paper_1803_04209_b200 import sharding
    wl = inputs.WORKLOADS["n128"]
    S = 1024
    stream = torch.cuda.current_stream()
    w = inputs.workload_weights(wl)
    trace = inputs.workload_trace(wl, 8)
    cfg = sharding.shard_config(0, 1, S)
    ctx = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, cfg["n_samples"], precision=wl.precision, seed=SEED,
                         stream=stream.cuda_stream, sample_offset=cfg["sample_offset"], total_samples=cfg["total_samples"])
    ref = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=wl.precision, seed=SEED)
    for c in (ctx, ref):
        c.load_weights(w)
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    try:
        shared = sharding.ShardedDecision(ctx, device="cuda")
        assert shared.predict() == (binding.WARMUP, wl.N)
        for x in trace:
            ctx.push(x)
            ref.push(x)
        for _ in range(3):
            assert shared.predict() == ref.predict()
            assert np.array_equal(ctx.get_stats()[0], ref.get_stats()[0])
    finally:
        dist.destroy_process_group()
