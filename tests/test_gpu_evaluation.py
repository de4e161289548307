"""The library's evaluation of cutoff rules on recorded traces against the oracle's (Sections 3, 3.1.1, 4.1).

Throughputs are ratios of an integer and an observed fp32 run-time, formed in double on both sides, so the
hindsight cutoffs must agree exactly and the throughputs to fp32 rounding.  The "order" rule goes through running
sums and a normal quantile, which the two sides round differently in the last bits of a double: its cutoffs must
agree unless two cutoffs tie to within 1e-9.
"""
import numpy as np
import pytest

from oracle import evaluation as E
from paper_1803_04209_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    import torch
    assert torch.cuda.is_available(), "these tests need a GPU"
    build.build()
    return binding.load_library()


def _trace(N, T, seed):
    return inputs.make_trace(N, T, seed=seed, sigma=0.3, groups=min(4, N), stay=0.85, slowdown=2.0,
                             straggler_p=0.03, straggler_scale=1.5)


@pytest.mark.parametrize("N,T", [(1, 5), (2, 9), (16, 40), (33, 17), (158, 64), (1024, 50), (1025, 9), (2175, 12), (4096, 10)])
def test_eval_trace_matches_the_oracle(N, T):
    import torch
    trace = _trace(N, T, seed=N + T)
    trace[T // 2] = trace[T // 2, 0]                                   # one step of equal run-times
    if N >= 4:
        trace[1] = (np.arange(N) + 1) * np.float32(0.125)              # Omega constant: the tie goes to c = N
    rng = np.random.default_rng(N)
    rules = np.stack([np.full(T, N), np.full(T, max(1, N // 2)), rng.integers(1, N + 1, size=T),
                      np.array([E.hindsight_best(row)[0] for row in trace])]).astype(np.int32)
    got = binding.eval_trace(torch.from_numpy(trace).cuda(), torch.from_numpy(rules).cuda())
    want = E.evaluate(trace, {f"r{m}": rules[m] for m in range(rules.shape[0])})
    assert np.array_equal(got["best_c"].cpu().numpy(), want["best_c"])
    assert np.allclose(got["best"].cpu().numpy(), want["best"], rtol=1e-6, atol=0)
    assert np.allclose(got["all"].cpu().numpy(), want["all"], rtol=1e-6, atol=0)
    for m in range(rules.shape[0]):
        assert np.allclose(got["achieved"][m].cpu().numpy(), want[f"r{m}"], rtol=1e-6, atol=0)
        assert np.array_equal(got["step_time"][m].cpu().numpy(), want[f"r{m}_time"].astype(np.float32))
    assert np.array_equal(got["achieved"][3].cpu().numpy(), got["best"].cpu().numpy())   # the hindsight rule attains the maximum
    assert int(got["static_c"].item()) == E.best_static_cutoff(trace)
    # a padded leading dimension and no rules at all
    padded = torch.zeros((T, N + 5), dtype=torch.float32, device="cuda")
    padded[:, :N] = torch.from_numpy(trace).cuda()
    bare = binding.eval_trace(padded[:, :N], None, want_static=False)
    assert np.array_equal(bare["best_c"].cpu().numpy(), want["best_c"])


@pytest.mark.parametrize("N,T", [(1, 4), (24, 30), (158, 100), (1024, 60), (4096, 8)])
def test_order_baseline_matches_the_oracle(N, T):
    import torch
    trace = _trace(N, T, seed=7 * N + T)
    got = binding.order_baseline(torch.from_numpy(trace).cuda()).cpu().numpy()
    want = E.order_cutoffs(trace)
    assert got[0] == N
    x = trace.astype(np.float64)
    for t in np.flatnonzero(got != want):
        seen = x[:t].reshape(-1)
        e = E.elfving_expected(N, float(seen.mean()), float(seen.std()))
        om_got, om_want = got[t] / e[got[t] - 1], want[t] / e[want[t] - 1]
        assert abs(om_got - om_want) <= 1e-9 * abs(om_want), f"step {t}: cutoff {got[t]} != oracle {want[t]}"
    assert np.mean(got == want) >= 0.9


def test_eval_trace_rejects_bad_arguments():
    import torch
    lib = binding.load_library()
    t = torch.ones((3, 8), dtype=torch.float32, device="cuda")
    o = torch.zeros(3, dtype=torch.float32, device="cuda")
    oi = torch.zeros(3, dtype=torch.int32, device="cuda")
    assert lib.cutoff_eval_trace(0, None, 3, 8, 8, None, 0, oi.data_ptr(), o.data_ptr(), o.data_ptr(), None, None, None, None) == binding.ERR_BAD_ARG
    assert lib.cutoff_eval_trace(0, t.data_ptr(), 3, 4097, 4097, None, 0, oi.data_ptr(), o.data_ptr(), o.data_ptr(), None, None, None, None) == binding.ERR_BAD_ARG
    assert lib.cutoff_eval_trace(0, t.data_ptr(), 3, 8, 8, None, 1, oi.data_ptr(), o.data_ptr(), o.data_ptr(), None, None, None, None) == binding.ERR_BAD_ARG
    assert lib.cutoff_order_baseline(0, t.data_ptr(), 0, 8, 8, oi.data_ptr(), None) == binding.ERR_BAD_ARG
