"""The allocation-free entry point against the ordinary decision path.

Some programs cannot call cudaMalloc when they need order statistics (all device memory already
belongs to their own pool, or nothing may be allocated after start-up).  For them the library
has cutoff_sorted_row_sums_static, whose only scratch is a fixed array inside the library.  This
test feeds it the very samples a decision draws and checks the sums against the ones the
ordinary, allocating path (cutoff_predict + cutoff_get_partial_sums) reports, twice in a row,
so that whatever the first call left in the shared array cannot leak into the second.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  It also passes when run alone in a fresh process.
"""
import numpy as np
import pytest

from paper_1803_04209_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


def _context(name, S):
    wl = inputs.WORKLOADS[name]
    ctx = binding.Cutoff(wl.N, wl.D, wl.H, wl.lag, S, precision=0, seed=99)
    ctx.load_weights(inputs.workload_weights(wl))
    for x in inputs.workload_trace(wl, wl.window + 3):
        ctx.push(x)
    return wl, ctx


def _static_sums(x_host, torch):
    x = torch.from_numpy(np.ascontiguousarray(x_host)).cuda()       # caller-owned input
    sums = torch.full((x.shape[1],), -1.0, dtype=torch.float64, device="cuda")   # caller-owned output
    rc = binding.sorted_row_sums_static(x, sums, stream=torch.cuda.current_stream().cuda_stream)
    assert rc == binding.OK
    torch.cuda.synchronize()
    return sums.cpu().numpy()


def test_static_scratch_entry_point_matches_the_allocating_path_twice():
    import torch
    assert torch.cuda.is_available()
    build.build()
    # first call: 1024 workers, enough rows to use every scratch row
    wl, ctx = _context("n1024", 3000)
    x = ctx.debug_samples(0, 3000)                 # the draws of the coming decision
    got = _static_sums(x, torch)
    assert np.allclose(got, np.sort(x.astype(np.float64), axis=1).sum(axis=0), rtol=1e-6, atol=0)   # the definition
    assert ctx.predict()[0] == binding.OK
    want = ctx.get_partial_sums()
    assert np.allclose(got, want, rtol=1e-6, atol=0)
    # second call right after, on a smaller problem that reuses only part of the scratch
    wl2, ctx2 = _context("n158", 70)
    x2 = ctx2.debug_samples(0, 70)
    got2 = _static_sums(x2, torch)
    assert np.allclose(got2, np.sort(x2.astype(np.float64), axis=1).sum(axis=0), rtol=1e-6, atol=0)
    assert ctx2.predict()[0] == binding.OK
    want2 = ctx2.get_partial_sums()
    assert np.allclose(got2, want2, rtol=1e-6, atol=0)
    # and once more on the first shape, with the next decision's fresh noise
    x3 = ctx.debug_samples(0, 3000)
    assert not np.array_equal(x3, x)
    got3 = _static_sums(x3, torch)
    ctx.predict()
    assert np.allclose(got3, ctx.get_partial_sums(), rtol=1e-6, atol=0)


def test_static_scratch_entry_point_many_rows_go_through_in_blocks():
    # more rows than one pass over the scratch array takes (131072): the sums continue in double across passes,
    # so a long input loses no more digits than a short one
    import torch
    build.build()
    rng = np.random.default_rng(5)
    n, rows = 40, 131072 + 4096 + 3
    x = rng.lognormal(0.0, 0.4, size=(rows, n)).astype(np.float32)
    want = np.sort(x.astype(np.float64), axis=1).sum(axis=0)
    for _ in range(2):
        got = _static_sums(x, torch)
        assert np.allclose(got, want, rtol=2e-6, atol=0)


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    import torch
    build.build()
    lib = binding.load_library()
    x = torch.ones((4, binding.STATIC_MAX_N + 1), dtype=torch.float32, device="cuda")
    sums = torch.zeros(binding.STATIC_MAX_N + 1, dtype=torch.float64, device="cuda")
    with pytest.raises(binding.CutoffError) as e:
        binding.sorted_row_sums_static(x, sums)
    assert e.value.code == binding.ERR_TOO_LARGE
    assert "capacity" in binding.strerror(binding.ERR_TOO_LARGE)
    torch.cuda.synchronize()
    assert float(sums.abs().sum()) == 0.0          # nothing was written
    assert lib.cutoff_sorted_row_sums_static(0, None, 4, 8, 8, sums.data_ptr(), None) == binding.ERR_BAD_ARG
    assert lib.cutoff_sorted_row_sums_static(0, x.data_ptr(), 4, 8, 4, sums.data_ptr(), None) == binding.ERR_BAD_ARG
    assert lib.cutoff_sorted_row_sums_static(0, x.data_ptr(), (1 << 24) + 1, 8, 8, sums.data_ptr(), None) == binding.ERR_BAD_ARG
