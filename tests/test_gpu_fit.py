"""The library's ELBO, its gradient and its Adam step against the oracle's (Section 3.1.3; Section 4.1).

The library computes in fp32, the oracle in fp64, on the same weights, windows and noise.  Tolerances: the ELBO of
a window is a sum of a few hundred to a few thousand log-density terms, compared to 2e-5 relative to the largest
|ELBO|; a gradient tensor is compared to 2e-4 of its own largest entry (sums over the batch and the window of
fp32 products); an Adam update is compared through the parameters after several steps, to 1e-5 absolute (steps
are of the size of the learning rate).
"""
import numpy as np
import pytest

from oracle import elbo as L
from paper_1803_04209_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    import torch
    assert torch.cuda.is_available(), "these tests need a GPU"
    build.build()
    return binding.load_library()


def _case(N, D, H, lag, B, seed):
    rng = np.random.default_rng(seed)
    w = inputs.make_weights(N, D, H, seed=seed, fan_in_ref=32, offsets=True)
    for k in ("a0", "b0", "z0"):
        w[k] = (rng.standard_normal(w[k].shape) * 0.2).astype(np.float32)
    trace = inputs.make_trace(N, B + lag, seed=seed + 1, sigma=0.25, groups=min(4, N), stay=0.9, slowdown=2.0)
    scale = 2.0 * float(trace[: lag + 1].astype(np.float64).mean())
    x = L.windows_of(trace.astype(np.float64) / scale, lag + 1)[:B].astype(np.float32)
    eps = rng.standard_normal((B, lag + 1, D)).astype(np.float32)
    return w, x, eps


@pytest.mark.parametrize("N,D,H,lag,B", [(5, 3, 4, 2, 2), (16, 4, 32, 1, 7), (128, 8, 128, 2, 64), (158, 8, 64, 20, 5),
                                          (1024, 16, 256, 4, 33), (33, 32, 96, 0, 40)])
def test_elbo_and_gradient_match_the_oracle(N, D, H, lag, B):
    import torch
    w, x, eps = _case(N, D, H, lag, B, seed=N + B)
    want_elbo, want_g = L.elbo_and_grad(w, x, eps)
    fitter = binding.Fitter(N, D, H, lag, B, w)
    elbo, grads = fitter.elbo_grad(torch.from_numpy(x).cuda(), torch.from_numpy(eps).cuda())
    torch.cuda.synchronize()
    got_elbo = elbo.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(got_elbo - want_elbo)) <= 2e-5 * np.max(np.abs(want_elbo))
    got = binding.unflatten_weights(grads.cpu().numpy(), N, D, H)
    for name in L.PARAMS:
        ref = want_g[name]
        denom = max(float(np.max(np.abs(ref))), 1e-6)
        err = float(np.max(np.abs(got[name].astype(np.float64) - ref))) / denom
        assert err <= 2e-4, f"{name}: {err:.2e}"
    # the forward pass alone gives the same ELBO and leaves the gradients alone
    before = grads.clone()
    elbo2, _ = fitter.elbo_grad(torch.from_numpy(x).cuda(), torch.from_numpy(eps).cuda(), want_grad=False)
    torch.cuda.synchronize()
    assert torch.equal(elbo2.cpu(), torch.from_numpy(got_elbo.astype(np.float32)))
    assert torch.equal(before, fitter.grads)
    # and the whole step is reproducible bit for bit
    _, grads3 = fitter.elbo_grad(torch.from_numpy(x).cuda(), torch.from_numpy(eps).cuda())
    torch.cuda.synchronize()
    assert torch.equal(before, grads3)


def test_graph_replay_of_the_step_equals_the_plain_call():
    import torch
    N, D, H, lag, B = 128, 8, 128, 2, 16
    w, x, eps = _case(N, D, H, lag, B, seed=77)
    plain = binding.Fitter(N, D, H, lag, B, w)
    e_ref, g_ref = plain.elbo_grad(torch.from_numpy(x).cuda(), torch.from_numpy(eps).cuda())
    torch.cuda.synchronize()
    e_ref, g_ref = e_ref.clone(), g_ref.clone()
    fitter = binding.Fitter(N, D, H, lag, B, w)
    xs, es = torch.zeros((B, lag + 1, N), device="cuda"), torch.zeros((B, lag + 1, D), device="cuda")
    fitter.capture_elbo_grad(xs, es)                      # captured on other contents
    xs.copy_(torch.from_numpy(x)); es.copy_(torch.from_numpy(eps))
    e1, g1 = fitter.replay_elbo_grad()
    torch.cuda.synchronize()
    assert torch.equal(e1, e_ref) and torch.equal(g1, g_ref)
    # a second replay on new inputs follows them; back on the first inputs it gives the first result again
    xs.mul_(1.01)
    e2, _ = fitter.replay_elbo_grad()
    torch.cuda.synchronize()
    assert not torch.equal(e2, e_ref)
    xs.copy_(torch.from_numpy(x))
    e3, g3 = fitter.replay_elbo_grad()
    torch.cuda.synchronize()
    assert torch.equal(e3, e_ref) and torch.equal(g3, g_ref)


def test_adam_steps_with_clipping_match_the_oracle():
    import torch
    N, D, H, lag, B = 24, 4, 16, 1, 12
    w, x, eps = _case(N, D, H, lag, B, seed=3)
    fitter = binding.Fitter(N, D, H, lag, B, w)
    params = {k: np.asarray(w[k], dtype=np.float64).copy() for k in L.PARAMS}
    opt = L.Adam(lr=3e-3)
    xd, ed = torch.from_numpy(x).cuda(), torch.from_numpy(eps).cuda()
    clipped = 0
    for it in range(6):
        clip = 0.5 if it % 2 == 0 else 1e9                      # steps with and without the clip taking hold
        _, g = L.elbo_and_grad(params, x, eps)
        loss_g = {k: -v / B for k, v in g.items()}
        loss_g, norm = L.clip_by_global_norm(loss_g, clip)
        clipped += norm > clip
        opt.step(params, loss_g)
        fitter.elbo_grad(xd, ed)
        fitter.adam_step(lr=3e-3, clip=clip)
        torch.cuda.synchronize()
        assert abs(float(fitter.norm.item()) - norm) <= 2e-4 * norm
    assert clipped >= 2
    got = fitter.weights()
    for name in L.PARAMS:
        assert np.max(np.abs(got[name].astype(np.float64) - params[name])) <= 1e-5, name
    # the parameters really moved
    assert max(np.max(np.abs(got[k] - w[k])) for k in L.PARAMS) > 5e-3


def test_fitting_on_the_gpu_raises_the_elbo():
    import torch
    N, D, H, lag, B = 12, 4, 16, 1, 32
    trace = inputs.make_trace(N, 160, seed=4, sigma=0.15, groups=2, stay=0.97, slowdown=2.0)
    w0 = inputs.make_weights(N, D, H, seed=1, offsets=False)
    scale = 2.0 * float(trace[: lag + 1].astype(np.float64).mean())
    data = torch.from_numpy(L.windows_of(trace.astype(np.float64) / scale, lag + 1).astype(np.float32)).cuda()
    fitter = binding.Fitter(N, D, H, lag, B, w0)
    gen = torch.Generator(device="cuda").manual_seed(5)
    first = last = None
    for it in range(300):
        idx = torch.randint(0, data.shape[0], (B,), device="cuda", generator=gen)
        eps = torch.randn((B, lag + 1, D), device="cuda", generator=gen)
        elbo, _ = fitter.elbo_grad(data[idx].contiguous(), eps)
        fitter.adam_step(lr=5e-3)
        if it == 0:
            first = float(elbo.mean().item())
        last = float(elbo.mean().item())
    assert last > first + 10.0 * N * (lag + 1) * 0.05
    # the fitted weights are ordinary weights: the oracle's ELBO on them agrees with the library's
    fitted = fitter.weights()
    eps = np.random.default_rng(0).standard_normal((B, lag + 1, D)).astype(np.float32)
    xb = data[:B].cpu().numpy()
    want, _ = L.elbo_and_grad(fitted, xb, eps, want_grad=False)
    got, _ = fitter.elbo_grad(torch.from_numpy(xb).cuda(), torch.from_numpy(eps).cuda(), want_grad=False)
    torch.cuda.synchronize()
    assert np.max(np.abs(got.cpu().numpy() - want)) <= 2e-5 * np.max(np.abs(want))


def test_learning_calls_reject_bad_arguments():
    import torch
    lib = binding.load_library()
    assert lib.cutoff_fit_param_count(0, 4, 8) == 0
    n = lib.cutoff_fit_param_count(16, 4, 32)
    assert n == binding.flatten_weights(inputs.make_weights(16, 4, 32)).size
    buf = torch.zeros(n, dtype=torch.float32, device="cuda")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    args = (0, 16, 4, 32, 1, 4, buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), buf.data_ptr())
    assert lib.cutoff_elbo_grad(*args, ws.data_ptr(), 16, None) == binding.ERR_BAD_ARG          # workspace too small
    assert lib.cutoff_elbo_grad(0, 16, 4, 32, 1, 0, *args[6:], ws.data_ptr(), ws.numel(), None) == binding.ERR_BAD_ARG
    assert lib.cutoff_adam_step(0, n, buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), 0, 1e-3, 0.9, 0.999,
                                1e-8, 1.0, 1.0, buf.data_ptr(), ws.data_ptr(), ws.numel(), None) == binding.ERR_BAD_ARG
