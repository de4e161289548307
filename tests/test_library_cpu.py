"""Host-side checks that need no GPU: the shared library loads and exports the declared C ABI."""
import os
import re
import struct

import numpy as np
import pytest

from paper_1803_04209_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "cutoff.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cutoff_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    declared = _declared_functions()
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib, name), f"libcutoff.so does not export {name}"
    assert sorted(binding.EXPORTS) == declared


def test_strerror_needs_no_gpu(lib):
    assert "finite" in binding.strerror(binding.ERR_BAD_VALUE)
    assert binding.strerror(binding.OK) == "ok"
    assert binding.strerror(12345) == "unknown code"


def test_null_arguments_are_rejected_without_touching_a_device(lib):
    assert lib.cutoff_create(None, None) == binding.ERR_BAD_ARG
    assert lib.cutoff_predict(None, None) == binding.ERR_BAD_ARG
    assert lib.cutoff_push(None, None, 0, None) == binding.ERR_BAD_ARG
    assert lib.cutoff_launch_count(None) == 0
    lib.cutoff_destroy(None)


def test_config_validation_happens_before_any_cuda_call(lib):
    import ctypes as C
    h = C.c_void_p()
    for kw in (dict(n_workers=0), dict(n_samples=0), dict(lag=-1), dict(precision=7), dict(device=-1)):
        base = dict(n_workers=16, latent_dim=4, hidden=32, lag=1, n_samples=64, precision=0, device=0, flags=0,
                    sample_offset=0, total_samples=0, stream=None, seed=1)
        base.update(kw)
        cfg = binding.CutoffConfig(**base)
        assert lib.cutoff_create(C.byref(h), C.byref(cfg)) == binding.ERR_BAD_ARG
    for kw in (dict(latent_dim=5), dict(hidden=30), dict(n_workers=5000)):
        base = dict(n_workers=16, latent_dim=4, hidden=32, lag=1, n_samples=64, precision=0, device=0, flags=0,
                    sample_offset=0, total_samples=0, stream=None, seed=1)
        base.update(kw)
        cfg = binding.CutoffConfig(**base)
        assert lib.cutoff_create(C.byref(h), C.byref(cfg)) == binding.ERR_UNSUPPORTED


def test_weight_blob_layout():
    wl = inputs.WORKLOADS["tiny"]
    w = inputs.workload_weights(wl)
    blob = binding.pack_weights(w, wl.N, wl.D, wl.H)
    assert struct.unpack("<6I", blob[:24]) == (0x31465443, 1, wl.N, wl.D, wl.H, 0)
    n_floats = sum(int(np.prod(s)) for s in inputs.tensor_shapes(wl.N, wl.D, wl.H).values())
    assert len(blob) == 24 + 4 * n_floats
    first = np.frombuffer(blob, dtype=np.float32, count=wl.H * wl.N, offset=24).reshape(wl.H, wl.N)
    assert np.array_equal(first, w["Wxf"])
    last = np.frombuffer(blob, dtype=np.float32, count=2 * wl.N, offset=len(blob) - 8 * wl.N)
    assert np.array_equal(last, w["b4"])
    with pytest.raises(ValueError):
        bad = dict(w)
        bad["Wxf"] = w["Wxf"].T
        binding.pack_weights(bad, wl.N, wl.D, wl.H)


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library(str(tmp_path / "libcutoff.so"))
