"""Run-time cutoff decision of Cutoff SGD (arXiv 1803.04209) for one B200, behind a C ABI.

`binding` wraps libcutoff.so (hand-written sm_100a CUDA kernels), `build` compiles it in-tree,
`inputs` draws the seeded synthetic weights and run-time traces.
"""
from . import binding, inputs  # noqa: F401
from .binding import Cutoff, CutoffError, debug_normals, load_library, pack_weights  # noqa: F401
