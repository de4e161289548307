"""ctypes binding of libcutoff.so: the same names as include/cutoff.h, argument marshalling only.

Every step of a decision runs in the library's CUDA kernels.  There is no CPU fallback: if the
shared library is missing or does not load, every entry point raises.
"""
from __future__ import annotations

import ctypes as C
import os
import struct

import numpy as np

from .inputs import TENSOR_ORDER, TENSOR_ORDER_LITERAL, tensor_shapes, tensor_shapes_literal

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG_DIR, "libcutoff.so")

OK, WARMUP, DEGENERATE = 0, 1, 2
ERR_BAD_ARG, ERR_BAD_BLOB, ERR_BAD_VALUE, ERR_CUDA = -1, -2, -3, -4
ERR_UNSUPPORTED, ERR_NOMEM, ERR_STATE, ERR_TIMEOUT, ERR_TOO_LARGE = -5, -6, -7, -8, -9
STATIC_MAX_N = 1024
PRECISION_FP32, PRECISION_TF32, PRECISION_BF16W = 0, 1, 2
FLAG_GRAPH = 1
FLAG_LITERAL = 2
BLOB_MAGIC = 0x31465443

EXPORTS = (
    "cutoff_create", "cutoff_destroy", "cutoff_load_weights", "cutoff_push", "cutoff_push_async",
    "cutoff_predict", "cutoff_predict_async", "cutoff_fetch", "cutoff_step", "cutoff_step_device", "cutoff_get_stats",
    "cutoff_get_order_stat_std", "cutoff_get_partial_sums", "cutoff_decide_from_sums", "cutoff_reset", "cutoff_save_state",
    "cutoff_restore_state", "cutoff_strerror", "cutoff_last_error", "cutoff_set_timing",
    "cutoff_get_timing", "cutoff_stage_name", "cutoff_launch_count", "cutoff_set_option",
    "cutoff_debug_normals", "cutoff_debug_samples", "cutoff_debug_window", "cutoff_debug_sort",
    "cutoff_debug_sort_values", "cutoff_predict_partial_async", "cutoff_partial_sums_device",
    "cutoff_decide_from_device_sums", "cutoff_measure_pipe_rates", "cutoff_measure_operand_stream", "cutoff_eval_trace", "cutoff_order_baseline",
    "cutoff_fit_param_count", "cutoff_fit_workspace_bytes", "cutoff_elbo_grad", "cutoff_adam_step",
    "cutoff_sorted_row_sums_static",
)


class CutoffConfig(C.Structure):
    _fields_ = [
        ("n_workers", C.c_int32), ("latent_dim", C.c_int32), ("hidden", C.c_int32), ("lag", C.c_int32),
        ("n_samples", C.c_int32), ("precision", C.c_int32), ("device", C.c_int32), ("flags", C.c_int32),
        ("sample_offset", C.c_int64), ("total_samples", C.c_int64), ("stream", C.c_void_p), ("seed", C.c_uint64),
    ]


class CutoffError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})" + (f": {detail}" if detail else ""))


_lib = None


def load_library(path: str | None = None) -> C.CDLL:
    """Load libcutoff.so (built in-tree by paper_1803_04209_b200.build).  Raises if it is absent."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_1803_04209_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(path)
    vp, i32p, f32p, f64p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_double)
    sig = {
        "cutoff_create": (C.c_int, [C.POINTER(vp), C.POINTER(CutoffConfig)]),
        "cutoff_destroy": (None, [vp]),
        "cutoff_load_weights": (C.c_int, [vp, vp, C.c_size_t]),
        "cutoff_push": (C.c_int, [vp, vp, C.c_int, vp]),
        "cutoff_push_async": (C.c_int, [vp, vp]),
        "cutoff_predict": (C.c_int, [vp, i32p]),
        "cutoff_predict_async": (C.c_int, [vp]),
        "cutoff_fetch": (C.c_int, [vp, i32p]),
        "cutoff_step": (C.c_int, [vp, vp, i32p]),
        "cutoff_step_device": (C.c_int, [vp, vp, i32p]),
        "cutoff_get_stats": (C.c_int, [vp, vp, vp]),
        "cutoff_get_order_stat_std": (C.c_int, [vp, vp]),
        "cutoff_get_partial_sums": (C.c_int, [vp, vp]),
        "cutoff_decide_from_sums": (C.c_int, [vp, vp, i32p]),
        "cutoff_reset": (C.c_int, [vp]),
        "cutoff_save_state": (C.c_int, [vp, vp, C.POINTER(C.c_size_t)]),
        "cutoff_restore_state": (C.c_int, [vp, vp, C.c_size_t]),
        "cutoff_strerror": (C.c_char_p, [C.c_int]),
        "cutoff_last_error": (C.c_char_p, [vp]),
        "cutoff_set_timing": (C.c_int, [vp, C.c_int]),
        "cutoff_get_timing": (C.c_int, [vp, f32p, C.c_int]),
        "cutoff_stage_name": (C.c_char_p, [C.c_int]),
        "cutoff_launch_count": (C.c_int64, [vp]),
        "cutoff_set_option": (C.c_int, [vp, C.c_char_p, C.c_int64]),
        "cutoff_debug_normals": (C.c_int, [C.c_int, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int64, C.c_int64,
                                           C.c_int32, vp, vp]),
        "cutoff_debug_samples": (C.c_int, [vp, C.c_int64, C.c_int64, vp]),
        "cutoff_debug_window": (C.c_int, [vp, vp]),
        "cutoff_debug_sort": (C.c_int, [vp, vp, C.c_int64, C.c_int32, vp, vp]),
        "cutoff_debug_sort_values": (C.c_int, [vp, vp, C.c_int64, C.c_int32, vp]),
        "cutoff_predict_partial_async": (C.c_int, [vp]),
        "cutoff_partial_sums_device": (C.c_int, [vp, C.POINTER(vp)]),
        "cutoff_decide_from_device_sums": (C.c_int, [vp, vp, i32p]),
        "cutoff_measure_pipe_rates": (C.c_int, [C.c_int, f32p]),
        "cutoff_measure_operand_stream": (C.c_int, [C.c_int, f32p]),
        "cutoff_eval_trace": (C.c_int, [C.c_int, vp, C.c_int64, C.c_int32, C.c_int32, vp, C.c_int32, vp, vp, vp, vp, vp,
                                        vp, vp]),
        "cutoff_order_baseline": (C.c_int, [C.c_int, vp, C.c_int64, C.c_int32, C.c_int32, vp, vp]),
        "cutoff_fit_param_count": (C.c_int64, [C.c_int32, C.c_int32, C.c_int32]),
        "cutoff_fit_workspace_bytes": (C.c_int64, [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32]),
        "cutoff_elbo_grad": (C.c_int, [C.c_int, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, vp, vp, vp, vp, vp, vp,
                                       C.c_size_t, vp]),
        "cutoff_adam_step": (C.c_int, [C.c_int, C.c_int64, vp, vp, vp, vp, C.c_int32, C.c_float, C.c_float, C.c_float,
                                       C.c_float, C.c_float, C.c_float, vp, vp, C.c_size_t, vp]),
        "cutoff_sorted_row_sums_static": (C.c_int, [C.c_int, vp, C.c_int64, C.c_int32, C.c_int32, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)          # AttributeError if the library does not export it
        fn.restype = res
        fn.argtypes = args
    if path == LIB_PATH:
        _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().cutoff_strerror(code).decode()


def pack_weights(weights: dict, N: int, D: int, H: int) -> bytes:
    """Serialise a weight dictionary into the blob cutoff_load_weights expects.

    A dictionary that holds "Wg1" is the literal variant (gated transition, emission I / J): its blob
    carries 1 in the header's last word and goes to a context created with FLAG_LITERAL.
    """
    literal = "Wg1" in weights
    shapes = tensor_shapes_literal(N, D, H) if literal else tensor_shapes(N, D, H)
    parts = [struct.pack("<6I", BLOB_MAGIC, 1, N, D, H, 1 if literal else 0)]
    for name in (TENSOR_ORDER_LITERAL if literal else TENSOR_ORDER):
        a = np.ascontiguousarray(weights[name], dtype=np.float32)
        if a.shape != shapes[name]:
            raise ValueError(f"{name}: shape {a.shape}, expected {shapes[name]}")
        parts.append(a.tobytes())
    return b"".join(parts)


def _ptr(a) -> int:
    """Address of a numpy array (host) or of a torch CUDA tensor (device)."""
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()


class Cutoff:
    """One decision context on one GPU and one stream (thin wrapper over the C ABI)."""

    def __init__(self, n_workers: int, latent_dim: int, hidden: int, lag: int, n_samples: int,
                 precision: int = PRECISION_FP32, seed: int = 0, device: int = 0, stream: int | None = None,
                 flags: int = 0, sample_offset: int = 0, total_samples: int = 0):
        self._lib = load_library()
        self.N, self.D, self.H, self.lag, self.S = n_workers, latent_dim, hidden, lag, n_samples
        self.cfg = CutoffConfig(n_workers, latent_dim, hidden, lag, n_samples, precision, device, flags,
                                sample_offset, total_samples, stream or None, seed)
        self._h = C.c_void_p()
        rc = self._lib.cutoff_create(C.byref(self._h), C.byref(self.cfg))
        if rc != OK:
            self._h = C.c_void_p()
            raise CutoffError(rc, "cutoff_create")

    def _check(self, rc: int, where: str) -> int:
        if rc < 0:
            raise CutoffError(rc, where, self._lib.cutoff_last_error(self._h).decode())
        return rc

    def close(self):
        if self._h:
            self._lib.cutoff_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def load_weights(self, weights: dict | bytes):
        blob = weights if isinstance(weights, (bytes, bytearray)) else pack_weights(weights, self.N, self.D, self.H)
        self._check(self._lib.cutoff_load_weights(self._h, blob, len(blob)), "cutoff_load_weights")

    def push(self, runtimes_sec, censored=None) -> int:
        """Host numpy array (fp32, N) or torch CUDA tensor; `censored` (same kind, N bytes / bools) marks killed workers."""
        if isinstance(runtimes_sec, np.ndarray):
            a = np.ascontiguousarray(runtimes_sec, dtype=np.float32)
            if a.shape != (self.N,):
                raise ValueError("expected N run-times")
            mask = None
            if censored is not None:
                mask = np.ascontiguousarray(np.asarray(censored).astype(np.uint8))
                if mask.shape != (self.N,):
                    raise ValueError("expected N censoring flags")
            return self._check(self._lib.cutoff_push(self._h, a.ctypes.data, 0, mask.ctypes.data if mask is not None else None),
                               "cutoff_push")
        if tuple(runtimes_sec.shape) != (self.N,) or not runtimes_sec.is_cuda or not runtimes_sec.is_contiguous():
            raise ValueError("expected a contiguous CUDA tensor of N fp32 run-times")
        mask_ptr = None
        if censored is not None:
            if tuple(censored.shape) != (self.N,) or not censored.is_cuda or censored.element_size() != 1:
                raise ValueError("expected a CUDA tensor of N one-byte censoring flags")
            mask_ptr = censored.data_ptr()
        return self._check(self._lib.cutoff_push(self._h, runtimes_sec.data_ptr(), 1, mask_ptr), "cutoff_push")

    def push_async(self, runtimes_sec_device) -> int:
        return self._check(self._lib.cutoff_push_async(self._h, runtimes_sec_device.data_ptr()), "cutoff_push_async")

    def predict(self):
        """Returns (code, c)."""
        c = C.c_int32(0)
        rc = self._check(self._lib.cutoff_predict(self._h, C.byref(c)), "cutoff_predict")
        return rc, c.value

    def predict_async(self) -> int:
        return self._check(self._lib.cutoff_predict_async(self._h), "cutoff_predict_async")

    def fetch(self):
        c = C.c_int32(0)
        rc = self._check(self._lib.cutoff_fetch(self._h, C.byref(c)), "cutoff_fetch")
        return rc, c.value

    def step(self, runtimes_sec: np.ndarray):
        """push + predict in one call (a CUDA-graph replay when the context has FLAG_GRAPH); returns (code, c)."""
        a = np.ascontiguousarray(runtimes_sec, dtype=np.float32)
        if a.shape != (self.N,):
            raise ValueError("expected N run-times")
        c = C.c_int32(0)
        rc = self._check(self._lib.cutoff_step(self._h, a.ctypes.data, C.byref(c)), "cutoff_step")
        return rc, c.value

    def step_device(self, runtimes_sec_device):
        """As step(), with the run-times in a contiguous CUDA tensor of N fp32 values; returns (code, c)."""
        if tuple(runtimes_sec_device.shape) != (self.N,) or not runtimes_sec_device.is_cuda or not runtimes_sec_device.is_contiguous():
            raise ValueError("expected a contiguous CUDA tensor of N fp32 run-times")
        c = C.c_int32(0)
        rc = self._check(self._lib.cutoff_step_device(self._h, runtimes_sec_device.data_ptr(), C.byref(c)), "cutoff_step_device")
        return rc, c.value

    def get_stats(self):
        """(E[x~_(j)] in seconds, Omega(c) per second) of the last decision."""
        e = np.empty(self.N, dtype=np.float32)
        om = np.empty(self.N, dtype=np.float32)
        self._check(self._lib.cutoff_get_stats(self._h, e.ctypes.data, om.ctypes.data), "cutoff_get_stats")
        return e, om

    def get_order_stat_std(self) -> np.ndarray:
        """Standard deviation of each order statistic over the samples (seconds); needs option order_stat_std."""
        sd = np.empty(self.N, dtype=np.float32)
        self._check(self._lib.cutoff_get_order_stat_std(self._h, sd.ctypes.data), "cutoff_get_order_stat_std")
        return sd

    def get_partial_sums(self) -> np.ndarray:
        s = np.empty(self.N, dtype=np.float64)
        self._check(self._lib.cutoff_get_partial_sums(self._h, s.ctypes.data), "cutoff_get_partial_sums")
        return s

    def decide_from_sums(self, sums: np.ndarray):
        s = np.ascontiguousarray(sums, dtype=np.float64)
        if s.shape != (self.N,):
            raise ValueError("expected N sums")
        c = C.c_int32(0)
        rc = self._check(self._lib.cutoff_decide_from_sums(self._h, s.ctypes.data, C.byref(c)), "cutoff_decide_from_sums")
        return rc, c.value

    def predict_partial_async(self) -> int:
        """Enqueue this context's share of a decision up to the per-position sums; returns OK or WARMUP."""
        return self._check(self._lib.cutoff_predict_partial_async(self._h), "cutoff_predict_partial_async")

    def partial_sums_device_ptr(self) -> int:
        """Device address of the context's N doubles (the per-position sums)."""
        p = C.c_void_p()
        self._check(self._lib.cutoff_partial_sums_device(self._h, C.byref(p)), "cutoff_partial_sums_device")
        return p.value

    def partial_sums_tensor(self):
        """The same array as a torch CUDA tensor that aliases the library's memory (no copy)."""
        import torch

        class _Alias:
            pass
        a = _Alias()
        a.__cuda_array_interface__ = {"shape": (self.N,), "typestr": "<f8", "data": (self.partial_sums_device_ptr(), False),
                                      "version": 2}
        return torch.as_tensor(a, device=torch.device("cuda", self.cfg.device))

    def decide_from_device_sums(self, sums_device):
        """sums_device: a CUDA tensor of N doubles (possibly partial_sums_tensor()); returns (code, c)."""
        if tuple(sums_device.shape) != (self.N,) or not sums_device.is_cuda or sums_device.element_size() != 8:
            raise ValueError("expected a CUDA tensor of N doubles")
        c = C.c_int32(0)
        rc = self._check(self._lib.cutoff_decide_from_device_sums(self._h, sums_device.data_ptr(), C.byref(c)),
                         "cutoff_decide_from_device_sums")
        return rc, c.value

    def reset(self):
        self._check(self._lib.cutoff_reset(self._h), "cutoff_reset")

    def save_state(self) -> bytes:
        n = C.c_size_t(0)
        self._check(self._lib.cutoff_save_state(self._h, None, C.byref(n)), "cutoff_save_state")
        buf = C.create_string_buffer(n.value)
        self._check(self._lib.cutoff_save_state(self._h, buf, C.byref(n)), "cutoff_save_state")
        return buf.raw[: n.value]

    def restore_state(self, blob: bytes):
        self._check(self._lib.cutoff_restore_state(self._h, blob, len(blob)), "cutoff_restore_state")

    def set_timing(self, on: bool):
        self._check(self._lib.cutoff_set_timing(self._h, int(on)), "cutoff_set_timing")

    def get_timing(self) -> dict:
        ms = (C.c_float * 16)()
        n = self._check(self._lib.cutoff_get_timing(self._h, ms, 16), "cutoff_get_timing")
        return {self._lib.cutoff_stage_name(i).decode(): ms[i] for i in range(n)}

    def launch_count(self) -> int:
        return self._lib.cutoff_launch_count(self._h)

    def set_option(self, name: str, value: int):
        self._check(self._lib.cutoff_set_option(self._h, name.encode(), value), "cutoff_set_option")

    def debug_samples(self, k0: int, count: int) -> np.ndarray:
        x = np.empty((count, self.N), dtype=np.float32)
        rc = self._check(self._lib.cutoff_debug_samples(self._h, k0, count, x.ctypes.data), "cutoff_debug_samples")
        if rc == WARMUP:
            raise CutoffError(ERR_STATE, "cutoff_debug_samples", "fewer than lag+1 observations")
        return x

    def debug_window(self) -> np.ndarray:
        w = np.empty((self.lag + 1, self.N), dtype=np.float32)
        rc = self._check(self._lib.cutoff_debug_window(self._h, w.ctypes.data), "cutoff_debug_window")
        if rc == WARMUP:
            raise CutoffError(ERR_STATE, "cutoff_debug_window", "fewer than lag+1 observations")
        return w

    def debug_sort(self, rows: np.ndarray):
        r = np.ascontiguousarray(rows, dtype=np.float32)
        keys = np.empty_like(r)
        perm = np.empty(r.shape, dtype=np.int32)
        self._check(self._lib.cutoff_debug_sort(self._h, r.ctypes.data, r.shape[0], r.shape[1], keys.ctypes.data,
                                                perm.ctypes.data), "cutoff_debug_sort")
        return keys, perm

    def debug_sort_values(self, rows: np.ndarray) -> np.ndarray:
        """Rows sorted ascending by the fp32 network of the decision path."""
        r = np.ascontiguousarray(rows, dtype=np.float32)
        keys = np.empty_like(r)
        self._check(self._lib.cutoff_debug_sort_values(self._h, r.ctypes.data, r.shape[0], r.shape[1], keys.ctypes.data),
                    "cutoff_debug_sort_values")
        return keys


def debug_normals(seed: int, step: int, stream: int, k0: int, count: int, n_elems: int, device: int = 0):
    """(normals[count, n_elems] fp32, words[count, ceil(n_elems/4), 4] uint32) from the GPU generator."""
    lib = load_library()
    nq = (n_elems + 3) // 4
    normals = np.empty((count, n_elems), dtype=np.float32)
    words = np.empty((count, nq, 4), dtype=np.uint32)
    rc = lib.cutoff_debug_normals(device, seed, step, stream, k0, count, n_elems, normals.ctypes.data, words.ctypes.data)
    if rc < 0:
        raise CutoffError(rc, "cutoff_debug_normals")
    return normals, words


def measure_pipe_rates(device: int = 0) -> dict:
    """Measured issue rates (warp-instructions per clock per SM) of fp32 min/max, shuffles and fp32 FMA."""
    lib = load_library()
    out = (C.c_float * 3)()
    rc = lib.cutoff_measure_pipe_rates(device, out)
    if rc < 0:
        raise CutoffError(rc, "cutoff_measure_pipe_rates")
    return {"minmax": float(out[0]), "shuffle": float(out[1]), "fma": float(out[2])}


def measure_operand_stream(device: int = 0) -> dict:
    """Measured rate (GB/s, whole device) of the emission kernel's operand copies L2 -> shared memory."""
    lib = load_library()
    out = (C.c_float * 2)()
    rc = lib.cutoff_measure_operand_stream(device, out)
    if rc < 0:
        raise CutoffError(rc, "cutoff_measure_operand_stream")
    return {"weights_2mb": float(out[0]), "hidden_64mb": float(out[1])}


def eval_trace(trace, cutoffs=None, want_static: bool = True, stream: int | None = None) -> dict:
    """Scores of cutoff rules on a recorded trace (torch CUDA fp32 [T, N]); cutoffs: torch CUDA int32 [M, T] or None.

    Returns torch CUDA tensors: best_c [T] int32, best [T], all [T], achieved [M, T], step_time [M, T] and, if asked
    for, static_c (one int32).  Every number is computed by the library's kernels; this only allocates the outputs.
    """
    import torch
    lib = load_library()
    T, N = trace.shape
    dev = trace.device
    M = 0 if cutoffs is None else cutoffs.shape[0]
    out = {"best_c": torch.empty(T, dtype=torch.int32, device=dev), "best": torch.empty(T, dtype=torch.float32, device=dev),
           "all": torch.empty(T, dtype=torch.float32, device=dev),
           "achieved": torch.empty((M, T), dtype=torch.float32, device=dev),
           "step_time": torch.empty((M, T), dtype=torch.float32, device=dev)}
    if want_static:
        out["static_c"] = torch.zeros(1, dtype=torch.int32, device=dev)
    rc = lib.cutoff_eval_trace(dev.index or 0, trace.data_ptr(), T, N, trace.stride(0),
                               cutoffs.data_ptr() if M else None, M, out["best_c"].data_ptr(), out["best"].data_ptr(),
                               out["all"].data_ptr(), out["achieved"].data_ptr() if M else None,
                               out["step_time"].data_ptr() if M else None,
                               out["static_c"].data_ptr() if want_static else None, stream or None)
    if rc < 0:
        raise CutoffError(rc, "cutoff_eval_trace")
    return out


def order_baseline(trace, stream: int | None = None):
    """Cutoffs of the "order" rule (Elfving's formula on running moments) for a trace (torch CUDA fp32 [T, N])."""
    import torch
    lib = load_library()
    T, N = trace.shape
    out = torch.empty(T, dtype=torch.int32, device=trace.device)
    rc = lib.cutoff_order_baseline(trace.device.index or 0, trace.data_ptr(), T, N, trace.stride(0), out.data_ptr(),
                                   stream or None)
    if rc < 0:
        raise CutoffError(rc, "cutoff_order_baseline")
    return out


def flatten_weights(weights: dict) -> np.ndarray:
    """The compact model's tensors in blob order as one fp32 vector (the parameter vector of the learning calls)."""
    return np.concatenate([np.ascontiguousarray(weights[name], dtype=np.float32).reshape(-1) for name in TENSOR_ORDER])


def unflatten_weights(flat: np.ndarray, N: int, D: int, H: int) -> dict:
    out, o = {}, 0
    for name in TENSOR_ORDER:
        shape = tensor_shapes(N, D, H)[name]
        n = int(np.prod(shape))
        out[name] = np.asarray(flat[o:o + n], dtype=np.float32).reshape(shape).copy()
        o += n
    return out


class Fitter:
    """Training steps of the compact model on one GPU: device buffers owned here, arithmetic in the library."""

    def __init__(self, N: int, D: int, H: int, lag: int, batch: int, weights: dict, device: int = 0):
        import torch
        self._lib = load_library()
        self.N, self.D, self.H, self.lag, self.batch, self.device = N, D, H, lag, batch, device
        dev = torch.device("cuda", device)
        self.n = int(self._lib.cutoff_fit_param_count(N, D, H))
        flat = flatten_weights(weights)
        assert flat.size == self.n
        self.params = torch.from_numpy(flat).to(dev)
        self.grads = torch.zeros(self.n, dtype=torch.float32, device=dev)
        self.m = torch.zeros_like(self.grads)
        self.v = torch.zeros_like(self.grads)
        self.elbo = torch.zeros(batch, dtype=torch.float32, device=dev)
        self.norm = torch.zeros(1, dtype=torch.float32, device=dev)
        ws = int(self._lib.cutoff_fit_workspace_bytes(N, D, H, lag, batch))
        self.ws = torch.empty(max(ws, 4096), dtype=torch.uint8, device=dev)
        self.t = 0

    def elbo_grad(self, xhat, eps, want_grad: bool = True):
        """xhat [batch, lag+1, N], eps [batch, lag+1, D]: contiguous fp32 CUDA tensors.  Returns (elbo, grads) tensors."""
        import torch
        rc = self._lib.cutoff_elbo_grad(self.device, self.N, self.D, self.H, self.lag, self.batch, self.params.data_ptr(),
                                        xhat.data_ptr(), eps.data_ptr(), self.elbo.data_ptr(),
                                        self.grads.data_ptr() if want_grad else None, self.ws.data_ptr(), self.ws.numel(),
                                        torch.cuda.current_stream().cuda_stream)
        if rc < 0:
            raise CutoffError(rc, "cutoff_elbo_grad")
        return self.elbo, self.grads

    def capture_elbo_grad(self, xhat, eps):
        """Capture elbo_grad(xhat, eps) in a CUDA graph.  xhat and eps are fixed tensors: the caller refills them (on the
        current stream) before every replay_elbo_grad().  A step is some 150 small dependent launches, so a replay
        costs a fraction of launching them one by one."""
        import torch
        self.elbo_grad(xhat, eps)                      # once outside the capture
        torch.cuda.current_stream().synchronize()
        self._graph_inputs = (xhat, eps)
        self._graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self._graph):
            self.elbo_grad(xhat, eps)

    def replay_elbo_grad(self):
        """Replay the captured step on the current contents of the captured input tensors; returns (elbo, grads)."""
        self._graph.replay()
        return self.elbo, self.grads

    def adam_step(self, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, clip=10.0, grad_scale=None):
        """One Adam step on the negative mean ELBO (grad_scale = -1/batch) with clipping by the global norm."""
        import torch
        self.t += 1
        scale = -1.0 / self.batch if grad_scale is None else grad_scale
        rc = self._lib.cutoff_adam_step(self.device, self.n, self.params.data_ptr(), self.grads.data_ptr(), self.m.data_ptr(),
                                        self.v.data_ptr(), self.t, lr, beta1, beta2, eps, clip, scale, self.norm.data_ptr(),
                                        self.ws.data_ptr(), self.ws.numel(), torch.cuda.current_stream().cuda_stream)
        if rc < 0:
            raise CutoffError(rc, "cutoff_adam_step")

    def weights(self) -> dict:
        return unflatten_weights(self.params.cpu().numpy(), self.N, self.D, self.H)


def sorted_row_sums_static(x, sums, n: int | None = None, stream: int | None = None) -> int:
    """Allocation-free sum of sorted rows: x (torch CUDA fp32 [rows, ldx]) -> sums (torch CUDA fp64 [n]).

    Both tensors belong to the caller; the call itself allocates nothing (its scratch is a fixed
    array inside the library).  Returns the library's code; raises on an error code.
    """
    lib = load_library()
    n = x.shape[1] if n is None else n
    rc = lib.cutoff_sorted_row_sums_static(x.device.index or 0, x.data_ptr(), x.shape[0], n, x.stride(0),
                                           sums.data_ptr(), stream or None)
    if rc < 0:
        raise CutoffError(rc, "cutoff_sorted_row_sums_static")
    return rc
