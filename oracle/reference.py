"""ctypes front end of the C reference (oracle/softsync_oracle.c, arrival_sim.c).

TEST INFRASTRUCTURE: argument marshalling only; all reference arithmetic is in
the C sources.  numpy in, numpy out.
"""
from __future__ import annotations

import contextlib
import ctypes as C
from typing import Optional, Tuple

import numpy as np

from . import build as _build

MOD_CONSTANT = 0
MOD_INV_STALENESS = 1
MOD_EXP_STALENESS = 2
GRAD_FP32 = 0
GRAD_BF16 = 1

ARRIVAL_MODELS = {"rounds": 0, "exp": 1, "uniform": 2, "lognormal": 3}
PULL = 0
PUSH = 1

LOG_DTYPE = np.dtype([
    ("update", "<i8"), ("push_index", "<i8"), ("ts_grad", "<i8"), ("tau", "<i8"), ("sigma", "<i8"),
    ("learner", "<i4"), ("position", "<i4"), ("scale", "<f8"), ("decay", "<f8"),
], align=True)

_lib = None


def load(path: str) -> C.CDLL:
    """Load one build of the C reference and declare its signatures."""
    if True:
        L = C.CDLL(path)
        L.oracle_ps_create.restype = C.c_void_p
        L.oracle_ps_create.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_float, C.c_float, C.c_float, C.c_int, C.c_int]
        L.oracle_ps_destroy.argtypes = [C.c_void_p]
        L.oracle_ps_set_weights.argtypes = [C.c_void_p, C.c_void_p]
        L.oracle_ps_set_alpha0.argtypes = [C.c_void_p, C.c_float]
        L.oracle_ps_set_hardsync.argtypes = [C.c_void_p, C.c_int]
        L.oracle_ps_set_penalty_base.argtypes = [C.c_void_p, C.c_float]
        L.oracle_ps_set_layer_multipliers.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_ps_timestamp.restype = C.c_int64
        L.oracle_ps_timestamp.argtypes = [C.c_void_p]
        L.oracle_ps_group_size.argtypes = [C.c_void_p]
        L.oracle_ps_pull.restype = C.c_int64
        L.oracle_ps_pull.argtypes = [C.c_void_p, C.c_int]
        L.oracle_ps_push.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int]
        L.oracle_ps_push_with_timestamp.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int64]
        L.oracle_ps_get_state.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_ps_get_weights_bf16.argtypes = [C.c_void_p, C.c_void_p]
        L.oracle_round_to_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.oracle_ps_log_size.restype = C.c_int64
        L.oracle_ps_log_size.argtypes = [C.c_void_p]
        L.oracle_ps_get_log.argtypes = [C.c_void_p, C.c_void_p]
        L.oracle_simulate_arrivals.restype = C.c_int64
        L.oracle_simulate_arrivals.argtypes = [C.c_int, C.c_int, C.c_int64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_int64]
        L.oracle_simulate_arrivals_timed.restype = C.c_int64
        L.oracle_simulate_arrivals_timed.argtypes = [C.c_int, C.c_int, C.c_int64, C.c_uint64, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_int64]
        assert LOG_DTYPE.itemsize == 64
    return L


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = load(_build.build())
    return _lib


@contextlib.contextmanager
def use_library(path: str):
    """Temporarily route every call to another build (the tests' planted-mistake builds)."""
    global _lib
    saved = _lib
    _lib = load(path)
    try:
        yield
    finally:
        _lib = saved


def simulate_arrivals(model: str, num_learners: int, num_pushes: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Event trace (kind, learner) of the reference's arrival simulator."""
    cap = num_learners + 2 * num_pushes
    kind = np.empty(cap, dtype=np.int32)
    learner = np.empty(cap, dtype=np.int32)
    n = lib().oracle_simulate_arrivals(ARRIVAL_MODELS[model], num_learners, num_pushes, seed,
                                       kind.ctypes.data, learner.ctypes.data, cap)
    if n < 0:
        raise ValueError("oracle_simulate_arrivals rejected its arguments")
    return kind[:n].copy(), learner[:n].copy()


def simulate_arrivals_timed(model: str, num_learners: int, num_pushes: int, seed: int):
    """(kind, learner, simulated time) of the same trace simulate_arrivals returns."""
    cap = num_learners + 2 * num_pushes
    kind = np.empty(cap, dtype=np.int32)
    learner = np.empty(cap, dtype=np.int32)
    when = np.empty(cap, dtype=np.float64)
    n = lib().oracle_simulate_arrivals_timed(ARRIVAL_MODELS[model], num_learners, num_pushes, seed,
                                             kind.ctypes.data, learner.ctypes.data, when.ctypes.data, cap)
    if n < 0:
        raise ValueError("oracle_simulate_arrivals_timed rejected its arguments")
    return kind[:n].copy(), learner[:n].copy(), when[:n].copy()


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even, by the reference's own routine."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.size, dtype=np.uint16)
    lib().oracle_round_to_bf16(x.ctypes.data, out.ctypes.data, x.size)
    return out.reshape(x.shape)


class ReferencePS:
    """The reference parameter server; precision 32 (fp32 state) or 64."""

    def __init__(self, num_params: int, num_learners: int, n: int, alpha0: float, momentum: float,
                 weight_decay: float, modulation: int = MOD_INV_STALENESS, precision: int = 32):
        self._h = lib().oracle_ps_create(num_params, num_learners, n, alpha0, momentum, weight_decay,
                                         modulation, precision)
        if not self._h:
            raise ValueError("oracle_ps_create rejected its arguments")
        self.num_params = num_params
        self.c = lib().oracle_ps_group_size(self._h)

    def close(self) -> None:
        if self._h:
            lib().oracle_ps_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:              # interpreter shutdown: the module's globals may be gone already
            pass

    def set_weights(self, w0: np.ndarray) -> None:
        w0 = np.ascontiguousarray(w0, dtype=np.float32)
        assert w0.size == self.num_params
        lib().oracle_ps_set_weights(self._h, w0.ctypes.data)

    def set_hardsync(self, on: bool = True) -> None:
        """Switch to the hardsync protocol (needs n = 1, nothing pending)."""
        if lib().oracle_ps_set_hardsync(self._h, int(on)) != 0:
            raise ValueError("hardsync needs n = 1 and no pending gradient")

    def set_penalty_base(self, rho: float) -> None:
        """Base of the exponential staleness penalty alpha0 * rho**tau (MOD_EXP_STALENESS)."""
        if lib().oracle_ps_set_penalty_base(self._h, rho) != 0:
            raise ValueError("penalty base must lie in (0, 1]")

    def set_layer_multipliers(self, bounds, lr_mult, wd_mult) -> None:
        """Layer q = elements [bounds[q], bounds[q+1]) with learning-rate and decay multipliers."""
        bounds = np.ascontiguousarray(bounds, dtype=np.int64)
        lr_mult = np.ascontiguousarray(lr_mult, dtype=np.float32)
        wd_mult = np.ascontiguousarray(wd_mult, dtype=np.float32)
        nseg = lr_mult.size
        assert wd_mult.size == nseg and bounds.size == nseg + 1
        if lib().oracle_ps_set_layer_multipliers(self._h, nseg, bounds.ctypes.data, lr_mult.ctypes.data,
                                                 wd_mult.ctypes.data) != 0:
            raise ValueError("layer bounds must tile [0, num_params)")

    def set_alpha0(self, alpha0: float) -> None:
        """Base learning rate for gradients pushed from now on."""
        lib().oracle_ps_set_alpha0(self._h, alpha0)

    @property
    def timestamp(self) -> int:
        return lib().oracle_ps_timestamp(self._h)

    def pull(self, learner: int) -> int:
        ts = lib().oracle_ps_pull(self._h, learner)
        if ts < 0:
            raise ValueError("bad learner id")
        return ts

    def push(self, learner: int, grad: np.ndarray, timestamp: Optional[int] = None) -> bool:
        """grad: float32 values, or uint16 holding bf16 bit patterns.  timestamp: the clock value the
        gradient carries; by default the one this learner pulled last."""
        grad = np.ascontiguousarray(grad)
        assert grad.size == self.num_params
        if grad.dtype == np.float32:
            kind = GRAD_FP32
        elif grad.dtype == np.uint16:
            kind = GRAD_BF16
        else:
            raise TypeError("gradient must be float32 or uint16 (bf16 bits)")
        if timestamp is None:
            r = lib().oracle_ps_push(self._h, learner, grad.ctypes.data, kind)
        else:
            r = lib().oracle_ps_push_with_timestamp(self._h, learner, grad.ctypes.data, kind, timestamp)
        if r < 0:
            raise ValueError("oracle_ps_push failed with %d" % r)
        return bool(r)

    def state(self) -> Tuple[np.ndarray, np.ndarray]:
        """(w, v) widened to float64 (exact for precision 32)."""
        w = np.empty(self.num_params, dtype=np.float64)
        v = np.empty(self.num_params, dtype=np.float64)
        lib().oracle_ps_get_state(self._h, w.ctypes.data, v.ctypes.data)
        return w, v

    def weights_bf16(self) -> np.ndarray:
        """Weights rounded to bf16 (uint16 bit patterns); fp32 state only."""
        out = np.empty(self.num_params, dtype=np.uint16)
        if lib().oracle_ps_get_weights_bf16(self._h, out.ctypes.data) != 0:
            raise ValueError("bf16 weights are defined for precision 32 only")
        return out

    def log(self) -> np.ndarray:
        n = lib().oracle_ps_log_size(self._h)
        out = np.empty(n, dtype=LOG_DTYPE)
        if n:
            lib().oracle_ps_get_log(self._h, out.ctypes.data)
        return out
