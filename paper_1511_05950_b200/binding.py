"""ctypes binding of libsoftsync_ps.so: argument marshalling only.

Every step of the parameter-server path (timestamps, staleness, grouping, the
scale table, the fused update kernel) runs inside the C-ABI library declared in
include/softsync_ps.h.  PyTorch is used here for device memory and streams.
There is no CPU fallback: if the library has not been built, importing this
module raises.
"""
from __future__ import annotations

import collections
import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np
import torch

from . import build as _build

# ---- constants mirrored from include/softsync_ps.h ---------------------------
PS_MOD_CONSTANT, PS_MOD_INV_STALENESS, PS_MOD_EXP_STALENESS = 0, 1, 2
PS_OK, PS_READY = 0, 1
PS_ERR_INVALID_ARG, PS_ERR_BAD_LEARNER, PS_ERR_BAD_TIMESTAMP, PS_ERR_NOT_READY = -1, -2, -3, -4
PS_ERR_QUEUE_FULL, PS_ERR_CUDA, PS_ERR_NOMEM, PS_ERR_NO_STATE, PS_ERR_LOG_EVICTED, PS_ERR_BARRIER = -5, -6, -7, -8, -9, -10
PS_ERR_DEVICE_WAIT, PS_ERR_STATIC_LIMIT = -11, -12
PS_STATIC_MAX_BLOCKS, PS_STATIC_MAX_GRADS = 1024, 16
PS_GRAD_FP32, PS_GRAD_BF16 = 0, 1
(PS_OPT_GRAD_DTYPE, PS_OPT_FUSE_T, PS_OPT_STREAM, PS_OPT_QUEUE_GROUPS, PS_OPT_LOG_UPDATES,
 PS_OPT_TIMING, PS_OPT_KERNEL, PS_OPT_BLOCK_THREADS, PS_OPT_OVERLAP_LAUNCH, PS_OPT_PROTOCOL,
 PS_OPT_GROUP_SIZE, PS_OPT_LAST_KERNEL, PS_OPT_LAUNCHES_SCALAR, PS_OPT_LAUNCHES_VECTOR, PS_OPT_LAUNCHES_BULK,
 PS_OPT_BULK_TILE, PS_OPT_BULK_STAGES, PS_OPT_BULK_WAIT_LIMIT, PS_OPT_BULK_SELFTEST, PS_OPT_ZIGZAG) = range(1, 21)
PS_PROTOCOL_SOFTSYNC, PS_PROTOCOL_HARDSYNC = 0, 1
PS_KERNEL_AUTO, PS_KERNEL_SCALAR, PS_KERNEL_VECTOR, PS_KERNEL_BULK = 0, 1, 2, 3
PS_MAX_GROUP, PS_MAX_FUSE_T, PS_MAX_ENTRIES, PS_MAX_LAYERS, PS_MAX_REPLICAS = 256, 16, 512, 64, 8

MODULATIONS = {"constant": PS_MOD_CONSTANT, "inv_staleness": PS_MOD_INV_STALENESS, "exp_staleness": PS_MOD_EXP_STALENESS}
KERNELS = {"auto": PS_KERNEL_AUTO, "scalar": PS_KERNEL_SCALAR, "vector": PS_KERNEL_VECTOR, "bulk": PS_KERNEL_BULK}
TORCH_DTYPE = {"fp32": torch.float32, "bf16": torch.bfloat16}
GRAD_DTYPES = {"fp32": PS_GRAD_FP32, "bf16": PS_GRAD_BF16}

LOG_DTYPE = np.dtype([
    ("update", "<i8"), ("push_index", "<i8"), ("ts_grad", "<i8"), ("tau", "<i8"), ("sigma", "<i8"),
    ("learner", "<i4"), ("position", "<i4"), ("scale", "<f4"), ("decay", "<f4"),
], align=True)

EXPORTS = (
    "ps_create", "ps_destroy", "ps_bind_state", "ps_init_weights", "ps_bind_staging", "ps_bind_weight_mirror",
    "ps_pull_weights_bf16",
    "ps_set_option", "ps_get_option", "ps_set_alpha0", "ps_set_penalty_base", "ps_set_layer_multipliers",
    "ps_slot_wait", "ps_slot_written", "ps_kernel_status", "ps_pull_weights", "ps_pull_weights_host", "ps_pull_weights_host_async",
    "ps_push_gradient", "ps_push_gradient_host", "ps_acquire_slot", "ps_push_slot", "ps_release_slot", "ps_apply_update", "ps_flush", "ps_synchronize",
    "ps_get_update_log", "ps_peek_state", "ps_export_state", "ps_import_state", "ps_kernel_time", "ps_last_cuda_error", "ps_status_string",
    "ps_fused_update_static", "ps_bind_weight_replicas",
)


class SoftsyncError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, status_string(status), status))


def _load() -> C.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise RuntimeError(
            "libsoftsync_ps.so is not built (%s). Run `python -m paper_1511_05950_b200.build`; "
            "there is no CPU fallback." % path)
    L = C.CDLL(path)
    vp, i64, i32, f32 = C.c_void_p, C.c_int64, C.c_int, C.c_float
    sig = {
        "ps_create": [C.POINTER(vp), i64, i32, i32, f32, f32, f32, i32],
        "ps_destroy": [vp],
        "ps_bind_state": [vp, vp, vp],
        "ps_init_weights": [vp, vp, i32],
        "ps_bind_staging": [vp, vp, i64, i32],
        "ps_bind_weight_mirror": [vp, vp],
        "ps_bind_weight_replicas": [vp, i32, C.POINTER(vp)],
        "ps_pull_weights_bf16": [vp, vp, C.POINTER(i64)],
        "ps_set_option": [vp, i32, i64],
        "ps_get_option": [vp, i32, C.POINTER(i64)],
        "ps_set_alpha0": [vp, f32],
        "ps_set_penalty_base": [vp, f32],
        "ps_set_layer_multipliers": [vp, i32, vp, vp, vp],
        "ps_slot_wait": [vp, i32, vp],
        "ps_slot_written": [vp, i32, vp],
        "ps_kernel_status": [vp, C.POINTER(i32), C.POINTER(i32), C.POINTER(i64), C.POINTER(i32)],
        "ps_pull_weights": [vp, vp, C.POINTER(i64)],
        "ps_pull_weights_host": [vp, vp, C.POINTER(i64)],
        "ps_pull_weights_host_async": [vp, vp, C.POINTER(i64)],
        "ps_push_gradient": [vp, i32, vp, i64],
        "ps_push_gradient_host": [vp, i32, vp, i64],
        "ps_acquire_slot": [vp, C.POINTER(vp), C.POINTER(i32)],
        "ps_push_slot": [vp, i32, i32, i64],
        "ps_release_slot": [vp, i32],
        "ps_apply_update": [vp],
        "ps_flush": [vp],
        "ps_synchronize": [vp],
        "ps_get_update_log": [vp, i64, i64, vp],
        "ps_peek_state": [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(i64), C.POINTER(i64)],
        "ps_export_state": [vp, vp, i64],
        "ps_import_state": [vp, vp, i64],
        "ps_kernel_time": [vp, C.POINTER(C.c_double), C.POINTER(i64)],
        "ps_last_cuda_error": [vp],
        "ps_status_string": [i32],
        "ps_fused_update_static": [vp, vp, i64, C.POINTER(vp), C.POINTER(f32), i32, f32, f32, i32, i32, vp, C.POINTER(i32)],
    }
    for name, argtypes in sig.items():
        fn = getattr(L, name)
        fn.argtypes = argtypes
        fn.restype = C.c_char_p if name == "ps_status_string" else C.c_int
    assert LOG_DTYPE.itemsize == 56
    return L


lib = _load()

# The C entry points under their own names, for callers that want the raw ABI.
ps_create = lib.ps_create
ps_destroy = lib.ps_destroy
ps_bind_state = lib.ps_bind_state
ps_init_weights = lib.ps_init_weights
ps_bind_staging = lib.ps_bind_staging
ps_bind_weight_mirror = lib.ps_bind_weight_mirror
ps_bind_weight_replicas = lib.ps_bind_weight_replicas
ps_pull_weights_bf16 = lib.ps_pull_weights_bf16
ps_set_option = lib.ps_set_option
ps_get_option = lib.ps_get_option
ps_set_alpha0 = lib.ps_set_alpha0
ps_set_penalty_base = lib.ps_set_penalty_base
ps_set_layer_multipliers = lib.ps_set_layer_multipliers
ps_slot_wait = lib.ps_slot_wait
ps_slot_written = lib.ps_slot_written
ps_kernel_status = lib.ps_kernel_status
ps_pull_weights = lib.ps_pull_weights
ps_pull_weights_host = lib.ps_pull_weights_host
ps_pull_weights_host_async = lib.ps_pull_weights_host_async
ps_push_gradient = lib.ps_push_gradient
ps_push_gradient_host = lib.ps_push_gradient_host
ps_acquire_slot = lib.ps_acquire_slot
ps_push_slot = lib.ps_push_slot
ps_release_slot = lib.ps_release_slot
ps_apply_update = lib.ps_apply_update
ps_flush = lib.ps_flush
ps_synchronize = lib.ps_synchronize
ps_get_update_log = lib.ps_get_update_log
ps_peek_state = lib.ps_peek_state
ps_kernel_time = lib.ps_kernel_time
ps_export_state = lib.ps_export_state
ps_import_state = lib.ps_import_state
ps_last_cuda_error = lib.ps_last_cuda_error
ps_fused_update_static = lib.ps_fused_update_static


def status_string(status: int) -> str:
    return lib.ps_status_string(status).decode()


def _check(status: int, where: str) -> int:
    if status < 0:
        raise SoftsyncError(status, where)
    return status


def require_tensor(t: torch.Tensor, dtype: torch.dtype, count: int, what: str, on_gpu: bool,
                   device: Optional[torch.device] = None) -> None:
    """The library sees only an address.  Refuse a tensor whose memory is not what a kernel or copy that
    reads or writes `count` elements of `dtype` there will assume: wrong element type, too short, strided,
    or (on_gpu) not on the server's GPU."""
    if t.dtype != dtype:
        raise TypeError("%s must be %s, got %s" % (what, dtype, t.dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % what)
    if t.numel() < count:
        raise ValueError("%s holds %d elements, the server has %d parameters" % (what, t.numel(), count))
    if on_gpu and count > 0:
        if not t.is_cuda:
            raise ValueError("%s must live on the server's GPU" % what)
        if device is not None and t.device != device:
            raise ValueError("%s is on %s, the server on %s" % (what, t.device, device))
    if not on_gpu and t.is_cuda:
        raise ValueError("%s must live in host memory" % what)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def fused_update_static(w: torch.Tensor, v: torch.Tensor, grads, scales, decay: float, momentum: float,
                        blocks: int = 0, read_status: bool = True) -> int:
    """ps_fused_update_static: one weight update from `grads` (a list of c device tensors, fp32 or bf16)
    with the given per-gradient scales, for callers that may not allocate device or pinned memory while
    they run (the kernel's status records sit in the library's static device memory).  Marshals the
    arguments and nothing else; the work goes to torch's current stream on w's device.  Returns how many
    blocks gave up on a copy wait (0: complete) when read_status is set, which waits for the stream."""
    n = w.numel()
    require_tensor(w, torch.float32, n, "weights", on_gpu=True)
    require_tensor(v, torch.float32, n, "momentum", on_gpu=True, device=w.device)
    if len(grads) != len(scales) or not grads:
        raise ValueError("one scale per gradient, at least one gradient")
    gdt = grads[0].dtype
    if gdt not in (torch.float32, torch.bfloat16):
        raise TypeError("gradients must be fp32 or bf16")
    for g in grads:
        require_tensor(g, gdt, n, "gradient", on_gpu=True, device=w.device)
    ptrs = (C.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
    sc = (C.c_float * len(grads))(*[float(x) for x in scales])
    gave_up = C.c_int(0)
    with torch.cuda.device(w.device):
        stream = torch.cuda.current_stream(w.device).cuda_stream
        _check(ps_fused_update_static(w.data_ptr(), v.data_ptr(), n, ptrs, sc, len(grads), decay, momentum,
                                      PS_GRAD_BF16 if gdt == torch.bfloat16 else PS_GRAD_FP32, blocks,
                                      C.c_void_p(stream), C.byref(gave_up) if read_status else None),
               "ps_fused_update_static")
    return gave_up.value


class ParameterServer:
    """One n-softsync parameter server on the current CUDA device.

    Owns the device memory (torch tensors) that the library is bound to and
    keeps pushed gradient tensors alive until the update that consumes them
    has been enqueued.  Method names follow the C ABI.
    """

    def __init__(self, num_params: int, num_learners: int, n: int, alpha0: float, momentum: float = 0.0,
                 weight_decay: float = 0.0, modulation: str = "inv_staleness", grad_dtype: str = "fp32",
                 fuse_t: int = 1, device: Optional[torch.device] = None,
                 state: Optional[Tuple[torch.Tensor, torch.Tensor]] = None, allocate: bool = True):
        self._h = C.c_void_p()
        self.num_params = int(num_params)
        self.num_learners = int(num_learners)
        self.c = 0                    # group size of Eq. 2, asked from the library once it exists
        self.grad_dtype = grad_dtype
        self._held = collections.deque()
        self._host_held = []          # pinned host gradients whose upload may still be in flight
        self._staging = None
        self.w = self.v = self.mirror = None
        self.replicas = []
        if device is None and (allocate or state is not None) and num_params > 0:
            device = torch.device("cuda", torch.cuda.current_device())
        self.device = device
        ctx = torch.cuda.device(device) if device is not None and device.type == "cuda" else _NullCtx()
        with ctx:
            _check(ps_create(C.byref(self._h), num_params, num_learners, n, alpha0, momentum, weight_decay,
                             MODULATIONS[modulation]), "ps_create")
        self.c = self.get_option(PS_OPT_GROUP_SIZE)
        if state is not None:
            self.bind_state(*state)
        elif allocate and num_params > 0:
            self.bind_state(torch.empty(num_params, dtype=torch.float32, device=device),
                            torch.empty(num_params, dtype=torch.float32, device=device))
        if grad_dtype != "fp32":
            self.set_option(PS_OPT_GRAD_DTYPE, GRAD_DTYPES[grad_dtype])
        if fuse_t != 1:
            self.set_option(PS_OPT_FUSE_T, fuse_t)
        if device is not None and device.type == "cuda":
            self.set_option(PS_OPT_STREAM, torch.cuda.current_stream(device).cuda_stream)

    # -- lifetime -------------------------------------------------------------
    def destroy(self) -> None:
        if self._h:
            _check(ps_destroy(self._h), "ps_destroy")
            self._h = C.c_void_p()
            self._held.clear()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- set-up ---------------------------------------------------------------
    def _check_device_tensor(self, t: torch.Tensor, dtype: torch.dtype, what: str) -> None:
        require_tensor(t, dtype, self.num_params, what, on_gpu=True, device=self.device)

    def bind_state(self, w: torch.Tensor, v: torch.Tensor) -> None:
        self._check_device_tensor(w, torch.float32, "weights")
        self._check_device_tensor(v, torch.float32, "momentum")
        _check(ps_bind_state(self._h, w.data_ptr(), v.data_ptr()), "ps_bind_state")
        self.w, self.v = w, v

    def init_weights(self, w0: torch.Tensor) -> None:
        if w0.is_cuda:
            self._check_device_tensor(w0, torch.float32, "initial weights")
        else:
            self._check_host_tensor(w0, torch.float32, "initial weights")
        _check(ps_init_weights(self._h, w0.data_ptr(), 0 if w0.is_cuda else 1), "ps_init_weights")
        self._held.clear()

    def bind_staging(self, num_slots: int) -> None:
        elem = 2 if self.grad_dtype == "bf16" else 4
        slot_bytes = (self.num_params * elem + 255) // 256 * 256
        buf = torch.empty(max(1, slot_bytes * num_slots), dtype=torch.uint8, device=self.device)
        _check(ps_bind_staging(self._h, buf.data_ptr(), slot_bytes, num_slots), "ps_bind_staging")
        self._staging = buf

    def bind_weight_mirror(self, mirror: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Keep a bf16 copy of the weights current in `mirror` (allocated here if not given)."""
        if mirror is None:
            mirror = torch.empty(max(1, self.num_params), dtype=torch.bfloat16, device=self.device)
        self._check_device_tensor(mirror, torch.bfloat16, "weight mirror")
        _check(ps_bind_weight_mirror(self._h, mirror.data_ptr()), "ps_bind_weight_mirror")
        self.mirror = mirror
        return mirror

    def bind_weight_replicas(self, replicas) -> None:
        """Keep further fp32 copies of the weights current: every update stores the new theta into each tensor of
        `replicas` as well (tensors of num_params fp32 this GPU can address; an empty list unbinds)."""
        replicas = list(replicas)
        for t in replicas:
            require_tensor(t, torch.float32, self.num_params, "weight replica", on_gpu=True)
        ptrs = (C.c_void_p * max(1, len(replicas)))(*[t.data_ptr() for t in replicas])
        _check(ps_bind_weight_replicas(self._h, len(replicas), ptrs), "ps_bind_weight_replicas")
        self.replicas = replicas

    def set_option(self, key: int, value: int) -> None:
        _check(ps_set_option(self._h, key, int(value)), "ps_set_option")

    def set_alpha0(self, alpha0: float) -> None:
        """Base learning rate for gradients pushed from now on."""
        _check(ps_set_alpha0(self._h, alpha0), "ps_set_alpha0")

    def set_penalty_base(self, rho: float) -> None:
        """Base of the exponential staleness penalty alpha0 * rho**tau (modulation "exp_staleness")."""
        _check(ps_set_penalty_base(self._h, rho), "ps_set_penalty_base")

    def set_layer_multipliers(self, bounds, lr_mult, wd_mult) -> None:
        """Layer q = elements [bounds[q], bounds[q+1]) with learning-rate and weight-decay multipliers;
        empty lists remove the table."""
        bounds = np.ascontiguousarray(bounds, dtype=np.int64)
        lr_mult = np.ascontiguousarray(lr_mult, dtype=np.float32)
        wd_mult = np.ascontiguousarray(wd_mult, dtype=np.float32)
        n = int(lr_mult.size)
        if n and (wd_mult.size != n or bounds.size != n + 1):
            raise ValueError("need num_layers multipliers of each kind and num_layers + 1 bounds")
        _check(ps_set_layer_multipliers(self._h, n, bounds.ctypes.data if n else None,
                                        lr_mult.ctypes.data if n else None, wd_mult.ctypes.data if n else None),
               "ps_set_layer_multipliers")

    def get_option(self, key: int) -> int:
        out = C.c_int64()
        _check(ps_get_option(self._h, key, C.byref(out)), "ps_get_option")
        return out.value

    # -- the protocol ----------------------------------------------------------
    def pull_weights(self, out: Optional[torch.Tensor] = None, non_blocking: bool = False) -> int:
        """Timestamp a gradient computed from now on must carry; fills `out` with the weights if given
        (fp32 on the device or the host, or bf16 on the device when a mirror is bound).
        non_blocking (host `out` only): return once the copy is enqueued; call synchronize() before reading."""
        ts = C.c_int64()
        if out is None:
            _check(ps_pull_weights(self._h, None, C.byref(ts)), "ps_pull_weights")
            return ts.value
        applied_before = self.timestamps()[0]
        if out.dtype == torch.bfloat16:
            self._check_device_tensor(out, torch.bfloat16, "bf16 pull target")
            _check(ps_pull_weights_bf16(self._h, out.data_ptr(), C.byref(ts)), "ps_pull_weights_bf16")
        elif out.is_cuda:
            self._check_device_tensor(out, torch.float32, "pull target")
            _check(ps_pull_weights(self._h, out.data_ptr(), C.byref(ts)), "ps_pull_weights")
        else:
            self._check_host_tensor(out, torch.float32, "host pull target")
            if non_blocking:
                _check(ps_pull_weights_host_async(self._h, out.data_ptr(), C.byref(ts)), "ps_pull_weights_host_async")
            else:
                _check(ps_pull_weights_host(self._h, out.data_ptr(), C.byref(ts)), "ps_pull_weights_host")
        self._release(self.timestamps()[0] - applied_before)     # the pull applied every complete group first
        return ts.value

    def _check_host_tensor(self, t: torch.Tensor, dtype: torch.dtype, what: str) -> None:
        require_tensor(t, dtype, self.num_params, what, on_gpu=False)

    def _release(self, groups: int) -> None:
        """Drop the references to the gradients of `groups` applied groups (oldest first)."""
        for _ in range(groups * self.c):
            self._held.popleft()

    def push_gradient(self, learner: int, grad: torch.Tensor, ts: int) -> bool:
        """True if this push completed a group of c (an update can be applied)."""
        want = TORCH_DTYPE[self.grad_dtype]
        if grad.is_cuda:
            self._check_device_tensor(grad, want, "gradient")
            r = _check(ps_push_gradient(self._h, learner, grad.data_ptr(), ts), "ps_push_gradient")
            self._held.append(grad)
        else:
            self._check_host_tensor(grad, want, "host gradient")
            r = _check(ps_push_gradient_host(self._h, learner, grad.data_ptr(), ts), "ps_push_gradient_host")
            self._held.append(None)
            self._host_held.append(grad)
            if len(self._host_held) > 1024:
                self.synchronize()
        return r == PS_READY

    def acquire_slot(self, dtype: Optional[torch.dtype] = None):
        """(slot id, tensor view of a server-owned receive slot) for a learner to write its gradient into."""
        ptr, sid = C.c_void_p(), C.c_int()
        _check(ps_acquire_slot(self._h, C.byref(ptr), C.byref(sid)), "ps_acquire_slot")
        elem = 2 if self.grad_dtype == "bf16" else 4
        off = ptr.value - self._staging.data_ptr()
        view = self._staging[off: off + self.num_params * elem].view(
            torch.bfloat16 if self.grad_dtype == "bf16" else torch.float32)
        return sid.value, view

    def push_slot(self, learner: int, slot_id: int, ts: int) -> bool:
        r = _check(ps_push_slot(self._h, learner, slot_id, ts), "ps_push_slot")
        self._held.append(None)
        return r == PS_READY

    def slot_wait(self, slot_id: int, stream: torch.cuda.Stream) -> None:
        """Make `stream` wait until the update kernel that last read this (recycled) slot has finished."""
        _check(ps_slot_wait(self._h, slot_id, stream.cuda_stream), "ps_slot_wait")

    def slot_written(self, slot_id: int, stream: torch.cuda.Stream) -> None:
        """Tell the server that the slot's gradient is produced by the work enqueued on `stream` so far."""
        _check(ps_slot_written(self._h, slot_id, stream.cuda_stream), "ps_slot_written")

    def release_slot(self, slot_id: int) -> None:
        _check(ps_release_slot(self._h, slot_id), "ps_release_slot")

    def apply_update(self) -> int:
        done = _check(ps_apply_update(self._h), "ps_apply_update")
        self._release(done)
        return done

    def flush(self) -> int:
        done = _check(ps_flush(self._h), "ps_flush")
        self._release(done)
        return done

    def synchronize(self) -> None:
        _check(ps_synchronize(self._h), "ps_synchronize")
        self._host_held.clear()

    # -- inspection -------------------------------------------------------------
    def timestamps(self) -> Tuple[int, int]:
        """(applied, logical)."""
        a, l = C.c_int64(), C.c_int64()
        _check(ps_peek_state(self._h, None, None, C.byref(a), C.byref(l)), "ps_peek_state")
        return a.value, l.value

    def update_log(self, first_update: int = 0, count: Optional[int] = None) -> np.ndarray:
        if count is None:
            count = self.timestamps()[0] - first_update
        out = np.empty(count * self.c, dtype=LOG_DTYPE)
        _check(ps_get_update_log(self._h, first_update, count, out.ctypes.data if out.size else None),
               "ps_get_update_log")
        return out

    def export_state(self) -> np.ndarray:
        """Protocol state (timestamp, rate, push counts) as int64 words; weights and momentum are self.w, self.v."""
        out = np.empty(8 + self.num_learners, dtype=np.int64)          # PS_STATE_WORDS(lambda)
        n = _check(ps_export_state(self._h, out.ctypes.data, out.size), "ps_export_state")
        return out[:n].copy()

    def import_state(self, words: np.ndarray) -> None:
        words = np.ascontiguousarray(words, dtype=np.int64)
        _check(ps_import_state(self._h, words.ctypes.data, words.size), "ps_import_state")

    def staleness_histogram(self, first_update: int = 0) -> np.ndarray:
        """counts[t] = gradients applied with staleness t (the quantity of Fig. 1), from the held update log."""
        return np.bincount(self.update_log(first_update)["tau"])

    def kernel_status(self):
        """(code, block, tile, stage) of the bulk-copy kernel's status record; code 0 = no wait has run out."""
        code, block, tile, stage = C.c_int(), C.c_int(), C.c_int64(), C.c_int()
        _check(ps_kernel_status(self._h, C.byref(code), C.byref(block), C.byref(tile), C.byref(stage)), "ps_kernel_status")
        return code.value, block.value, tile.value, stage.value

    def kernel_time(self) -> Tuple[float, int]:
        ms, n = C.c_double(), C.c_int64()
        _check(ps_kernel_time(self._h, C.byref(ms), C.byref(n)), "ps_kernel_time")
        return ms.value, n.value


class _NullCtx:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False
