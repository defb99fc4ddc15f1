"""C-ABI surface and host-side protocol logic, without a GPU.

A server with zero parameters launches nothing, so its whole state machine
(timestamps, staleness, grouping, scale table, log, error codes) can be driven
here and compared field by field with the reference.
"""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_1511_05950_b200 as P
from oracle import reference as R
from tests.helpers import PULL

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE_GRAD = 0x1000          # never dereferenced: zero-length gradients


def declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"^\s*(?:int|const char \*)\s*\*?(ps_\w+)\s*\(", text, flags=re.M)
    return names


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 30 and "ps_apply_update" in names and "ps_slot_wait" in names
    for n in names:
        assert hasattr(P.lib, n), n
    assert sorted(names) == sorted(P.binding.EXPORTS)


def make(lam, n, alpha0=0.01, m=0.9, wd=5e-4, mod=P.PS_MOD_INV_STALENESS, num_params=0):
    h = C.c_void_p()
    rc = P.ps_create(C.byref(h), num_params, lam, n, alpha0, m, wd, mod)
    return rc, h


def drive(h, kinds, learners, fuse_t=1, lazy=False):
    """Replay a trace; apply as soon as a group completes (or lazily, T at a time)."""
    assert P.ps_set_option(h, P.PS_OPT_FUSE_T, fuse_t) == 0
    pulled = {}
    ts = C.c_int64()
    ready = 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            assert P.ps_pull_weights(h, None, C.byref(ts)) == 0
            pulled[l] = ts.value
        else:
            rc = P.ps_push_gradient(h, l, FAKE_GRAD, pulled[l])
            assert rc in (P.PS_OK, P.PS_READY)
            ready += rc == P.PS_READY
            if ready and (not lazy or ready == fuse_t):
                assert P.ps_apply_update(h) == ready
                ready = 0
    assert P.ps_flush(h) == ready


def fetch_log(h, c):
    a = C.c_int64()
    assert P.ps_peek_state(h, None, None, C.byref(a), None) == 0
    out = np.empty(a.value * c, dtype=P.binding.LOG_DTYPE)
    assert P.ps_get_update_log(h, 0, a.value, out.ctypes.data) == 0
    return a.value, out


@pytest.mark.parametrize("model,lam,n,mod", [
    ("rounds", 4, 1, "inv_staleness"), ("exp", 30, 30, "inv_staleness"), ("uniform", 18, 4, "inv_staleness"),
    ("lognormal", 54, 54, "inv_staleness"), ("exp", 12, 3, "constant"), ("lognormal", 9, 2, "inv_staleness"),
])
@pytest.mark.parametrize("fuse_t,lazy", [(1, False), (8, True)])
def test_schedule_matches_reference_bit_exactly(model, lam, n, mod, fuse_t, lazy):
    pushes = 600
    kinds, learners = R.simulate_arrivals(model, lam, pushes, 42)
    ref = R.ReferencePS(0, lam, n, 0.01, 0.9, 5e-4, P.binding.MODULATIONS[mod], 32)
    ref.set_weights(np.zeros(0, np.float32))
    nothing = np.zeros(0, np.float32)
    counts = {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        ref.pull(l) if k == PULL else ref.push(l, nothing)
    rlog = ref.log()

    rc, h = make(lam, n, mod=P.binding.MODULATIONS[mod])
    assert rc == 0
    drive(h, kinds, learners, fuse_t, lazy)
    c = lam // n
    ts, log = fetch_log(h, c)
    assert ts == ref.timestamp == pushes // c
    for f in ("update", "push_index", "ts_grad", "tau", "sigma", "learner", "position"):
        assert np.array_equal(log[f], rlog[f]), f
    assert np.array_equal(log["scale"], rlog["scale"].astype(np.float32))      # fp32 reference: exact widening
    assert np.array_equal(log["decay"], rlog["decay"].astype(np.float32))
    assert P.ps_destroy(h) == 0


@pytest.mark.parametrize("rho", [0.5, 0.75, 1.0])
@pytest.mark.parametrize("fuse_t,lazy", [(1, False), (4, True)])
def test_exponential_penalty_schedule_matches_reference(rho, fuse_t, lazy):
    """Scales alpha0 * rho^tau / c, the decay coefficient and the logged staleness, bit for bit."""
    lam, n, pushes = 12, 3, 480
    kinds, learners = R.simulate_arrivals("exp", lam, pushes, 7)
    ref = R.ReferencePS(0, lam, n, 0.02, 0.9, 5e-4, R.MOD_EXP_STALENESS, 32)
    ref.set_penalty_base(rho)
    nothing = np.zeros(0, np.float32)
    for k, l in zip(kinds.tolist(), learners.tolist()):
        ref.pull(l) if k == PULL else ref.push(l, nothing)
    rlog = ref.log()
    rc, h = make(lam, n, alpha0=0.02, mod=P.PS_MOD_EXP_STALENESS)
    assert rc == 0 and P.ps_set_penalty_base(h, rho) == 0
    drive(h, kinds, learners, fuse_t, lazy)
    ts, log = fetch_log(h, lam // n)
    assert ts == ref.timestamp
    for f in ("update", "push_index", "ts_grad", "tau", "sigma", "learner", "position"):
        assert np.array_equal(log[f], rlog[f]), f
    assert np.array_equal(log["scale"], rlog["scale"].astype(np.float32))
    assert np.array_equal(log["decay"], rlog["decay"].astype(np.float32))
    assert np.array_equal(log["sigma"], log["tau"]) and log["tau"].max() > 4
    P.ps_destroy(h)


def test_penalty_base_and_layer_table_argument_checks():
    rc, h = make(2, 1, num_params=0)
    for bad in (0.0, -0.5, 1.5, float("nan")):
        assert P.ps_set_penalty_base(h, bad) == P.PS_ERR_INVALID_ARG
    assert P.ps_set_penalty_base(h, 1.0) == 0
    b0 = np.array([0, 0, 0], np.int64)
    one = np.ones(2, np.float32)
    assert P.ps_set_layer_multipliers(h, 2, b0.ctypes.data, one.ctypes.data, one.ctypes.data) == 0   # empty layers are fine
    assert P.ps_set_layer_multipliers(h, 0, None, None, None) == 0
    assert P.ps_set_layer_multipliers(h, 2, None, one.ctypes.data, one.ctypes.data) == P.PS_ERR_INVALID_ARG
    assert P.ps_set_layer_multipliers(h, P.PS_MAX_LAYERS + 1, b0.ctypes.data, one.ctypes.data, one.ctypes.data) == P.PS_ERR_INVALID_ARG
    bad = np.array([0, 1, 0], np.int64)                                         # does not end at num_params
    assert P.ps_set_layer_multipliers(h, 2, bad.ctypes.data, one.ctypes.data, one.ctypes.data) == P.PS_ERR_INVALID_ARG
    nan = np.array([1.0, np.nan], np.float32)
    assert P.ps_set_layer_multipliers(h, 2, b0.ctypes.data, nan.ctypes.data, one.ctypes.data) == P.PS_ERR_INVALID_ARG
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, 0) == P.PS_OK                    # a gradient is pending now
    assert P.ps_set_penalty_base(h, 0.5) == P.PS_ERR_INVALID_ARG
    assert P.ps_set_layer_multipliers(h, 2, b0.ctypes.data, one.ctypes.data, one.ctypes.data) == P.PS_ERR_INVALID_ARG
    P.ps_destroy(h)
    h2 = C.c_void_p()
    assert P.ps_create(C.byref(h2), 0, 2, 1, 0.1, 0.0, 0.0, 3) == P.PS_ERR_INVALID_ARG     # no such modulation


def test_read_only_options_and_kernel_options():
    rc, h = make(7, 2)
    v = C.c_int64()
    assert P.ps_get_option(h, P.PS_OPT_GROUP_SIZE, C.byref(v)) == 0 and v.value == 3        # floor(7 / 2)
    for key in (P.PS_OPT_LAST_KERNEL, P.PS_OPT_LAUNCHES_SCALAR, P.PS_OPT_LAUNCHES_VECTOR, P.PS_OPT_LAUNCHES_BULK):
        assert P.ps_get_option(h, key, C.byref(v)) == 0 and v.value == 0
        assert P.ps_set_option(h, key, 1) == P.PS_ERR_INVALID_ARG
    assert P.ps_set_option(h, P.PS_OPT_GROUP_SIZE, 4) == P.PS_ERR_INVALID_ARG
    assert P.ps_set_option(h, P.PS_OPT_KERNEL, P.PS_KERNEL_BULK) == 0
    assert P.ps_set_option(h, P.PS_OPT_KERNEL, 4) == P.PS_ERR_INVALID_ARG
    for key, good, bads in ((P.PS_OPT_BULK_TILE, (0, 256, 1024, 8192), (100, 384, 16384, -1)),
                            (P.PS_OPT_BULK_STAGES, (2, 8), (1, 9)),
                            (P.PS_OPT_BULK_WAIT_LIMIT, (16, 1 << 20), (0, 15)),
                            (P.PS_OPT_BULK_SELFTEST, (0, 1), (2, -1)),
                            (P.PS_OPT_ZIGZAG, (0, 1), (2, -1))):
        for g in good:
            assert P.ps_set_option(h, key, g) == 0
            assert P.ps_get_option(h, key, C.byref(v)) == 0 and v.value == g
        for b in bads:
            assert P.ps_set_option(h, key, b) == P.PS_ERR_INVALID_ARG
    code, tile = C.c_int(-1), C.c_int64(-1)
    assert P.ps_kernel_status(h, C.byref(code), None, C.byref(tile), None) == 0 and code.value == 0
    P.ps_destroy(h)


def test_binding_refuses_tensors_the_kernel_would_misread():
    """The library sees addresses only; the binding checks type, length, layout and placement before it
    hands one over.  Nothing here launches a kernel."""
    import torch
    from paper_1511_05950_b200.binding import require_tensor
    f32, bf = torch.float32, torch.bfloat16
    require_tensor(torch.zeros(16), f32, 16, "x", on_gpu=False)
    require_tensor(torch.zeros(20)[2:18], f32, 16, "x", on_gpu=False)       # an offset view is fine
    with pytest.raises(TypeError):
        require_tensor(torch.zeros(16, dtype=bf), f32, 16, "x", on_gpu=False)          # would read 4N bytes of a 2N buffer
    with pytest.raises(TypeError):
        require_tensor(torch.zeros(16, dtype=torch.float64), f32, 16, "x", on_gpu=False)
    with pytest.raises(ValueError):
        require_tensor(torch.zeros(15), f32, 16, "x", on_gpu=False)                   # too short
    with pytest.raises(ValueError):
        require_tensor(torch.zeros(32)[::2], f32, 16, "x", on_gpu=False)              # strided
    with pytest.raises(ValueError):
        require_tensor(torch.zeros(16), f32, 16, "x", on_gpu=True)                    # host memory as a device operand
    # through the class, on a server without parameters (no GPU needed): the element type is still checked
    ps = P.ParameterServer(0, 2, 1, 0.1)
    with pytest.raises(TypeError):
        ps.push_gradient(0, torch.zeros(0, dtype=bf), 0)
    with pytest.raises(TypeError):
        ps.pull_weights(torch.zeros(0, dtype=torch.float16))
    with pytest.raises(TypeError):
        ps.init_weights(torch.zeros(0, dtype=torch.float64))
    assert ps.timestamps() == (0, 0)                                        # nothing reached the server
    ps.destroy()
    b16 = P.ParameterServer(0, 2, 1, 0.1, grad_dtype="bf16")
    with pytest.raises(TypeError):
        b16.push_gradient(0, torch.zeros(0), 0)                             # fp32 into a bf16 server
    b16.destroy()


def test_rate_schedule_applies_to_later_pushes_only():
    rc, h = make(2, 1, alpha0=0.5, m=0.0, wd=0.0)
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, 0) == P.PS_OK
    assert P.ps_set_alpha0(h, 0.25) == 0
    assert P.ps_set_alpha0(h, float("nan")) == P.PS_ERR_INVALID_ARG
    assert P.ps_push_gradient(h, 1, FAKE_GRAD, 0) == P.PS_READY
    assert P.ps_apply_update(h) == 1
    ts, log = fetch_log(h, 2)
    assert log["scale"].tolist() == [0.25, 0.125]          # as in the hand-worked example
    P.ps_destroy(h)


def test_logical_clock_runs_ahead_of_applied_clock():
    rc, h = make(2, 2)
    ts, a, l = C.c_int64(), C.c_int64(), C.c_int64()
    for i in range(5):
        assert P.ps_pull_weights(h, None, C.byref(ts)) == 0 and ts.value == i
        assert P.ps_push_gradient(h, 0, FAKE_GRAD, ts.value) == P.PS_READY
    P.ps_peek_state(h, None, None, C.byref(a), C.byref(l))
    assert (a.value, l.value) == (0, 5)
    P.ps_set_option(h, P.PS_OPT_FUSE_T, 3)
    assert P.ps_apply_update(h) == 3 and P.ps_apply_update(h) == 2
    assert P.ps_apply_update(h) == P.PS_ERR_NOT_READY
    P.ps_peek_state(h, None, None, C.byref(a), C.byref(l))
    assert (a.value, l.value) == (5, 5)
    P.ps_destroy(h)


def test_error_codes():
    h = C.c_void_p()
    assert P.ps_create(None, 0, 1, 1, 0.1, 0.0, 0.0, 1) == P.PS_ERR_INVALID_ARG
    assert P.ps_create(C.byref(h), 0, 3, 4, 0.1, 0.0, 0.0, 1) == P.PS_ERR_INVALID_ARG      # n > lambda
    assert P.ps_create(C.byref(h), 0, 3, 0, 0.1, 0.0, 0.0, 1) == P.PS_ERR_INVALID_ARG
    assert P.ps_create(C.byref(h), -1, 3, 1, 0.1, 0.0, 0.0, 1) == P.PS_ERR_INVALID_ARG
    assert P.ps_create(C.byref(h), 0, 3, 1, 0.1, 0.0, 0.0, 7) == P.PS_ERR_INVALID_ARG      # modulation
    assert P.ps_create(C.byref(h), 0, 1000, 1, 0.1, 0.0, 0.0, 1) == P.PS_ERR_INVALID_ARG   # c > PS_MAX_GROUP
    assert P.ps_create(C.byref(h), 0, 3, 1, float("nan"), 0.0, 0.0, 1) == P.PS_ERR_INVALID_ARG
    rc, h = make(3, 1)
    assert rc == 0
    ts = C.c_int64()
    assert P.ps_pull_weights(h, None, None) == P.PS_ERR_INVALID_ARG
    assert P.ps_push_gradient(h, 3, FAKE_GRAD, 0) == P.PS_ERR_BAD_LEARNER
    assert P.ps_push_gradient(h, -1, FAKE_GRAD, 0) == P.PS_ERR_BAD_LEARNER
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, 1) == P.PS_ERR_BAD_TIMESTAMP       # from the future: tau < 0
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, -1) == P.PS_ERR_BAD_TIMESTAMP
    assert P.ps_push_gradient(h, 0, FAKE_GRAD + 2, 0) == P.PS_ERR_INVALID_ARG     # fp32 needs 4-byte alignment
    assert P.ps_apply_update(h) == P.PS_ERR_NOT_READY
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, 0) == P.PS_OK
    assert P.ps_push_gradient(h, 1, FAKE_GRAD, 0) == P.PS_OK
    assert P.ps_apply_update(h) == P.PS_ERR_NOT_READY                             # 2 of 3 pending
    assert P.ps_set_option(h, P.PS_OPT_GRAD_DTYPE, P.PS_GRAD_BF16) == P.PS_ERR_INVALID_ARG  # while pending
    assert P.ps_push_gradient(h, 1, FAKE_GRAD, 0) == P.PS_READY
    # rejected calls left the state untouched
    a, l = C.c_int64(), C.c_int64()
    P.ps_peek_state(h, None, None, C.byref(a), C.byref(l))
    assert (a.value, l.value) == (0, 1)
    for key, bad in ((P.PS_OPT_FUSE_T, 0), (P.PS_OPT_FUSE_T, 17), (P.PS_OPT_QUEUE_GROUPS, 0), (P.PS_OPT_KERNEL, 9),
                     (P.PS_OPT_BLOCK_THREADS, 100), (P.PS_OPT_BLOCK_THREADS, 1024), (99, 1), (P.PS_OPT_GRAD_DTYPE, 5)):
        assert P.ps_set_option(h, key, bad) == P.PS_ERR_INVALID_ARG
    assert P.ps_get_update_log(h, 0, 1, None) == P.PS_ERR_INVALID_ARG
    buf = np.empty(3, dtype=P.binding.LOG_DTYPE)
    assert P.ps_get_update_log(h, 0, 1, buf.ctypes.data) == P.PS_ERR_LOG_EVICTED   # not applied yet
    assert P.ps_apply_update(h) == 1
    assert P.ps_get_update_log(h, 0, 1, buf.ctypes.data) == 0
    assert buf["learner"].tolist() == [0, 1, 1] and buf["push_index"].tolist() == [0, 0, 1]
    assert P.ps_destroy(h) == 0
    assert P.ps_destroy(h) == P.PS_ERR_INVALID_ARG                                 # use after destroy is refused
    assert P.ps_apply_update(h) == P.PS_ERR_INVALID_ARG
    assert P.ps_destroy(None) == P.PS_ERR_INVALID_ARG


def test_queue_limit_and_log_window():
    rc, h = make(1, 1)
    assert P.ps_set_option(h, P.PS_OPT_QUEUE_GROUPS, 4) == 0
    assert P.ps_set_option(h, P.PS_OPT_LOG_UPDATES, 3) == 0
    for i in range(4):
        assert P.ps_push_gradient(h, 0, FAKE_GRAD, i) == P.PS_READY
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, 4) == P.PS_ERR_QUEUE_FULL
    assert P.ps_flush(h) == 4
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, 4) == P.PS_READY
    assert P.ps_flush(h) == 1
    buf = np.empty(3, dtype=P.binding.LOG_DTYPE)
    assert P.ps_get_update_log(h, 1, 3, buf.ctypes.data) == P.PS_ERR_LOG_EVICTED
    assert P.ps_get_update_log(h, 2, 3, buf.ctypes.data) == 0
    assert buf["update"].tolist() == [2, 3, 4]
    P.ps_destroy(h)


def test_group_larger_than_one_launch_clamps_fusion():
    rc, h = make(256, 1)                      # c = 256: at most 2 groups fit PS_MAX_ENTRIES
    assert rc == 0
    P.ps_set_option(h, P.PS_OPT_FUSE_T, 16)
    for g in range(5):
        for l in range(256):
            P.ps_push_gradient(h, l, FAKE_GRAD, 0)
    assert [P.ps_apply_update(h) for _ in range(3)] == [2, 2, 1]
    P.ps_destroy(h)


def test_weight_mirror_argument_checks():
    rc, h = make(2, 1)
    assert P.ps_bind_weight_mirror(h, 0x1001) == P.PS_ERR_INVALID_ARG           # odd address
    assert P.ps_bind_weight_mirror(None, 0x1000) == P.PS_ERR_INVALID_ARG
    assert P.ps_bind_weight_mirror(h, 0x1000) == 0                              # zero parameters: nothing is written
    ts = C.c_int64()
    assert P.ps_pull_weights_bf16(h, None, C.byref(ts)) == P.PS_ERR_INVALID_ARG
    assert P.ps_pull_weights_bf16(h, 0x2000, C.byref(ts)) == 0 and ts.value == 0
    assert P.ps_bind_weight_mirror(h, None) == 0                                # unbind
    assert P.ps_pull_weights_bf16(h, 0x2000, C.byref(ts)) == P.PS_ERR_NO_STATE
    P.ps_destroy(h)


def test_weight_replica_argument_checks():
    rc, h = make(2, 1)
    ptrs = (C.c_void_p * 9)(*[0x1000 * (k + 1) for k in range(9)])
    assert P.ps_bind_weight_replicas(h, 9, ptrs) == P.PS_ERR_INVALID_ARG         # more than PS_MAX_REPLICAS
    assert P.ps_bind_weight_replicas(h, -1, ptrs) == P.PS_ERR_INVALID_ARG
    assert P.ps_bind_weight_replicas(h, 2, None) == P.PS_ERR_INVALID_ARG
    assert P.ps_bind_weight_replicas(None, 1, ptrs) == P.PS_ERR_INVALID_ARG
    odd = (C.c_void_p * 1)(0x1002)
    assert P.ps_bind_weight_replicas(h, 1, odd) == P.PS_ERR_INVALID_ARG          # not 4-byte aligned
    null = (C.c_void_p * 2)(0x1000, None)
    assert P.ps_bind_weight_replicas(h, 2, null) == P.PS_ERR_INVALID_ARG
    assert P.ps_bind_weight_replicas(h, 8, ptrs) == 0                            # zero parameters: nothing is written
    assert P.ps_push_gradient(h, 0, FAKE_GRAD, 0) == P.PS_OK
    assert P.ps_push_gradient(h, 1, FAKE_GRAD, 0) == P.PS_READY
    assert P.ps_bind_weight_replicas(h, 0, None) == P.PS_ERR_INVALID_ARG         # a complete group is pending
    assert P.ps_apply_update(h) == 1
    assert P.ps_bind_weight_replicas(h, 0, None) == 0                            # unbind
    P.ps_destroy(h)


def test_checkpoint_on_a_group_boundary_resumes_the_same_schedule():
    lam, n, pushes = 6, 2, 120
    c = lam // n
    kinds, learners = R.simulate_arrivals("lognormal", lam, pushes, 77)
    ref = R.ReferencePS(0, lam, n, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(np.zeros(0, np.float32))
    nothing = np.zeros(0, np.float32)
    rc, h = make(lam, n)
    pulled, ts, done, cut = {}, C.c_int64(), 0, None
    words = np.empty(8 + lam, dtype=np.int64)
    for i, (k, l) in enumerate(zip(kinds.tolist(), learners.tolist())):
        if k == PULL:
            ref.pull(l)
            assert P.ps_pull_weights(h, None, C.byref(ts)) == 0
            pulled[l] = ts.value
            continue
        ref.push(l, nothing)
        if cut is None and done == 58 and done % c != 0:
            assert P.ps_export_state(h, words.ctypes.data, words.size) == P.PS_ERR_NOT_READY    # mid-group
        r = P.ps_push_gradient(h, l, FAKE_GRAD, pulled[l])
        done += 1
        if r == P.PS_READY:
            assert P.ps_apply_update(h) == 1
            if cut is None and done >= 60:
                if done == 60:
                    P.ps_set_alpha0(h, 0.005); ref.set_alpha0(0.005)
                assert P.ps_export_state(h, words.ctypes.data, 3) == P.PS_ERR_INVALID_ARG      # too small
                assert P.ps_export_state(h, words.ctypes.data, words.size) == 8 + lam
                cut = done // c
                assert P.ps_destroy(h) == 0
                rc, h = make(lam, n)                                    # a new server takes over
                bad = words.copy(); bad[3] = lam + 1
                assert P.ps_import_state(h, bad.ctypes.data, bad.size) == P.PS_ERR_INVALID_ARG
                assert P.ps_import_state(h, words.ctypes.data, words.size - 1) == P.PS_ERR_INVALID_ARG
                assert P.ps_import_state(h, words.ctypes.data, words.size) == 0
                assert P.ps_peek_state(h, None, None, C.byref(ts), None) == 0 and ts.value == cut
    n_upd = pushes // c
    out = np.empty((n_upd - cut) * c, dtype=P.binding.LOG_DTYPE)
    assert P.ps_get_update_log(h, cut, n_upd - cut, out.ctypes.data) == 0
    assert P.ps_get_update_log(h, cut - 1, 1, out.ctypes.data) == P.PS_ERR_LOG_EVICTED          # log restarts at the cut
    rlog = ref.log()[cut * c:]
    for f in ("update", "push_index", "ts_grad", "tau", "sigma", "learner", "position"):
        assert np.array_equal(out[f], rlog[f]), f
    assert np.array_equal(out["scale"], rlog["scale"].astype(np.float32))
    P.ps_destroy(h)


def test_hardsync_mode_enforces_the_barrier():
    rc, h = make(3, 3)
    assert P.ps_set_option(h, P.PS_OPT_PROTOCOL, P.PS_PROTOCOL_HARDSYNC) == P.PS_ERR_INVALID_ARG   # needs n = 1
    P.ps_destroy(h)
    rc, h = make(3, 1)
    assert P.ps_set_option(h, P.PS_OPT_PROTOCOL, 2) == P.PS_ERR_INVALID_ARG
    assert P.ps_set_option(h, P.PS_OPT_PROTOCOL, P.PS_PROTOCOL_HARDSYNC) == 0
    out = C.c_int64()
    assert P.ps_get_option(h, P.PS_OPT_PROTOCOL, C.byref(out)) == 0 and out.value == 1
    for rnd in range(4):
        assert P.ps_push_gradient(h, 1, FAKE_GRAD, rnd) == P.PS_OK
        assert P.ps_push_gradient(h, 1, FAKE_GRAD, rnd) == P.PS_ERR_BARRIER        # twice in one round
        if rnd:
            assert P.ps_push_gradient(h, 0, FAKE_GRAD, rnd - 1) == P.PS_ERR_BAD_TIMESTAMP   # old weights
        assert P.ps_push_gradient(h, 0, FAKE_GRAD, rnd) == P.PS_OK
        assert P.ps_set_option(h, P.PS_OPT_PROTOCOL, 0) == P.PS_ERR_INVALID_ARG   # not in mid-round
        assert P.ps_push_gradient(h, 2, FAKE_GRAD, rnd) == P.PS_READY
        assert P.ps_apply_update(h) == 1
    ts, log = fetch_log(h, 3)
    assert ts == 4 and (log["tau"] == 0).all() and log["learner"].tolist() == [0, 1, 2] * 4
    assert P.status_string(P.PS_ERR_BARRIER).startswith("hardsync")
    P.ps_destroy(h)


def test_receive_slot_bookkeeping():
    rc, h = make(2, 1)
    ptr, sid, sid2 = C.c_void_p(), C.c_int(), C.c_int()
    assert P.ps_acquire_slot(h, C.byref(ptr), C.byref(sid)) == P.PS_ERR_NO_STATE            # nothing bound
    assert P.ps_bind_staging(h, 0x10000, 256, 2) == 0
    assert P.ps_acquire_slot(h, C.byref(ptr), C.byref(sid)) == 0 and ptr.value in (0x10000, 0x10100)
    assert P.ps_acquire_slot(h, C.byref(ptr), C.byref(sid2)) == 0 and sid2.value != sid.value
    assert P.ps_acquire_slot(h, C.byref(ptr), C.byref(sid2)) == P.PS_ERR_QUEUE_FULL
    assert P.ps_push_slot(h, 5, sid.value, 0) == P.PS_ERR_BAD_LEARNER                      # slot stays lent
    assert P.ps_push_slot(h, 0, sid.value, 0) == P.PS_OK
    assert P.ps_push_slot(h, 0, sid.value, 0) == P.PS_ERR_INVALID_ARG                      # already handed over
    assert P.ps_release_slot(h, sid.value) == P.PS_ERR_INVALID_ARG
    assert P.ps_release_slot(h, sid2.value) == 0
    assert P.ps_release_slot(h, sid2.value) == P.PS_ERR_INVALID_ARG                        # not lent any more
    P.ps_destroy(h)


def test_status_strings():
    assert P.status_string(P.PS_ERR_BAD_TIMESTAMP).startswith("gradient timestamp")
    assert P.status_string(0) == "ok"


def test_compute_without_a_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    rc, h = make(2, 1, num_params=1024)
    assert rc == P.PS_ERR_CUDA and not h.value
    with pytest.raises(P.SoftsyncError):
        P.ParameterServer(1024, 2, 1, 0.1, allocate=False)


def test_unbuilt_library_fails_loudly_but_build_module_imports(tmp_path):
    """A checkout without the built .so: the build module is importable, anything else raises."""
    import shutil
    import subprocess
    import sys
    pkg = tmp_path / "paper_1511_05950_b200"
    pkg.mkdir()
    src = os.path.join(ROOT, "paper_1511_05950_b200")
    for fn in os.listdir(src):
        if fn.endswith(".py"):
            shutil.copy(os.path.join(src, fn), pkg / fn)
    code = ("from paper_1511_05950_b200 import build\n"
            "assert build.is_stale()\n"
            "import paper_1511_05950_b200 as P\n"
            "try:\n    P.ParameterServer\nexcept RuntimeError as e:\n    assert 'not built' in str(e); print('loud')\n")
    out = subprocess.run([sys.executable, "-c", code], cwd=tmp_path, capture_output=True, text=True,
                         env={**os.environ, "PYTHONPATH": str(tmp_path)})
    assert out.returncode == 0 and "loud" in out.stdout, out.stderr


def test_plain_c_client_compiles_links_and_runs(tmp_path):
    """The header is C (not only C++): a C99 program built with gcc drives the protocol calls."""
    import subprocess
    libdir = os.path.join(ROOT, "paper_1511_05950_b200")
    exe = str(tmp_path / "c_abi_client")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "c_abi_client.c"), "-o", exe,
                    "-L", libdir, "-l:libsoftsync_ps.so", "-Wl,-rpath," + libdir], check=True)
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0 and "c client ok" in out.stdout, out.stdout + out.stderr


@pytest.mark.gpu
def test_c_latency_client_drives_the_small_configuration_from_c(tmp_path):
    """The per-update latency figures of the small (launch-bound) configurations come from a C program,
    tests/c_latency_client.c, so that no interpreter sits between the calls.  Built with gcc against the
    library and the CUDA runtime, run for a short while; its lines are printed (pytest -s shows them)."""
    import subprocess
    libdir = os.path.join(ROOT, "paper_1511_05950_b200")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = str(tmp_path / "c_latency_client")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-O2", "-I", os.path.join(ROOT, "include"),
                    "-isystem", os.path.join(cuda, "include"), os.path.join(ROOT, "tests", "c_latency_client.c"),
                    "-o", exe, "-L", libdir, "-l:libsoftsync_ps.so", "-Wl,-rpath," + libdir,
                    "-L", os.path.join(cuda, "lib64"), "-lcudart", "-Wl,-rpath," + os.path.join(cuda, "lib64")], check=True)
    out = subprocess.run([exe, "4000"], capture_output=True, text=True, timeout=300)
    print(out.stdout)
    assert out.returncode == 0 and "c latency client ok" in out.stdout, out.stdout + out.stderr
    per_update = [float(line.split()[-4]) for line in out.stdout.splitlines() if line.endswith("us per update")]
    assert len(per_update) == 5 and all(0.0 < x < 200.0 for x in per_update)
