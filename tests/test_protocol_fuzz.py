"""Randomised protocol schedules: the library's decisions against the reference's, call by call.

A seeded random driver mixes timestamp pulls, pushes, learning-rate changes, explicit applies (any number
of groups may be pending, any fusion depth), flushes and weight pulls.  The reference applies every group
the moment it completes; the library may defer and fuse.  Timestamps returned by every pull, and the
complete update log (membership, order, staleness, scales, decay), must agree exactly.  Runs with zero
parameters on the CPU; the GPU variant adds a small vector and compares the weights too.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_1511_05950_b200 as P
from oracle import reference as R
from workloads import generators as G

FAKE = 0x1000


def drive(seed, lam, n, num_params=0, device=None, steps=400):
    rng = np.random.default_rng(seed)
    mod = R.MOD_INV_STALENESS if seed % 3 else R.MOD_CONSTANT
    ref = R.ReferencePS(num_params, lam, n, 0.05, 0.9, 5e-4, mod, 32)
    w0 = G.normal_like(G.stream_key(seed, G.STREAM_WEIGHTS), 0, num_params, 0.01) if num_params else torch.zeros(0)
    ref.set_weights(w0.numpy())
    ps = P.ParameterServer(num_params, lam, n, 0.05, 0.9, 5e-4, "inv_staleness" if seed % 3 else "constant",
                           device=device, allocate=num_params > 0)
    if num_params:
        ps.init_weights(w0.to(device))
    h = ps._h
    queue_cap = 6
    ps.set_option(P.PS_OPT_QUEUE_GROUPS, queue_cap)
    pulled = {l: None for l in range(lam)}
    counts = {l: 0 for l in range(lam)}
    rate = 0.05
    c = lam // n
    for step in range(steps):
        op = rng.choice(["pull", "push", "push", "push", "apply", "fuse", "rate", "flush", "pullw"],
                        p=[0.2, 0.2, 0.2, 0.15, 0.1, 0.04, 0.04, 0.03, 0.04])
        applied, logical = ps.timestamps()
        if op == "pull" or (op == "push" and all(v is None for v in pulled.values())):
            l = int(rng.integers(lam))
            ts = ps.pull_weights()
            assert ts == ref.pull(l) == logical
            pulled[l] = ts
        elif op == "push":
            l = int(rng.choice([k for k, v in pulled.items() if v is not None]))
            if logical - applied >= queue_cap:                       # the queue refuses; nothing changes
                assert P.ps_push_gradient(h, l, FAKE, pulled[l]) == P.PS_ERR_QUEUE_FULL
                assert ps.flush() == queue_cap
            if num_params:
                g = G.gradient(seed, l, counts[l], num_params, 1e-2, device=device)
                fired = ps.push_gradient(l, g, pulled[l])
                ref_fired = ref.push(l, g.cpu().numpy(), timestamp=pulled[l])
            else:
                r = P.ps_push_gradient(h, l, FAKE, pulled[l])
                assert r in (P.PS_OK, P.PS_READY)
                fired = r == P.PS_READY
                ref_fired = ref.push(l, np.zeros(0, np.float32), timestamp=pulled[l])
                ps._held.append(None)
            counts[l] += 1
            assert fired == ref_fired
        elif op == "apply":
            if logical > applied:
                assert ps.apply_update() == min(ps.get_option(P.PS_OPT_FUSE_T), logical - applied)
            else:
                assert P.ps_apply_update(h) == P.PS_ERR_NOT_READY
        elif op == "fuse":
            ps.set_option(P.PS_OPT_FUSE_T, int(rng.integers(1, 9)))
        elif op == "rate":
            rate = float(np.float32(rate * 0.5 if rate > 1e-4 else 0.05))
            ps.set_alpha0(rate)
            ref.set_alpha0(rate)
        elif op == "flush":
            assert ps.flush() == logical - applied
        elif op == "pullw" and num_params:
            out = torch.empty(num_params, device=device)
            assert ps.pull_weights(out) == ref.timestamp                 # flushes first
            assert np.array_equal(out.cpu().numpy(), ref.state()[0].astype(np.float32))
        assert ps.timestamps()[1] == ref.timestamp
    ps.flush()
    log, rlog = ps.update_log(), ref.log()
    assert np.array_equal(ps.staleness_histogram(), np.bincount(rlog["tau"])) if len(rlog) else True
    for f in ("update", "push_index", "ts_grad", "tau", "sigma", "learner", "position"):
        assert np.array_equal(log[f], rlog[f]), f
    assert np.array_equal(log["scale"], rlog["scale"].astype(np.float32))
    assert np.array_equal(log["decay"], rlog["decay"].astype(np.float32))
    if num_params:
        ps.synchronize()
        w, v = ref.state()
        assert np.array_equal(ps.w.cpu().numpy(), w.astype(np.float32))
        assert np.array_equal(ps.v.cpu().numpy(), v.astype(np.float32))
    ps.destroy()
    return len(log)


@pytest.mark.parametrize("seed,lam,n", [(1, 4, 1), (2, 6, 2), (3, 5, 5), (4, 7, 3), (5, 16, 4), (6, 3, 1), (7, 9, 9), (8, 1, 1)])
def test_random_schedules_without_a_gpu(seed, lam, n):
    assert drive(seed, lam, n) > 0


@pytest.mark.gpu
@pytest.mark.parametrize("seed,lam,n,num_params", [(11, 4, 2, 1003), (12, 6, 1, 4099), (13, 5, 5, 257), (14, 8, 2, 70001)])
def test_random_schedules_with_weights(seed, lam, n, num_params):
    assert drive(seed, lam, n, num_params, torch.device("cuda", 0), steps=250) > 0
