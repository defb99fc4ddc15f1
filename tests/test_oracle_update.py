"""Pins for the reference's update arithmetic (everything here runs on the CPU).

Each test compares the reference with something that is fixed outside it:
hand-worked numbers (tests/golden), a library optimiser, a closed form, or a
special case in which the method collapses to a textbook rule.
"""
import json
import os

import numpy as np
import pytest
import torch

from oracle import reference as R
from tests.helpers import replay_reference, staleness_by_recount, rel_l2
from workloads import generators as G

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_softsync.json")
MODS = {"inv_staleness": R.MOD_INV_STALENESS, "constant": R.MOD_CONSTANT, "exp_staleness": R.MOD_EXP_STALENESS}


def _grads(seed, lam, pushes_per_learner, n, std=1e-3, dtype=torch.float32):
    return {(l, p): G.gradient(seed, l, p, n, std, dtype=dtype) for l in range(lam) for p in range(pushes_per_learner)}


# ---------------------------------------------------------------- hand-worked examples
@pytest.mark.parametrize("precision", [32, 64])
@pytest.mark.parametrize("example", json.load(open(GOLDEN))["examples"], ids=lambda e: e["name"])
def test_hand_worked_examples_exact(example, precision):
    ex = example
    ps = R.ReferencePS(len(ex["w0"]), ex["num_learners"], ex["n"], ex["alpha0"], ex["momentum"],
                       ex["weight_decay"], MODS[ex["modulation"]], precision)
    ps.set_weights(np.asarray(ex["w0"], np.float32))
    if "penalty_base" in ex:
        ps.set_penalty_base(ex["penalty_base"])
    if "layers" in ex:
        ps.set_layer_multipliers(ex["layers"]["bounds"], ex["layers"]["lr_mult"], ex["layers"]["wd_mult"])
    done = 0
    for ev in ex["events"]:
        if ev[0] == "pull":
            ps.pull(ev[1])
            continue
        if ev[0] == "alpha0":
            ps.set_alpha0(ev[1])
            continue
        fired = ps.push(ev[1], np.asarray(ev[2], np.float32))
        if fired:
            exp = ex["updates"][done]
            done += 1
            w, v = ps.state()
            assert w.tolist() == exp["w"] and v.tolist() == exp["v"]
            assert ps.timestamp == exp["ts"]
            rows = ps.log()[-len(exp["members"]):]
            got = [[int(r["learner"]), int(r["push_index"]), int(r["ts_grad"]), int(r["tau"]),
                    int(r["sigma"]), float(r["scale"])] for r in rows]
            assert got == exp["members"]
            assert all(float(r["decay"]) == exp["decay"] for r in rows)
    assert done == len(ex["updates"])


# ---------------------------------------------------------------- collapses to textbook rules
def test_single_learner_is_sequential_momentum_sgd_bit_for_bit():
    """lambda = 1, n = 1: every gradient has tau = 0 and the method is plain momentum SGD."""
    n, steps = 257, 40
    a, m, wd = np.float32(0.01), np.float32(0.9), np.float32(5e-4)
    w0 = G.normal_like(G.stream_key(1, G.STREAM_WEIGHTS), 0, n, 0.01).numpy()
    ps = R.ReferencePS(n, 1, 1, float(a), float(m), float(wd), R.MOD_INV_STALENESS, 32)
    ps.set_weights(w0)
    w, v = w0.copy(), np.zeros(n, np.float32)
    awd = np.float32(np.float64(wd) * np.float64(a))
    for p in range(steps):
        g = G.gradient(1, 0, p, n, 1e-3).numpy()
        ps.pull(0)
        assert ps.push(0, g)
        v = m * v + (a * g + awd * w)          # textbook: v <- m v + lr (g + wd w); w <- w - v
        w = w - v
    wr, vr = ps.state()
    assert np.array_equal(wr.astype(np.float32), w) and np.array_equal(vr.astype(np.float32), v)
    assert ps.timestamp == steps
    assert (ps.log()["sigma"] == 1).all()


def test_single_learner_matches_library_sgd_optimizer():
    """Same special case against torch.optim.SGD (lr outside the velocity: v_here = lr * buf)."""
    n, steps = 64, 60
    lr, m, wd = 0.01, 0.9, 5e-4
    w0 = G.normal_like(G.stream_key(2, G.STREAM_WEIGHTS), 0, n, 0.01)
    ps = R.ReferencePS(n, 1, 1, lr, m, wd, R.MOD_INV_STALENESS, 64)
    ps.set_weights(w0.numpy())
    p = torch.nn.Parameter(w0.double().clone())
    f32 = lambda x: float(np.float32(x))
    opt = torch.optim.SGD([p], lr=f32(lr), momentum=f32(m), weight_decay=f32(wd))
    for s in range(steps):
        g = G.gradient(2, 0, s, n, 1e-3)
        ps.pull(0)
        ps.push(0, g.numpy())
        p.grad = g.double()
        opt.step()
    w, v = ps.state()
    assert rel_l2(w, p.detach().numpy()) < 1e-13
    buf = opt.state[p]["momentum_buffer"].numpy()
    assert rel_l2(v, f32(lr) * buf) < 1e-12


@pytest.mark.parametrize("lam", [2, 4, 5])
def test_one_softsync_with_barrier_is_synchronous_averaged_sgd(lam):
    """n = 1 and everybody pulls after the update: tau = 0, Eq. 2 becomes Eq. 1 (hardsync),
    i.e. SGD on the mean of the lambda gradients; with momentum and decay that is library SGD."""
    n, rounds = 48, 25
    lr, m, wd = 0.05, 0.9, 5e-4
    w0 = G.normal_like(G.stream_key(3, G.STREAM_WEIGHTS), 0, n, 0.01)
    f32 = lambda x: float(np.float32(x))
    for momentum, decay in ((0.0, 0.0), (m, wd)):
        ps = R.ReferencePS(n, lam, 1, lr, momentum, decay, R.MOD_INV_STALENESS, 64)
        ps.set_weights(w0.numpy())
        p = torch.nn.Parameter(w0.double().clone())
        opt = torch.optim.SGD([p], lr=f32(lr), momentum=f32(momentum), weight_decay=f32(decay))
        plain = w0.double().numpy().copy()
        for r in range(rounds):
            for l in range(lam):
                ps.pull(l)
            gs = [G.gradient(3, l, r, n, 1e-3).double() for l in range(lam)]
            order = np.random.default_rng(r).permutation(lam)
            for l in order:
                fired = ps.push(int(l), gs[l].float().numpy())
            assert fired
            p.grad = torch.stack(gs).mean(0)
            opt.step()
            plain = plain - f32(lr) * np.mean(np.stack([g.numpy() for g in gs]), axis=0)   # Eq. 1
        w, _ = ps.state()
        assert (ps.log()["tau"] == 0).all()
        assert rel_l2(w, p.detach().numpy()) < 1e-12
        if momentum == 0.0 and decay == 0.0:
            assert rel_l2(w, plain) < 1e-12
    # the fp32 reference agrees with the fp64 one to fp32 rounding
    ps32 = R.ReferencePS(n, lam, 1, lr, m, wd, R.MOD_INV_STALENESS, 32)
    ps32.set_weights(w0.numpy())
    for r in range(rounds):
        for l in range(lam):
            ps32.pull(l)
        for l in range(lam):
            ps32.push(l, G.gradient(3, l, r, n, 1e-3).numpy())
    assert rel_l2(ps32.state()[0], p.detach().numpy()) < 1e-6


def test_hardsync_protocol_is_eq_1_and_enforces_the_barrier():
    """Section 2.2 hardsync: theta <- theta - alpha * mean of one gradient per learner, staleness 0, and
    nobody contributes twice or with old weights."""
    lam, n_el, rounds = 5, 24, 12
    a0 = float(np.float32(0.1))
    w0 = G.normal_like(G.stream_key(15, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    ps = R.ReferencePS(n_el, lam, 1, a0, 0.0, 0.0, R.MOD_INV_STALENESS, 64)
    ps.set_weights(w0)
    ps.set_hardsync()
    w = w0.astype(np.float64)
    for r in range(rounds):
        for l in range(lam):
            assert ps.pull(l) == r
        gs = [G.gradient(15, l, r, n_el, 1e-2).numpy() for l in range(lam)]
        order = np.random.default_rng(r).permutation(lam)
        for i, l in enumerate(order):
            fired = ps.push(int(l), gs[l])
            assert fired == (i == lam - 1)
            if i == 0:
                with pytest.raises(ValueError):
                    ps.push(int(l), gs[l])                    # a second gradient in the same round
        w = w - a0 * np.mean(np.stack(gs).astype(np.float64), axis=0)         # Eq. 1
    assert rel_l2(ps.state()[0], w) < 1e-13
    assert (ps.log()["tau"] == 0).all() and ps.timestamp == rounds
    # a learner that did not pull the new weights is refused (its staleness would be 1)
    for l in range(lam - 1):
        ps.pull(l)
    with pytest.raises(ValueError):
        ps.push(lam - 1, gs[0])
    with pytest.raises(ValueError):
        R.ReferencePS(4, 4, 2, 0.1, 0.0, 0.0).set_hardsync()  # needs n = 1


def test_downpour_case_is_per_push_sgd():
    """n = lambda with a constant rate is Downpour SGD: theta <- theta - alpha0 * dtheta per push."""
    lam, n_el, pushes = 6, 32, 120
    a0 = float(np.float32(0.02))
    k, l = R.simulate_arrivals("exp", lam, pushes, 9)
    ps = R.ReferencePS(n_el, lam, lam, a0, 0.0, 0.0, R.MOD_CONSTANT, 64)
    w0 = G.normal_like(G.stream_key(4, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    ps.set_weights(w0)
    total = np.zeros(n_el)
    def grad(a, b):
        g = G.gradient(4, a, b, n_el, 1e-3).numpy()
        total[:] += g.astype(np.float64)
        return g
    replay_reference(ps, k, l, grad)
    assert ps.timestamp == pushes
    assert rel_l2(ps.state()[0], w0.astype(np.float64) - a0 * total) < 1e-13


def test_step_schedule_without_momentum_is_library_sgd_with_a_changing_rate():
    """Section 4.3 lowers alpha0 in steps.  With one learner and no momentum the method is SGD whose
    learning rate follows the schedule (library optimiser + StepLR)."""
    n, steps = 32, 30
    w0 = G.normal_like(G.stream_key(12, G.STREAM_WEIGHTS), 0, n, 0.01)
    f32 = lambda x: float(np.float32(x))
    lr0, wd = f32(0.1), f32(5e-4)
    ps = R.ReferencePS(n, 1, 1, lr0, 0.0, wd, R.MOD_INV_STALENESS, 64)
    ps.set_weights(w0.numpy())
    p = torch.nn.Parameter(w0.double().clone())
    opt = torch.optim.SGD([p], lr=lr0, momentum=0.0, weight_decay=wd)
    sched = torch.optim.lr_scheduler.StepLR(opt, step_size=10, gamma=0.5)     # exact in binary
    for s in range(steps):
        ps.set_alpha0(opt.param_groups[0]["lr"])
        g = G.gradient(12, 0, s, n, 1e-2)
        ps.pull(0)
        ps.push(0, g.numpy())
        p.grad = g.double()
        opt.step()
        sched.step()
    assert opt.param_groups[0]["lr"] == lr0 / 8
    assert rel_l2(ps.state()[0], p.detach().numpy()) < 1e-13


def test_rate_in_force_at_arrival_enters_the_geometric_sum():
    """With momentum the step of update i is u_i = sum_l alpha0(at arrival of l)/(c sigma_l) g_l and
    v_K = sum_i m^(K-1-i) u_i, whatever alpha0 is later."""
    lam, n, n_el, pushes = 4, 2, 8, 40
    c = lam // n
    m = float(np.float32(0.5))
    k, l = R.simulate_arrivals("exp", lam, pushes, 3)
    tau, _ = staleness_by_recount(k, l, c)
    ps = R.ReferencePS(n_el, lam, n, 0.25, m, 0.0, R.MOD_INV_STALENESS, 64)
    ps.set_weights(np.zeros(n_el, np.float32))
    seen, rates, counts = [], [], {}
    rate = 0.25
    for kind, who in zip(k.tolist(), l.tolist()):
        if kind == 0:
            ps.pull(who)
            continue
        if len(seen) % 7 == 3:
            rate = rate / 2
            ps.set_alpha0(rate)
        b = counts.get(who, 0); counts[who] = b + 1
        g = G.gradient(13, who, b, n_el, 1e-2).numpy()
        seen.append(g.astype(np.float64)); rates.append(rate)
        ps.push(who, g)
    K = pushes // c
    scaled = (np.asarray(rates[:K * c]) / (c * np.maximum(tau[:K * c], 1)))[:, None] * np.stack(seen[:K * c])
    u = scaled.reshape(K, c, n_el).sum(1)
    i = np.arange(K)
    w, v = ps.state()
    assert rel_l2(v, ((m ** (K - 1 - i))[:, None] * u).sum(0)) < 1e-12
    assert rel_l2(w, -(((1 - m ** (K - i)) / (1 - m))[:, None] * u).sum(0)) < 1e-12


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("model,lam,n", [("exp", 8, 8), ("exp", 12, 3), ("uniform", 18, 4), ("lognormal", 10, 5)])
def test_plain_rule_is_a_weighted_sum_of_gradients(model, lam, n):
    """m = 0, wd = 0: theta_K = theta_0 - sum over pushes of alpha0/(c max(tau,1)) * dtheta
    (Eq. 2 summed over updates, Eq. 3), with tau recounted from the raw trace."""
    n_el, pushes = 40, 240
    c = lam // n
    a0 = float(np.float32(0.03))
    k, l = R.simulate_arrivals(model, lam, pushes, 17)
    tau, _ = staleness_by_recount(k, l, c)
    ps = R.ReferencePS(n_el, lam, n, a0, 0.0, 0.0, R.MOD_INV_STALENESS, 64)
    w0 = G.normal_like(G.stream_key(5, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    ps.set_weights(w0)
    seen = []
    def grad(a, b):
        g = G.gradient(5, a, b, n_el, 1e-3).numpy()
        seen.append(g.astype(np.float64))
        return g
    replay_reference(ps, k, l, grad)
    used = (pushes // c) * c
    weights = a0 / (c * np.maximum(tau[:used], 1))
    expect = w0.astype(np.float64) - np.einsum("p,pk->k", weights, np.stack(seen[:used]))
    assert rel_l2(ps.state()[0], expect) < 1e-13
    assert tau.max() >= 2       # the case really exercises staleness


@pytest.mark.parametrize("rho", [0.5, 0.8, 1.0])
def test_exponential_penalty_is_a_weighted_sum_with_geometric_weights(rho):
    """m = 0, wd = 0 under the exponential penalty: theta_K = theta_0 - sum over pushes of
    alpha0 * rho^tau / c * dtheta, with tau recounted from the raw trace; rho = 1 is the constant rate."""
    lam, n, n_el, pushes = 12, 3, 40, 240
    c = lam // n
    a0, rho = float(np.float32(0.03)), float(np.float32(rho))
    k, l = R.simulate_arrivals("exp", lam, pushes, 19)
    tau, _ = staleness_by_recount(k, l, c)
    ps = R.ReferencePS(n_el, lam, n, a0, 0.0, 0.0, R.MOD_EXP_STALENESS, 64)
    ps.set_penalty_base(rho)
    w0 = G.normal_like(G.stream_key(5, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    ps.set_weights(w0)
    seen = []
    def grad(a, b):
        g = G.gradient(5, a, b, n_el, 1e-3).numpy()
        seen.append(g.astype(np.float64))
        return g
    replay_reference(ps, k, l, grad)
    used = (pushes // c) * c
    weights = a0 * np.exp(np.log(rho) * tau[:used]) / c
    expect = w0.astype(np.float64) - np.einsum("p,pk->k", weights, np.stack(seen[:used]))
    assert rel_l2(ps.state()[0], expect) < 1e-12
    assert tau.max() >= 3
    log = ps.log()
    assert np.array_equal(log["sigma"], log["tau"])
    if rho == 1.0:                                     # no penalty at all: the constant-rate control of Section 4.3
        const = R.ReferencePS(n_el, lam, n, a0, 0.0, 0.0, R.MOD_CONSTANT, 64)
        const.set_weights(w0)
        replay_reference(const, k, l, lambda a, b: G.gradient(5, a, b, n_el, 1e-3).numpy())
        assert np.array_equal(const.state()[0], ps.state()[0])
    with pytest.raises(ValueError):
        ps.set_penalty_base(0.0)
    with pytest.raises(ValueError):
        ps.set_penalty_base(1.5)


def test_exponential_penalty_shrinks_faster_than_inverse_staleness():
    """Section 1's objection to the exponential rule: at the staleness a large system sees, it leaves almost
    no step at all, whereas alpha0/tau decays only harmonically.  One gradient with tau = 40."""
    out = {}
    for mod in (R.MOD_INV_STALENESS, R.MOD_EXP_STALENESS):
        ps = R.ReferencePS(1, 2, 2, 1.0, 0.0, 0.0, mod, 64)
        ps.set_weights(np.zeros(1, np.float32))
        ps.pull(0); ps.pull(1)
        for _ in range(40):
            ps.pull(0)
            ps.push(0, np.zeros(1, np.float32))
        ps.push(1, np.ones(1, np.float32))            # pulled at clock 0, arrives at clock 40
        out[mod] = -ps.state()[0][0]
        assert ps.log()["tau"][-1] == 40
    assert out[R.MOD_INV_STALENESS] == 1.0 / 40
    assert out[R.MOD_EXP_STALENESS] == 0.5 ** 40


def test_exponential_penalty_runs_out_through_the_denormals_to_zero():
    """rho = 0.5 makes every scale an exact power of two, so the fp32 scale table is known in closed form all the
    way down: 2^-tau while that is a normal or denormal fp32 number (tau <= 149), exactly zero beyond.  The
    momentum right after such an update (m = 0, wd = 0, theta_0 = 0) is the bare product scale * g, a denormal
    that must be kept, not flushed."""
    ps = R.ReferencePS(4, 2, 2, 1.0, 0.0, 0.0, R.MOD_EXP_STALENESS, 32)
    ps.set_weights(np.zeros(4, np.float32))
    ps.pull(0); ps.pull(1)
    g = np.array([1.0, -3.0, 0.5, 2.0 ** -3], np.float32)
    seen = {}
    for clock in range(160):
        if clock in (100, 126, 127, 140, 149, 150, 155):
            ps.push(1, g)                                   # learner 1 never pulls again: tau = clock
            tau = int(ps.log()["tau"][-1])
            seen[tau] = (float(ps.log()["scale"][-1]), ps.state()[1].astype(np.float32).copy())
        ps.pull(0)
        ps.push(0, np.zeros(4, np.float32))
    assert sorted(seen) == [100, 127, 129, 143, 153, 155, 161]          # each stale push moved the clock on by one too
    tiny = float(np.finfo(np.float32).tiny)                              # 2^-126
    for tau, (scale, v) in seen.items():
        want = np.float32(2.0 ** -tau) if tau <= 149 else np.float32(0.0)
        assert scale == float(want) and (tau < 126 or scale < tiny)
        assert np.array_equal(v, (np.float64(want) * g.astype(np.float64)).astype(np.float32))   # exact: powers of two
    assert seen[143][1][0] > 0 and seen[143][1][3] > 0 and seen[153][0] == 0.0                   # denormal kept, then zero


def _caffe_like_layers(n_el):
    b = [0, n_el // 3, n_el // 3 + 5, n_el - 7, n_el]
    return b, [1.0, 2.0, 0.5, 2.0], [1.0, 0.0, 3.0, 0.0]


def test_layer_multipliers_are_per_layer_rates_and_decays_of_library_sgd():
    """One learner: the method with multipliers (lm_q, dm_q) is library momentum SGD with one parameter
    group per layer, lr = alpha0*lm_q and weight_decay = wd*dm_q (velocity here = lr * the library's buffer)."""
    n_el, steps = 60, 50
    f32 = lambda x: float(np.float32(x))
    lr, m, wd = f32(0.01), f32(0.9), f32(5e-3)
    bounds, lmul, dmul = _caffe_like_layers(n_el)
    w0 = G.normal_like(G.stream_key(21, G.STREAM_WEIGHTS), 0, n_el, 0.1)
    ps = R.ReferencePS(n_el, 1, 1, lr, m, wd, R.MOD_INV_STALENESS, 64)
    ps.set_weights(w0.numpy())
    ps.set_layer_multipliers(bounds, lmul, dmul)
    params = [torch.nn.Parameter(w0[a:b].double().clone()) for a, b in zip(bounds[:-1], bounds[1:])]
    opt = torch.optim.SGD([{"params": [p], "lr": lr * a, "weight_decay": wd * d} for p, a, d in zip(params, lmul, dmul)],
                          lr=lr, momentum=m)
    for s in range(steps):
        g = G.gradient(21, 0, s, n_el, 1e-2)
        ps.pull(0)
        ps.push(0, g.numpy())
        for p, a, b in zip(params, bounds[:-1], bounds[1:]):
            p.grad = g[a:b].double()
        opt.step()
    w, v = ps.state()
    assert rel_l2(w, torch.cat([p.detach() for p in params]).numpy()) < 1e-12
    buf = torch.cat([opt.state[p]["momentum_buffer"] * (lr * a) for p, a in zip(params, lmul)]).numpy()
    assert rel_l2(v, buf) < 1e-11


def test_layer_multipliers_of_one_change_nothing_and_zero_rate_freezes_a_layer():
    """Multiplying by 1.0f is exact, so all-ones multipliers give the same bits as none (fp32, real staleness);
    a layer with rate multiplier 0 never moves."""
    lam, n, n_el, pushes = 6, 2, 101, 60
    k, l = R.simulate_arrivals("lognormal", lam, pushes, 4)
    w0 = G.normal_like(G.stream_key(22, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    grad = lambda a, b: G.gradient(22, a, b, n_el, 1e-3).numpy()
    out = []
    for layers in (None, ([0, 40, n_el], [1.0, 1.0], [1.0, 1.0]), ([0, 40, n_el], [1.0, 0.0], [1.0, 1.0])):
        ps = R.ReferencePS(n_el, lam, n, 0.03, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
        ps.set_weights(w0)
        if layers:
            ps.set_layer_multipliers(*layers)
        replay_reference(ps, k, l, grad)
        out.append(ps.state())
    assert np.array_equal(out[0][0], out[1][0]) and np.array_equal(out[0][1], out[1][1])
    assert np.array_equal(out[2][0][:40], out[0][0][:40])
    assert np.array_equal(out[2][0][40:].astype(np.float32), w0[40:]) and not out[2][1][40:].any()
    with pytest.raises(ValueError):
        R.ReferencePS(10, 1, 1, 0.1, 0.0, 0.0).set_layer_multipliers([0, 4, 9], [1, 1], [1, 1])   # does not reach N


def test_layer_multipliers_fp32_rounding_order():
    """t = lm * (acc + (dm * d) * w): every product and sum rounded once, written out in numpy float32."""
    lam, n, n_el, pushes = 4, 2, 67, 24
    c = lam // n
    f = np.float32
    a0, m, wd = f(0.03), f(0.9), f(5e-3)
    bounds, lmul, dmul = _caffe_like_layers(n_el)
    lm = np.repeat(np.asarray(lmul, f), np.diff(bounds)); dm = np.repeat(np.asarray(dmul, f), np.diff(bounds))
    k, l = R.simulate_arrivals("exp", lam, pushes, 45)
    tau, _ = staleness_by_recount(k, l, c)
    w0 = G.normal_like(G.stream_key(45, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    ps = R.ReferencePS(n_el, lam, n, float(a0), float(m), float(wd), R.MOD_INV_STALENESS, 32)
    ps.set_weights(w0)
    ps.set_layer_multipliers(bounds, lmul, dmul)
    arr = []
    def grad(a, b):
        g = G.gradient(45, a, b, n_el, 1e-3).numpy()
        arr.append((a, b, g))
        return g
    replay_reference(ps, k, l, grad)
    w, v = w0.copy(), np.zeros(n_el, f)
    for i in range(pushes // c):
        group = sorted(((a, b, g, max(int(tau[i * c + j]), 1)) for j, (a, b, g) in enumerate(arr[i * c:(i + 1) * c])),
                       key=lambda x: (x[0], x[1]))
        s = [f(np.float64(a0) / (np.float64(c) * np.float64(sig))) for _, _, _, sig in group]
        d = f(np.float64(wd) * sum(np.float64(x) for x in s))
        acc = s[0] * group[0][2]
        for j in range(1, c):
            acc = acc + s[j] * group[j][2]
        t = lm * (acc + (dm * d) * w)
        v = m * v + t
        w = w - v
    wr, vr = ps.state()
    assert np.array_equal(wr.astype(f), w) and np.array_equal(vr.astype(f), v)


def test_momentum_is_a_geometric_sum_of_past_steps():
    """wd = 0: v_K = sum_i m^(K-1-i) u_i and theta_K = theta_0 - sum_i u_i (1 - m^(K-i))/(1 - m),
    where u_i is the Eq. 2 step of update i."""
    lam, n, n_el, pushes = 6, 2, 16, 90
    c = lam // n
    a0, m = float(np.float32(0.02)), float(np.float32(0.9))
    k, l = R.simulate_arrivals("exp", lam, pushes, 23)
    tau, _ = staleness_by_recount(k, l, c)
    ps = R.ReferencePS(n_el, lam, n, a0, m, 0.0, R.MOD_INV_STALENESS, 64)
    w0 = np.zeros(n_el, np.float32)
    ps.set_weights(w0)
    seen = []
    def grad(a, b):
        g = G.gradient(6, a, b, n_el, 1e-3).numpy()
        seen.append(g.astype(np.float64))
        return g
    replay_reference(ps, k, l, grad)
    K = pushes // c
    scaled = (a0 / (c * np.maximum(tau[:K * c], 1)))[:, None] * np.stack(seen[:K * c])
    u = scaled.reshape(K, c, n_el).sum(1)
    i = np.arange(K)
    v_expect = ((m ** (K - 1 - i))[:, None] * u).sum(0)
    w_expect = -(((1 - m ** (K - i)) / (1 - m))[:, None] * u).sum(0)
    w, v = ps.state()
    assert rel_l2(v, v_expect) < 1e-12 and rel_l2(w, w_expect) < 1e-12


def test_decay_and_momentum_follow_the_linear_recurrence_in_matrix_form():
    """Per element the update is x <- A_i x + b_i with x = (w, v),
    A_i = [[1 - d_i, -m], [d_i, m]], b_i = (-u_i, u_i), d_i = wd * sum_l s_l.
    Checked with an accumulated matrix product instead of stepping the scalars."""
    lam, n, pushes = 9, 3, 150
    c = lam // n
    a0, m, wd = float(np.float32(0.05)), float(np.float32(0.8)), float(np.float32(0.01))
    k, l = R.simulate_arrivals("lognormal", lam, pushes, 31)
    tau, _ = staleness_by_recount(k, l, c)
    ps = R.ReferencePS(1, lam, n, a0, m, wd, R.MOD_INV_STALENESS, 64)
    w0 = np.array([0.5], np.float32)
    ps.set_weights(w0)
    seen = []
    def grad(a, b):
        g = G.gradient(7, a, b, 1, 1e-2).numpy()
        seen.append(float(g[0]))
        return g
    replay_reference(ps, k, l, grad)
    K = pushes // c
    s = (a0 / (c * np.maximum(tau[:K * c], 1))).reshape(K, c)
    u = (s * np.asarray(seen[:K * c]).reshape(K, c)).sum(1)
    d = wd * s.sum(1)
    # homogeneous coordinates: one 3x3 affine map per update, multiplied up
    M = np.eye(3)
    for i in range(K):
        step = np.array([[1 - d[i], -m, -u[i]], [d[i], m, u[i]], [0, 0, 1]])
        M = step @ M
    x = M @ np.array([0.5, 0.0, 1.0])
    w, v = ps.state()
    assert abs(w[0] - x[0]) < 1e-12 * max(1, abs(x[0])) and abs(v[0] - x[1]) < 1e-12
    assert tau.max() >= 3


def test_fp32_rounding_order_is_the_documented_one():
    """The fp32 state is rounded after every multiply and every add, in this order: products s_l*g_l summed
    left to right in (learner, push) order; t = acc + d*w; v = m*v + t; w = w - v.  Written out with numpy
    float32 scalars-as-arrays (each numpy op rounds once) and compared bit for bit on random data."""
    lam, n, n_el, pushes = 6, 2, 301, 60
    c = lam // n
    f = np.float32
    a0, m, wd = f(0.03), f(0.9), f(5e-4)
    k, l = R.simulate_arrivals("lognormal", lam, pushes, 44)
    tau, _ = staleness_by_recount(k, l, c)
    w0 = G.normal_like(G.stream_key(44, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    ps = R.ReferencePS(n_el, lam, n, float(a0), float(m), float(wd), R.MOD_INV_STALENESS, 32)
    ps.set_weights(w0)
    arrivals_ = []
    def grad(a, b):
        g = G.gradient(44, a, b, n_el, 1e-3).numpy()
        arrivals_.append((a, b, g))
        return g
    replay_reference(ps, k, l, grad)
    w, v = w0.copy(), np.zeros(n_el, f)
    for i in range(pushes // c):
        group = sorted(((a, b, g, max(int(tau[i * c + j]), 1)) for j, (a, b, g) in enumerate(arrivals_[i * c:(i + 1) * c])),
                       key=lambda x: (x[0], x[1]))
        s = [f(np.float64(a0) / (np.float64(c) * np.float64(sig))) for _, _, _, sig in group]
        d = f(np.float64(wd) * sum(np.float64(x) for x in s))
        acc = s[0] * group[0][2]
        for j in range(1, c):
            acc = acc + s[j] * group[j][2]
        t = acc + d * w
        v = m * v + t
        w = w - v
    wr, vr = ps.state()
    assert np.array_equal(wr.astype(f), w) and np.array_equal(vr.astype(f), v)
    assert tau.max() >= 2


# ---------------------------------------------------------------- invariants of the readings
def test_arrival_order_inside_a_group_does_not_change_the_bits():
    lam, n_el = 5, 33
    w0 = G.normal_like(G.stream_key(8, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    results = []
    for perm_seed in range(4):
        ps = R.ReferencePS(n_el, lam, 1, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
        ps.set_weights(w0)
        for r in range(6):
            for l in range(lam):
                ps.pull(l)
            for l in np.random.default_rng(perm_seed * 100 + r).permutation(lam):
                ps.push(int(l), G.gradient(8, int(l), r, n_el, 1e-3).numpy())
        results.append(ps.state())
    for w, v in results[1:]:
        assert np.array_equal(w, results[0][0]) and np.array_equal(v, results[0][1])


def test_bf16_gradients_are_widened_exactly():
    n_el, lam = 64, 3
    w0 = G.normal_like(G.stream_key(9, G.STREAM_WEIGHTS), 0, n_el, 0.01).numpy()
    a = R.ReferencePS(n_el, lam, 3, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    b = R.ReferencePS(n_el, lam, 3, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    a.set_weights(w0); b.set_weights(w0)
    for l in range(lam):
        a.pull(l); b.pull(l)
    for p in range(5):
        for l in range(lam):
            g = G.gradient(9, l, p, n_el, 1e-4, dtype=torch.bfloat16)
            a.push(l, g.view(torch.int16).numpy().view(np.uint16))
            b.push(l, g.float().numpy())
    assert np.array_equal(a.state()[0], b.state()[0]) and np.array_equal(a.state()[1], b.state()[1])
    assert a.timestamp == 15


def test_bf16_rounding_matches_library_conversion_and_hand_cases():
    """Round-to-nearest-even fp32 -> bf16: against torch's conversion on random and special values,
    and against tie cases worked by hand (bf16 keeps 8 significand bits)."""
    rng = np.random.default_rng(0)
    bits = rng.integers(0, 1 << 32, size=200000, dtype=np.uint64).astype(np.uint32)
    x = bits.view(np.float32)
    x = x[np.isfinite(x)]
    special = np.array([0.0, -0.0, np.inf, -np.inf, 1.0, -1.0, 3.3895314e38, 3.4028235e38, 1e-40, -1e-45,
                        1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 2.0 ** -9], np.float32)
    x = np.concatenate([x, special])
    got = R.round_to_bf16(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)
    # hand cases: 1 + 2^-8 is exactly half-way between 1 (0x3F80) and 1 + 2^-7 (0x3F81): ties go to the even 0x3F80;
    # 1 + 3*2^-8 is half-way between 0x3F81 and 0x3F82: goes to the even 0x3F82; just above half-way goes up;
    # the largest fp32 rounds to +inf (0x7F80).
    hand = R.round_to_bf16(np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20,
                                     1.0 + 2.0 ** -9, 3.4028235e38], np.float32))
    assert hand.tolist() == [0x3F80, 0x3F82, 0x3F81, 0x3F80, 0x7F80]
    assert R.round_to_bf16(np.array([np.nan], np.float32)).tolist() == [0x7FFF]


def test_bf16_weights_are_the_rounded_fp32_state():
    ps = R.ReferencePS(5, 1, 1, 0.5, 0.0, 0.0, R.MOD_INV_STALENESS, 32)
    ps.set_weights(np.array([1.0, 2.0, 3.0, 4.0, 5.0], np.float32))
    ps.pull(0)
    ps.push(0, np.array([2.0 ** -8, 0.0, 3 * 2.0 ** -7, -1.0, 2.0 ** -6], np.float32) * -2)   # w += exact dyadics
    w, _ = ps.state()
    assert w.tolist() == [1.0 + 2.0 ** -8, 2.0, 3.0 + 3 * 2.0 ** -7, 3.0, 5.0 + 2.0 ** -6]
    # 3 + 3*2^-7 = 1.5*(2 + 2^-6): the dropped bits are exactly half an ulp (2^-6 at this exponent) with an odd
    # kept part: rounds up to 3 + 2^-5 (0x4042); 5 + 2^-6 is half-way between 5 (0x40A0) and 5 + 2^-5: stays even
    assert ps.weights_bf16().tolist() == [0x3F80, 0x4000, 0x4042, 0x4040, 0x40A0]
    with pytest.raises(ValueError):
        R.ReferencePS(2, 1, 1, 0.1, 0.0, 0.0, R.MOD_INV_STALENESS, 64).weights_bf16()


def test_fp32_reference_tracks_fp64_reference():
    """Noise floor of keeping the state in fp32, on the small benchmark shape."""
    from workloads import configs
    cfg = configs.TINY_SOFTSYNC
    n_el = 4096
    k, l = R.simulate_arrivals(cfg.arrival_model, cfg.num_learners, 400, 1)
    w0 = G.normal_like(G.stream_key(10, G.STREAM_WEIGHTS), 0, n_el, cfg.weight_std).numpy()
    out = []
    for prec in (32, 64):
        ps = R.ReferencePS(n_el, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                           R.MOD_INV_STALENESS, prec)
        ps.set_weights(w0)
        replay_reference(ps, k, l, lambda a, b: G.gradient(10, a, b, n_el, cfg.grad_std).numpy())
        out.append(ps.state())
    assert rel_l2(out[0][0], out[1][0]) < 1e-6
    assert rel_l2(out[0][1], out[1][1]) < 1e-5


def test_rejects_bad_arguments():
    with pytest.raises(ValueError):
        R.ReferencePS(4, 3, 4, 0.1, 0.0, 0.0)          # n > lambda
    ps = R.ReferencePS(4, 3, 3, 0.1, 0.0, 0.0)
    with pytest.raises(ValueError):
        ps.push(0, np.zeros(4, np.float32))            # push before any pull
    with pytest.raises(ValueError):
        ps.pull(3)
