"""Pins for the reference's arrival simulator and clock bookkeeping.

What fixes the expected values:
  - Section 2.4 / Fig. 1: lambda = 30 homogeneous learners, 1-softsync: tau in {0,1,2};
    15- and 30-softsync: mean staleness close to n, (almost) nothing beyond 2n.
  - With i.i.d. Exp(1) compute times, c = 1 and push-then-pull, the staleness of a push is
    the number of other learners' completions during one's own compute time: geometric,
    P(tau = k) = (lambda-1)^k / lambda^(k+1), mean lambda - 1 (memorylessness).
  - Section 2.1: clock rules, recounted by brute force from the raw trace.
"""
import numpy as np
import pytest

from oracle import reference as R
from tests.helpers import replay_reference, staleness_by_recount


def run_log(model, lam, n, pushes, seed, modulation=R.MOD_INV_STALENESS):
    k, l = R.simulate_arrivals(model, lam, pushes, seed)
    ps = R.ReferencePS(1, lam, n, 0.01, 0.0, 0.0, modulation, 64)
    ps.set_weights(np.zeros(1, np.float32))
    g = np.ones(1, np.float32)
    replay_reference(ps, k, l, lambda a, b: g)
    return k, l, ps


@pytest.mark.parametrize("n,lo,hi", [(1, 0.8, 1.2), (15, 13.5, 16.5), (30, 27.0, 33.0)])
def test_homogeneous_learners_match_measured_staleness(n, lo, hi):
    lam = 30
    k, l, ps = run_log("uniform", lam, n, 6000, seed=11)
    tau = ps.log()["tau"][600:]          # skip the start-up transient
    if n == 1:
        assert set(np.unique(tau).tolist()) <= {0, 1, 2}
    assert lo <= tau.mean() <= hi
    assert (tau > 2 * n).mean() < 1e-3
    assert tau.min() >= 0


def test_exponential_compute_times_give_geometric_staleness():
    lam, pushes = 30, 60000
    k, l, ps = run_log("exp", lam, lam, pushes, seed=5)
    tau = ps.log()["tau"][2000:]
    q = (lam - 1) / lam
    assert abs(tau.mean() - (lam - 1)) < 1.0
    assert abs((tau == 0).mean() - 1 / lam) < 0.004
    assert abs((tau > 60).mean() - q ** 61) < 0.01
    for kk in (1, 5, 20):
        assert abs((tau == kk).mean() - q ** kk / lam) < 0.004


def test_rounds_model_keeps_sigma_one():
    k, l, ps = run_log("rounds", 4, 1, 800, seed=3)
    log = ps.log()
    assert set(np.unique(log["tau"]).tolist()) <= {0, 1}
    assert (log["sigma"] == 1).all()
    assert ps.timestamp == 200


def test_lognormal_speeds_are_heavy_tailed():
    k, l, ps = run_log("lognormal", 54, 54, 2000, seed=8)
    tau = ps.log()["tau"]
    assert tau.max() > 100 and tau.min() >= 0
    pushes_per_learner = np.bincount(l[k == R.PUSH], minlength=54)
    assert pushes_per_learner.max() > 3 * max(1, pushes_per_learner.min())


def test_lognormal_model_has_the_stated_speed_and_jitter_laws():
    """Persistent speed exp(0.5 z), z ~ N(0,1), times a per-iteration jitter U[0.95, 1.05]: measured on the
    simulated times.  The log of a learner's mean iteration time has standard deviation 0.5 (a shape
    parameter of 1.0 or 0.25 fails), is symmetric and normal-shaped; every iteration lies within 5 % of the
    learner's speed, uniformly (standard deviation 0.1/sqrt(12))."""
    lam, pushes = 1500, 150000
    k, l, t = R.simulate_arrivals_timed("lognormal", lam, pushes, 77)
    k2, l2 = R.simulate_arrivals("lognormal", lam, pushes, 77)
    assert np.array_equal(k, k2) and np.array_equal(l, l2)             # the timed form is the same trace
    push = k == R.PUSH
    assert (np.diff(t[push]) >= 0).all()                                # the server serves in time order
    speeds, rel = [], []
    for who in range(lam):
        times = t[push & (l == who)]
        if times.size < 12:
            continue
        dur = np.diff(np.concatenate([[0.0], times]))
        centre = 0.5 * (dur.max() + dur.min())                          # jitter is symmetric about the speed
        speeds.append(dur.mean())
        rel.append(dur / centre)
    z = np.log(np.asarray(speeds))
    assert len(speeds) > 0.9 * lam
    rel = np.concatenate(rel)
    assert rel.min() > 0.94 and rel.max() < 1.06
    assert abs(rel.std() - 0.1 / np.sqrt(12)) < 0.003
    # slow learners drop out of the sample above (fewer than 12 pushes), which trims the upper tail a little
    assert 0.42 < z.std() < 0.53
    inside = (np.abs(z - np.median(z)) < 0.5).mean()
    assert 0.62 < inside < 0.75                                          # 68 % within one shape parameter
    # more pushes from faster learners, in proportion to 1 / speed
    counts = np.bincount(l[push], minlength=lam)
    fast, slow = counts[np.argsort(counts)[-50:]].mean(), counts[np.argsort(counts)[:50]].mean()
    assert fast > 4 * slow


@pytest.mark.parametrize("model,lam,n", [("exp", 7, 3), ("uniform", 18, 4), ("lognormal", 9, 9), ("rounds", 5, 1)])
def test_clock_and_staleness_against_brute_force_recount(model, lam, n):
    pushes = 500
    k, l, ps = run_log(model, lam, n, pushes, seed=21)
    c = lam // n
    tau, clock = staleness_by_recount(k, l, c)
    log = ps.log()
    n_upd = pushes // c
    assert ps.timestamp == n_upd                       # +1 per update, from 0
    assert len(log) == n_upd * c                       # exactly c members per update
    assert np.array_equal(log["update"], np.repeat(np.arange(n_upd), c))
    assert np.array_equal(log["position"], np.tile(np.arange(c), n_upd))
    # members of update i are pushes i*c .. i*c+c-1 in arrival order; compare as multisets per update
    pl = l[k == R.PUSH][:n_upd * c]
    for i in range(n_upd):
        rows = log[i * c:(i + 1) * c]
        arr = sorted(zip(pl[i * c:(i + 1) * c].tolist(), tau[i * c:(i + 1) * c].tolist()))
        got = sorted(zip(rows["learner"].tolist(), rows["tau"].tolist()))
        assert arr == got
        assert (clock[i * c:(i + 1) * c] == i).all()   # footnote to Eq. 5: one clock value per group
        keys = list(zip(rows["learner"].tolist(), rows["push_index"].tolist()))
        assert keys == sorted(keys)                    # summation order
    assert (log["tau"] == log["update"] - log["ts_grad"]).all()
    assert (log["tau"] >= 0).all() and (log["sigma"] >= 1).all()
    assert np.array_equal(log["sigma"], np.maximum(log["tau"], 1))


def test_constant_modulation_records_tau_but_sigma_one():
    k, l, ps = run_log("exp", 6, 6, 300, seed=2, modulation=R.MOD_CONSTANT)
    log = ps.log()
    assert log["tau"].max() > 1 and (log["sigma"] == 1).all()
    assert np.allclose(log["scale"], np.float64(np.float32(0.01)))
