"""Shared test plumbing: replaying an arrival trace and error measures."""
from __future__ import annotations

import numpy as np

PULL, PUSH = 0, 1


def replay_reference(ps, kinds, learners, grad_fn):
    """Feed a trace to a ReferencePS.  grad_fn(learner, push_index) -> ndarray."""
    counts = {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            ps.pull(l)
        else:
            p = counts.get(l, 0)
            counts[l] = p + 1
            ps.push(l, grad_fn(l, p))


def staleness_by_recount(kinds, learners, c):
    """Brute-force staleness of every push of a trace, in arrival order.

    Uses only the clock rules of Section 2.1: the clock equals the number of
    complete groups of c pushes seen so far, a learner's gradient carries the
    clock value of its latest pull, tau is the difference.
    """
    taus, clocks = [], []
    pulled = {}
    pushes = 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        clock = pushes // c
        if k == PULL:
            pulled[l] = clock
        else:
            taus.append(clock - pulled[l])
            clocks.append(clock)
            pushes += 1
    return np.asarray(taus, dtype=np.int64), np.asarray(clocks, dtype=np.int64)


def rel_l2(x, ref):
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    num = np.linalg.norm(x - ref)
    return num / den if den > 0 else num
