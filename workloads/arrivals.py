"""Seeded learner-arrival traces: the order in which learners reach the server.

A trace is workload data, like a gradient: a sequence of events (kind, learner)
with kind PULL = 0 or PUSH = 1.  Every learner follows the loop of Section 2.1
(pull weights, compute, push gradient) and, as in Section 2.3, pulls again
right after its push.  A trace says only who arrives when; timestamps,
staleness and grouping are derived from it by whoever consumes it.

Models (simulated time; ties broken by learner id):
  rounds     each round is one random permutation of the learners
  exp        compute time of every iteration ~ Exp(1), i.i.d.
  uniform    compute time ~ U[0.9, 1.1], i.i.d. (homogeneous learners)
  lognormal  learner l has a persistent speed exp(0.5 z_l), z_l ~ N(0,1),
             times a per-iteration jitter U[0.95, 1.05]
"""
from __future__ import annotations

import heapq
from typing import Tuple

import numpy as np

PULL = 0
PUSH = 1

MODELS = ("rounds", "exp", "uniform", "lognormal")


def make_trace(model: str, num_learners: int, num_pushes: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Return (kind, learner) int32 arrays; the trace ends after the last push's pull."""
    rng = np.random.Generator(np.random.Philox(seed))
    kinds, learners = [], []
    for l in range(num_learners):                     # everybody starts from the initial weights
        kinds.append(PULL)
        learners.append(l)
    pushes = 0
    if model == "rounds":
        while pushes < num_pushes:
            for l in rng.permutation(num_learners):
                if pushes == num_pushes:
                    break
                kinds += [PUSH, PULL]
                learners += [int(l), int(l)]
                pushes += 1
    elif model in ("exp", "uniform", "lognormal"):
        if model == "lognormal":
            speed = np.exp(0.5 * rng.standard_normal(num_learners))
        else:
            speed = np.ones(num_learners)

        def duration(l: int) -> float:
            if model == "exp":
                return float(rng.exponential(1.0))
            if model == "uniform":
                return float(rng.uniform(0.9, 1.1))
            return float(speed[l] * rng.uniform(0.95, 1.05))

        heap = [(duration(l), l) for l in range(num_learners)]
        heapq.heapify(heap)
        while pushes < num_pushes:
            t, l = heapq.heappop(heap)
            kinds += [PUSH, PULL]
            learners += [l, l]
            pushes += 1
            heapq.heappush(heap, (t + duration(l), l))
    else:
        raise ValueError("unknown arrival model %r" % (model,))
    return np.asarray(kinds, dtype=np.int32), np.asarray(learners, dtype=np.int32)
