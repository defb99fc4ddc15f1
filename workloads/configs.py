"""The benchmark configurations: sizes, hyper-parameters and input recipes.

Each configuration fixes the number of learners (lambda), the splitting
parameter n of the n-softsync protocol (Section 2.2; an update fires after
c = floor(lambda/n) gradients), the hyper-parameters the paper trains with
(momentum 0.9, alpha0 0.001 for the small net and 0.01 for the large one,
Section 4.3) and the synthetic stand-ins for its inputs.  Data only.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Callable

from . import layouts

SEED = 151105950


@dataclass(frozen=True)
class Config:
    name: str
    layout: Callable[[], layouts.Layout]
    num_learners: int          # lambda
    n: int                     # splitting parameter
    alpha0: float
    momentum: float
    weight_decay: float
    modulation: str            # "inv_staleness" | "constant"
    grad_dtype: str            # "fp32" | "bf16"
    grad_std: float
    weight_std: float
    arrival_model: str
    num_pushes: int
    fuse_t: int = 1
    seed: int = SEED

    @property
    def c(self) -> int:
        return self.num_learners // self.n

    @property
    def num_updates(self) -> int:
        return self.num_pushes // self.c

    def scaled(self, num_pushes: int) -> "Config":
        return replace(self, num_pushes=num_pushes)


TINY_SOFTSYNC = Config(
    name="tiny_softsync", layout=layouts.cifar_cnn, num_learners=4, n=1,
    alpha0=0.001, momentum=0.9, weight_decay=5e-4, modulation="inv_staleness",
    grad_dtype="fp32", grad_std=1e-3, weight_std=0.01,
    arrival_model="rounds", num_pushes=800)

PURE_ASYNC = Config(
    name="pure_async", layout=layouts.cifar_cnn, num_learners=30, n=30,
    alpha0=0.001, momentum=0.9, weight_decay=5e-4, modulation="inv_staleness",
    grad_dtype="fp32", grad_std=1e-3, weight_std=0.01,
    arrival_model="exp", num_pushes=10000)

LARGE_SOFTSYNC = Config(
    name="large_softsync", layout=layouts.alexnet_like, num_learners=18, n=4,
    alpha0=0.01, momentum=0.9, weight_decay=5e-4, modulation="inv_staleness",
    grad_dtype="fp32", grad_std=1e-4, weight_std=0.01,
    arrival_model="uniform", num_pushes=2000)

LARGE_STALE_BF16 = Config(
    name="large_stale_bf16", layout=layouts.alexnet_like, num_learners=54, n=54,
    alpha0=0.01, momentum=0.9, weight_decay=5e-4, modulation="inv_staleness",
    grad_dtype="bf16", grad_std=1e-4, weight_std=0.01,
    arrival_model="lognormal", num_pushes=2000, fuse_t=8)

ALL = (TINY_SOFTSYNC, PURE_ASYNC, LARGE_SOFTSYNC, LARGE_STALE_BF16)
BY_NAME = {c.name: c for c in ALL}

SWEEP_SIZES = (1 << 20, 1 << 24, 60965224, 1 << 28, 1 << 30)
SWEEP_C = (1, 4, 16, 64)
