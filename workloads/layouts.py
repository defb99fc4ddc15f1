"""Parameter-vector layouts of the synthetic workloads.

The paper trains two networks: a CIFAR10 CNN of about 90 K parameters (three
convolutions and one fully connected layer, Section 4.1) and an AlexNet-style
ImageNet CNN (five convolutions, three fully connected layers, Section 4.1).
Only their flat parameter-vector shapes matter to the parameter server, so a
layout here is an ordered list of segments (name, element count, is_bias).

This module holds shapes only: no update arithmetic, no timestamps.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple


@dataclass(frozen=True)
class Segment:
    name: str
    offset: int
    count: int
    is_bias: bool


@dataclass(frozen=True)
class Layout:
    name: str
    segments: Tuple[Segment, ...]

    @property
    def num_params(self) -> int:
        last = self.segments[-1]
        return last.offset + last.count


def _build(name: str, layers: List[Tuple[str, int, int]]) -> Layout:
    segs = []
    off = 0
    for lname, n_weight, n_bias in layers:
        segs.append(Segment(lname + ".weight", off, n_weight, False))
        off += n_weight
        if n_bias:
            segs.append(Segment(lname + ".bias", off, n_bias, True))
            off += n_bias
    return Layout(name, tuple(segs))


def cifar_cnn() -> Layout:
    """Small CNN, 89,578 elements: conv 32x3x5x5, 32x32x5x5, 64x32x5x5, fc 10x1024."""
    return _build("cifar_cnn", [
        ("conv1", 32 * 3 * 5 * 5, 32),
        ("conv2", 32 * 32 * 5 * 5, 32),
        ("conv3", 64 * 32 * 5 * 5, 64),
        ("fc", 10 * 1024, 10),
    ])


def alexnet_like() -> Layout:
    """Large CNN, 60,965,224 elements (grouped-convolution AlexNet shapes)."""
    return _build("alexnet_like", [
        ("conv1", 96 * 3 * 11 * 11, 96),
        ("conv2", 256 * 48 * 5 * 5, 256),
        ("conv3", 384 * 256 * 3 * 3, 384),
        ("conv4", 384 * 192 * 3 * 3, 384),
        ("conv5", 256 * 192 * 3 * 3, 256),
        ("fc6", 4096 * 9216, 4096),
        ("fc7", 4096 * 4096, 4096),
        ("fc8", 1000 * 4096, 1000),
    ])


def flat(num_params: int) -> Layout:
    """A single weight segment of `num_params` elements (bandwidth sweep)."""
    return _build("flat%d" % num_params, [("flat", int(num_params), 0)])
