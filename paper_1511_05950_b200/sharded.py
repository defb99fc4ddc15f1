"""Sharded parameter server: one contiguous range of the parameter vector per rank.

The paper shards its parameter server and notes that the shards need no synchronisation with each other
(Section 2.3): the update is element-wise, so every shard applies the same protocol decisions to its own
range.  Here rank r of a torch.distributed group owns elements [bounds[r], bounds[r+1]) and runs an ordinary
server (the C-ABI library) on them.  Every rank must see the same sequence of pulls and pushes; a push hands
each rank its own slice of the gradient; the only exchange is the all-gather that assembles the full weight
vector for a pull, or, with replica buffers bound, the stores with which every shard's update kernel writes its
range of the new weights into every GPU's buffer while it computes them.  With a world size of one this is the
plain server.
"""
from __future__ import annotations

from typing import Callable, List, Optional

import torch
import torch.distributed as dist

SHARD_ALIGN = 4          # elements: 16 bytes of fp32, so theta, v and fp32 gradients keep the vector kernel


def shard_align(grad_dtype: str = "fp32", bf16_arrays: bool = False) -> int:
    """Elements a shard start must be a multiple of so that every array the server touches starts on a
    16-byte boundary there: 4 for fp32 data, 8 as soon as bf16 gradients or a bf16 weight mirror are in
    play (the vector kernel itself needs only 8 bytes for those, the bulk-copy kernel and copies 16)."""
    return 8 if (grad_dtype == "bf16" or bf16_arrays) else SHARD_ALIGN


def shard_bounds(num_params: int, world: int, align: int = 0, grad_dtype: str = "fp32",
                 bf16_arrays: bool = False) -> List[int]:
    """world+1 offsets splitting [0, num_params) into contiguous ranges whose starts are multiples of
    `align` (default: shard_align of the data types); sizes differ by at most `align` and the last range
    takes the ragged end."""
    align = align or shard_align(grad_dtype, bf16_arrays)
    units = (num_params + align - 1) // align
    bounds = [min(num_params, (units * r // world) * align) for r in range(world)]
    return bounds + [num_params]


class ShardedParameterServer:
    def __init__(self, num_params: int, num_learners: int, n: int, alpha0: float, momentum: float = 0.0,
                 weight_decay: float = 0.0, modulation: str = "inv_staleness", grad_dtype: str = "fp32",
                 fuse_t: int = 1, device: Optional[torch.device] = None, group=None,
                 server_factory: Optional[Callable] = None):
        self.group = group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.num_params = int(num_params)
        self.bounds = shard_bounds(self.num_params, self.world, grad_dtype=grad_dtype)
        self.lo, self.hi = self.bounds[self.rank], self.bounds[self.rank + 1]
        self.device = device
        if server_factory is None:
            from .binding import ParameterServer
            server_factory = ParameterServer
        self.local = server_factory(self.hi - self.lo, num_learners, n, alpha0, momentum, weight_decay,
                                    modulation, grad_dtype, fuse_t, device=device)
        self._max_shard = max(b - a for a, b in zip(self.bounds[:-1], self.bounds[1:]))
        self.replica_buffers = []

    # -- set-up ---------------------------------------------------------------
    def init_weights(self, w0_full: torch.Tensor) -> None:
        """Every rank passes the same full-length initial vector and keeps its own range."""
        assert w0_full.numel() == self.num_params
        self.local.init_weights(w0_full[self.lo:self.hi].contiguous())

    # -- the protocol ----------------------------------------------------------
    def pull_weights(self, out_full: Optional[torch.Tensor] = None) -> int:
        """Timestamp only, or (out_full given) the whole weight vector assembled from all shards."""
        if out_full is None:
            return self.local.pull_weights()
        assert out_full.numel() == self.num_params and out_full.dtype == torch.float32
        if self.world == 1:
            return self.local.pull_weights(out_full)
        mine = torch.zeros(self._max_shard, dtype=torch.float32, device=out_full.device)   # equal-sized pieces
        ts = self.local.pull_weights(mine[: self.hi - self.lo]) if self.hi > self.lo else self.local.pull_weights()
        self.local.synchronize()
        gathered = torch.empty(self.world * self._max_shard, dtype=torch.float32, device=out_full.device)
        dist.all_gather_into_tensor(gathered, mine, group=self.group)
        for r in range(self.world):
            a, b = self.bounds[r], self.bounds[r + 1]
            out_full[a:b] = gathered[r * self._max_shard: r * self._max_shard + (b - a)]
        return ts

    def push_gradient(self, learner: int, grad_full: torch.Tensor, ts: int) -> bool:
        """`grad_full` is the full-length gradient as this rank holds it; only this rank's range is read
        (a learner on another machine would send each shard its range)."""
        assert grad_full.numel() == self.num_params
        return self.local.push_gradient(learner, grad_full[self.lo:self.hi], ts)

    def push_gradient_slice(self, learner: int, grad_slice: torch.Tensor, ts: int) -> bool:
        """The scattered push: a learner sends every shard only that shard's range of its gradient
        (elements [lo, hi) of this rank); nothing else of the gradient needs to exist on this rank."""
        if grad_slice.numel() != self.hi - self.lo:
            raise ValueError("slice of %d elements for a shard of %d" % (grad_slice.numel(), self.hi - self.lo))
        return self.local.push_gradient(learner, grad_slice, ts)

    # -- weight broadcast fused into the update ----------------------------------
    def bind_replica_buffers(self, full_buffers) -> None:
        """`full_buffers`: full-length fp32 tensors that THIS GPU can address, one per GPU whose learners should
        find the whole weight vector in their own memory (this GPU's own buffer, and peer mappings of the
        other GPUs' buffers, which the caller sets up).  This rank's update kernel then stores its range of the
        new theta into every one of them while it computes it: after all ranks' updates the buffers hold the
        assembled weights and a pull is a local read (`pull_weights_from_replica`).  The kernel only stores to
        the buffers; nothing of this library ever loads from another GPU's memory."""
        for t in full_buffers:
            if t.numel() != self.num_params or t.dtype != torch.float32:
                raise ValueError("a replica buffer holds the whole fp32 weight vector")
        self.replica_buffers = list(full_buffers)
        self.local.bind_weight_replicas([t[self.lo:self.hi] for t in self.replica_buffers])

    def pull_weights_from_replica(self) -> int:
        """The pull when replica buffers are bound: every rank waits for its own updates, the ranks meet at a
        barrier (control only, no weight bytes move), and this GPU's own replica buffer then holds the weights
        of the returned timestamp."""
        self.local.flush()
        ts = self.local.pull_weights()
        self.local.synchronize()
        if self.world > 1:
            dist.barrier(group=self.group)
        return ts

    # receive slots of this rank's shard: a learner on the same GPU writes its slice straight into server memory
    def bind_staging(self, num_slots: int) -> None:
        self.local.bind_staging(num_slots)

    def acquire_slot(self):
        return self.local.acquire_slot()

    def push_slot(self, learner: int, slot_id: int, ts: int) -> bool:
        return self.local.push_slot(learner, slot_id, ts)

    def apply_update(self) -> int:
        return self.local.apply_update()

    def flush(self) -> int:
        return self.local.flush()

    def synchronize(self) -> None:
        self.local.synchronize()

    def timestamps(self):
        return self.local.timestamps()

    def update_log(self, *a, **k):
        return self.local.update_log(*a, **k)

    def destroy(self) -> None:
        self.local.destroy()
