"""The sharded server's plumbing on CPU: two gloo ranks, each running the *reference* on its own range
(the CUDA library cannot run here), assembled weights compared with the unsharded reference."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1511_05950_b200.sharded import ShardedParameterServer, shard_bounds


def test_shard_bounds_are_aligned_contiguous_and_balanced():
    for n, world in [(60965224, 8), (89578, 4), (10, 4), (3, 8), (0, 2), (1 << 30, 3), (17, 1)]:
        b = shard_bounds(n, world)
        assert len(b) == world + 1 and b[0] == 0 and b[-1] == n
        assert all(x <= y for x, y in zip(b[:-1], b[1:]))
        assert all(x % 4 == 0 for x in b[:-1])
        sizes = [y - x for x, y in zip(b[:-1], b[1:])]
        assert max(sizes) - min(sizes) <= 4 or n < 4 * world


class ReferenceBackedServer:
    """Stands in for the CUDA server in this CPU test: same method names, reference arithmetic."""

    def __init__(self, num_params, num_learners, n, alpha0, momentum, weight_decay, modulation, grad_dtype, fuse_t,
                 device=None):
        from oracle import reference as R
        self.R = R
        self.ref = R.ReferencePS(num_params, num_learners, n, alpha0, momentum, weight_decay,
                                 R.MOD_INV_STALENESS if modulation == "inv_staleness" else R.MOD_CONSTANT, 32)
        self.num_params = num_params

    def init_weights(self, w0):
        self.ref.set_weights(w0.numpy())

    def pull_weights(self, out=None):
        if out is not None:
            out.copy_(torch.from_numpy(self.ref.state()[0].astype(np.float32)))
        return self.ref.timestamp

    def push_gradient(self, learner, grad, ts):
        return self.ref.push(learner, grad.contiguous().numpy(), timestamp=ts)

    def apply_update(self):
        return 1

    def flush(self):
        return 0

    def synchronize(self):
        pass

    def timestamps(self):
        return self.ref.timestamp, self.ref.timestamp

    def destroy(self):
        self.ref.close()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    from oracle import reference as R
    from workloads import generators as G, layouts
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n_el, lam, n = 10007, 6, 2
    w0 = G.initial_weights(layouts.flat(n_el), 5)
    sps = ShardedParameterServer(n_el, lam, n, 0.02, 0.9, 5e-4, server_factory=ReferenceBackedServer)
    sps.init_weights(w0)
    whole = R.ReferencePS(n_el, lam, n, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    whole.set_weights(w0.numpy())
    kinds, learners = R.simulate_arrivals("exp", lam, 40, 9)
    pulled, counts = {}, {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = sps.pull_weights()
            assert whole.pull(l) == pulled[l]
            continue
        b = counts.get(l, 0); counts[l] = b + 1
        g = G.gradient(5, l, b, n_el, 1e-3)
        whole.push(l, g.numpy())
        if sps.push_gradient(l, g, pulled[l]):
            sps.apply_update()
    full = torch.empty(n_el)
    ts = sps.pull_weights(full)                       # the all-gather
    ok = bool(np.array_equal(full.numpy(), whole.state()[0].astype(np.float32))) and ts == whole.timestamp
    out.put((rank, ok, sps.lo, sps.hi))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_assemble_the_unsharded_weights():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(ok for _, ok, _, _ in got)
    assert got[0][2] == 0 and got[0][3] == got[1][2] and got[1][3] == 10007


@pytest.mark.gpu
def test_world_of_one_is_the_plain_server():
    import paper_1511_05950_b200 as P
    from oracle import reference as R
    from workloads import generators as G, layouts
    dev = torch.device("cuda", 0)
    n_el = 5003
    w0 = G.initial_weights(layouts.flat(n_el), 2)
    sps = ShardedParameterServer(n_el, 2, 1, 0.05, 0.9, 5e-4, device=dev)
    sps.init_weights(w0.to(dev))
    ref = R.ReferencePS(n_el, 2, 1, 0.05, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    for u in range(3):
        ts = sps.pull_weights()
        for l in range(2):
            ref.pull(l)
            g = G.gradient(2, l, u, n_el, 1e-3, device=dev)
            ref.push(l, g.cpu().numpy())
            if sps.push_gradient(l, g, ts):
                sps.apply_update()
    out = torch.empty(n_el, device=dev)
    assert sps.pull_weights(out) == 3
    assert np.array_equal(out.cpu().numpy(), ref.state()[0].astype(np.float32))
    sps.destroy()
