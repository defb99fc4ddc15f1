"""The sharded server's plumbing on CPU with two gloo ranks.  The CUDA kernels cannot run here, so the
arithmetic of a shard is done by the *reference* behind the same method names (assembled weights compared
with the unsharded reference), and the CUDA library's own host state machine runs under gloo on shards
without parameters (its clocks and logs compared with the reference)."""
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


def test_every_shard_start_keeps_the_vector_kernel_for_every_array():
    """For the large network and 2..8 ranks: theta, v and fp32 gradients start on 16-byte boundaries in every
    shard; with bf16 gradients (or a bf16 weight mirror) the split moves to multiples of 8 elements so that the
    2-byte arrays do too.  The fp32 split would leave bf16 slices on 8-byte boundaries at some starts (which the
    vector kernel accepts, the bulk-copy kernel and 16-byte copies do not)."""
    n = 60965224
    on_8_only = 0
    for world in range(2, 9):
        fp32 = shard_bounds(n, world)
        assert all((4 * b) % 16 == 0 for b in fp32[:-1])
        on_8_only += sum((2 * b) % 16 == 8 for b in fp32[:-1])
        assert all((2 * b) % 8 == 0 for b in fp32[:-1])                     # the vector kernel's bf16 load width
        for kw in ({"grad_dtype": "bf16"}, {"bf16_arrays": True}):
            b16 = shard_bounds(n, world, **kw)
            assert b16[0] == 0 and b16[-1] == n and all(x <= y for x, y in zip(b16[:-1], b16[1:]))
            assert all((4 * b) % 16 == 0 and (2 * b) % 16 == 0 for b in b16[:-1])
            sizes = [y - x for x, y in zip(b16[:-1], b16[1:])]
            assert max(sizes) - min(sizes) <= 8
    assert on_8_only > 0


class ReferenceBackedServer:
    """Stands in for the CUDA server in this CPU test: same method names, reference arithmetic."""

    def __init__(self, num_params, num_learners, n, alpha0, momentum, weight_decay, modulation, grad_dtype, fuse_t,
                 device=None):
        from oracle import reference as R
        self.R = R
        self.ref = R.ReferencePS(num_params, num_learners, n, alpha0, momentum, weight_decay,
                                 R.MOD_INV_STALENESS if modulation == "inv_staleness" else R.MOD_CONSTANT, 32)
        self.num_params = num_params
        self.elements_received = 0

    def init_weights(self, w0):
        self.ref.set_weights(w0.numpy())

    def pull_weights(self, out=None):
        if out is not None:
            out.copy_(torch.from_numpy(self.ref.state()[0].astype(np.float32)))
        return self.ref.timestamp

    def push_gradient(self, learner, grad, ts):
        self.elements_received += grad.numel()
        fired = self.ref.push(learner, grad.contiguous().numpy(), timestamp=ts)
        if fired:                                 # the update "kernel" also stores theta into every replica
            self._write_replicas()
        return fired

    def bind_weight_replicas(self, replicas):
        self.replicas = list(replicas)
        self._write_replicas()

    def _write_replicas(self):
        for r in getattr(self, "replicas", []):
            r.copy_(torch.from_numpy(self.ref.state()[0].astype(np.float32)))

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


def _worker_scatter(rank, world, port, out):
    """Every rank is GIVEN only its own range of each gradient (generated for that range alone): the push is a
    scatter, no rank ever holds a full gradient."""
    from oracle import reference as R
    from workloads import generators as G, layouts
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n_el, lam, n = 10007, 6, 2
    w0 = G.initial_weights(layouts.flat(n_el), 5)
    sps = ShardedParameterServer(n_el, lam, n, 0.02, 0.9, 5e-4, server_factory=ReferenceBackedServer)
    sps.init_weights(w0)
    kinds, learners = R.simulate_arrivals("lognormal", lam, 48, 10)
    pulled, counts, pushes = {}, {}, 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = sps.pull_weights()
            continue
        b = counts.get(l, 0); counts[l] = b + 1
        key = G.stream_key(5, G.STREAM_GRADIENT, l, b)
        mine = G.normal_like(key, sps.lo, sps.hi - sps.lo, 1e-3)        # elements [lo, hi) only
        pushes += 1
        if sps.push_gradient_slice(l, mine, pulled[l]):
            sps.apply_update()
    full = torch.empty(n_el)
    ts = sps.pull_weights(full)
    ok = sps.local.elements_received == pushes * (sps.hi - sps.lo)
    if rank == 0:                                    # the unsharded reference, fed whole gradients
        whole = R.ReferencePS(n_el, lam, n, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
        whole.set_weights(w0.numpy())
        counts = {}
        for k, l in zip(kinds.tolist(), learners.tolist()):
            if k == 0:
                whole.pull(l)
                continue
            b = counts.get(l, 0); counts[l] = b + 1
            whole.push(l, G.gradient(5, l, b, n_el, 1e-3).numpy())
        ok = ok and bool(np.array_equal(full.numpy(), whole.state()[0].astype(np.float32))) and ts == whole.timestamp
    with pytest.raises(ValueError):
        sps.push_gradient_slice(0, torch.zeros(n_el), ts)              # a whole gradient is not a slice
    out.put((rank, ok, sps.lo, sps.hi))
    dist.barrier()
    dist.destroy_process_group()


def _worker_library_state_machine(rank, world, port, out):
    """The CUDA library itself under gloo: shards without parameters launch nothing, so its host side
    (clocks, staleness, grouping, scale table, log) runs here, once per rank, in lock-step."""
    import paper_1511_05950_b200 as P
    from oracle import reference as R
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lam, n = 9, 3
    sps = ShardedParameterServer(0, lam, n, 0.02, 0.9, 5e-4, fuse_t=4)
    assert isinstance(sps.local, P.ParameterServer) and (sps.lo, sps.hi) == (0, 0)
    ref = R.ReferencePS(0, lam, n, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    kinds, learners = R.simulate_arrivals("exp", lam, 90, 11)
    nothing = torch.zeros(0)
    pulled = {}
    ok = True
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = sps.pull_weights()
            ok = ok and ref.pull(l) == pulled[l]
            continue
        ref.push(l, nothing.numpy())
        sps.push_gradient_slice(l, nothing, pulled[l])
        a, lg = sps.timestamps()
        if lg - a >= 4:
            sps.apply_update()
    sps.flush()
    log, rlog = sps.update_log(), ref.log()
    for f in ("update", "push_index", "ts_grad", "tau", "sigma", "learner", "position"):
        ok = ok and bool(np.array_equal(log[f], rlog[f]))
    ok = ok and bool(np.array_equal(log["scale"], rlog["scale"].astype(np.float32)))
    stamps = torch.tensor(list(sps.timestamps()), dtype=torch.int64)
    both = [torch.zeros_like(stamps) for _ in range(world)]
    dist.all_gather(both, stamps)                    # every shard reached the same clock
    ok = ok and all(torch.equal(b, stamps) for b in both) and int(stamps[0]) == ref.timestamp == 30
    out.put((rank, ok, sps.lo, sps.hi))
    dist.barrier()
    sps.destroy()
    dist.destroy_process_group()


def _worker_replica_broadcast(rank, world, port, out, buffers):
    """`buffers[q]` is rank q's full-length weight buffer, in memory every rank can address (shared memory here,
    a peer mapping on GPUs).  Each rank's update writes its own range into every buffer; a pull is then a read
    of the rank's own buffer after a barrier, with no gather."""
    from oracle import reference as R
    from workloads import generators as G, layouts
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n_el, lam, n = 10007, 6, 2
    w0 = G.initial_weights(layouts.flat(n_el), 5)
    sps = ShardedParameterServer(n_el, lam, n, 0.02, 0.9, 5e-4, server_factory=ReferenceBackedServer)
    sps.init_weights(w0)
    sps.bind_replica_buffers(buffers)
    whole = R.ReferencePS(n_el, lam, n, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    whole.set_weights(w0.numpy())
    ok = sps.pull_weights_from_replica() == 0 and torch.equal(buffers[rank], w0)       # filled when bound
    kinds, learners = R.simulate_arrivals("exp", lam, 40, 9)
    pulled, counts = {}, {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = sps.pull_weights()
            whole.pull(l)
            continue
        b = counts.get(l, 0); counts[l] = b + 1
        g = G.gradient(5, l, b, n_el, 1e-3)
        whole.push(l, g.numpy())
        if sps.push_gradient_slice(l, g[sps.lo:sps.hi].clone(), pulled[l]):
            sps.apply_update()
            if whole.timestamp % 4 == 0:          # a weight pull: wait, meet, read the local buffer
                ts = sps.pull_weights_from_replica()
                mine = buffers[rank].clone()
                dist.barrier()                    # nobody runs ahead and overwrites while the others still compare
                ok = ok and ts == whole.timestamp and bool(np.array_equal(mine.numpy(), whole.state()[0].astype(np.float32)))
    ts = sps.pull_weights_from_replica()
    ok = ok and ts == whole.timestamp == 40 // (lam // n) and bool(np.array_equal(buffers[rank].numpy(), whole.state()[0].astype(np.float32)))
    out.put((rank, ok, sps.lo, sps.hi))
    dist.barrier()
    sps.destroy()
    dist.destroy_process_group()


def _guarded(worker, rank, world, port, out, *extra):
    """A rank that raises reports at once instead of leaving the parent to wait for its result."""
    try:
        worker(rank, world, port, out, *extra)
    except BaseException:
        out.put((rank, False, -1, -1))
        raise


def _run_two_ranks(worker, *extra):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_guarded, args=(worker, r, 2, port, out) + extra) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(ok for _, ok, _, _ in got)
    return got


def test_scattered_push_needs_only_the_ranks_own_slice():
    got = _run_two_ranks(_worker_scatter)
    assert got[0][2] == 0 and got[0][3] == got[1][2] and got[1][3] == 10007


def test_weight_broadcast_into_every_ranks_buffer_replaces_the_gather():
    buffers = [torch.zeros(10007).share_memory_() for _ in range(2)]
    _run_two_ranks(_worker_replica_broadcast, buffers)
    assert torch.equal(buffers[0], buffers[1]) and float(buffers[0].abs().sum()) > 0


def test_library_state_machine_runs_per_shard_under_gloo():
    _run_two_ranks(_worker_library_state_machine)


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
