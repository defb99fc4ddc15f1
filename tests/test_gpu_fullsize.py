"""Parity at the benchmark's full sizes, on sampled elements.

The update is element-wise, so the reference can follow any subset of elements on its own:
the GPU runs the whole 60,965,224-element vector through the default launch configuration
(the one bench.py times), gradients generated on the device; the reference runs the same
protocol on a few thousand sampled elements whose inputs the generator reproduces bit for
bit on the CPU.  Timestamps, staleness and grouping do not depend on the vector length and
are compared in full.
"""
import numpy as np
import pytest
import torch

import paper_1511_05950_b200 as P
from oracle import reference as R
from tests.gpu_harness import TORCH_DTYPE, as_reference_grad, assert_logs_equal, parity_line, same_bits
from tests.helpers import PULL, rel_l2
from workloads import configs, generators as G

pytestmark = pytest.mark.gpu


def sample_indices(layout, count, seed):
    n = layout.num_params
    rng = np.random.default_rng(seed)
    idx = set(rng.integers(0, n, size=count).tolist())
    for seg in layout.segments:                       # every layer boundary, both sides
        for k in range(-8, 8):
            for base in (seg.offset, seg.offset + seg.count):
                if 0 <= base + k < n:
                    idx.add(base + k)
    idx.update(range(0, 64))
    idx.update(range(n - 64, n))
    return torch.tensor(sorted(idx), dtype=torch.int64)


def run_full(cfg, lazy, num_pushes=None, overlap=False):
    dev = torch.device("cuda", 0)
    layout = cfg.layout()
    n = layout.num_params
    pushes = num_pushes or cfg.num_pushes
    tdt = TORCH_DTYPE[cfg.grad_dtype]
    idx = sample_indices(layout, 6000, 1)
    idx_dev = idx.to(dev)
    kinds, learners = R.simulate_arrivals(cfg.arrival_model, cfg.num_learners, pushes, cfg.seed)

    refs = {}
    w0_s = G.initial_weights_at(layout, cfg.seed, idx, cfg.weight_std)
    for prec in (32, 64):
        r = R.ReferencePS(idx.numel(), cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                          P.binding.MODULATIONS[cfg.modulation], prec)
        r.set_weights(w0_s.numpy())
        refs[prec] = r

    ps = P.ParameterServer(n, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                           cfg.modulation, cfg.grad_dtype, cfg.fuse_t, device=dev)
    ps.init_weights(G.initial_weights(layout, cfg.seed, cfg.weight_std, device=dev))
    if overlap:
        ps.set_option(P.PS_OPT_OVERLAP_LAUNCH, 1)
    assert torch.equal(ps.w[idx_dev].cpu(), w0_s)      # same generator bits on both devices

    pulled, counts, ready = {}, {}, 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            pulled[l] = ps.pull_weights()
            for r in refs.values():
                assert r.pull(l) == pulled[l]
            continue
        p = counts.get(l, 0)
        counts[l] = p + 1
        g = G.gradient(cfg.seed, l, p, n, cfg.grad_std, dtype=tdt, device=dev)
        gs = G.gradient_at(cfg.seed, l, p, idx, cfg.grad_std, dtype=tdt)
        if p == 0:
            assert torch.equal(g[idx_dev].cpu(), gs)
        host = as_reference_grad(gs)
        for r in refs.values():
            r.push(l, host)
        ready += ps.push_gradient(l, g, pulled[l])
        if ready and (not lazy or ready >= cfg.fuse_t):
            if overlap:
                torch.cuda.synchronize()      # the gradient just generated is complete before the update starts
            ready -= ps.apply_update()
    ps.flush()
    ps.synchronize()

    w = ps.w[idx_dev].cpu().numpy()
    v = ps.v[idx_dev].cpu().numpy()
    log = ps.update_log()
    assert ps.timestamps() == (pushes // cfg.c, pushes // cfg.c)
    assert torch.isfinite(ps.w).all() and torch.isfinite(ps.v).all()
    ps.destroy()

    w32, v32 = refs[32].state()
    assert_logs_equal(log, refs[32].log())
    assert same_bits(w, w32) and same_bits(v, v32)
    w64, v64 = refs[64].state()
    tol = 1e-3 if cfg.grad_dtype == "bf16" else 1e-5
    assert rel_l2(w, w64) <= tol and rel_l2(v, v64) <= tol
    parity_line(cfg.name, n, pushes // cfg.c, "%d sampled elements" % idx.numel(), w, v, w32, v32, w64, v64)
    return log


def test_large_softsync_full_size():
    """Config 3: 60,965,224 elements, lambda=18, n=4 (c=4), fp32 gradients, 500 updates."""
    log = run_full(configs.LARGE_SOFTSYNC, lazy=False, overlap=True)     # launch mode bench.py times
    assert log["update"][-1] == 499
    assert 3.0 < log["tau"][200:].mean() < 5.5          # <tau> close to n = 4 (Section 2.4)


def test_large_stale_bf16_full_size():
    """Config 4: same vector, lambda=54, n=54 (c=1), bf16 gradients, 2,000 pushes applied 8 per pass."""
    log = run_full(configs.LARGE_STALE_BF16, lazy=True)
    assert len(log) == 2000 and log["tau"].max() > 100


class PartitionedReference:
    """The unmodified reference on the whole vector, one instance per contiguous range and host thread (the
    update is element-wise, so the ranges are independent; the C calls release the interpreter lock)."""

    def __init__(self, cfg, w0: np.ndarray, threads: int, layers=None):
        from concurrent.futures import ThreadPoolExecutor
        n = w0.size
        self.bounds = [n * t // threads for t in range(threads + 1)]
        self.pool = ThreadPoolExecutor(threads)
        self.parts = []
        for a, b in zip(self.bounds[:-1], self.bounds[1:]):
            r = R.ReferencePS(b - a, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                              P.binding.MODULATIONS[cfg.modulation], 32)
            r.set_weights(w0[a:b])
            if layers is not None:                       # the layer table restricted to [a, b)
                bounds, lm, dm = layers
                cut = [min(max(x, a), b) - a for x in bounds]
                r.set_layer_multipliers(cut, lm, dm)
            self.parts.append((a, b, r))

    def pull(self, learner):
        return [r.pull(learner) for _, _, r in self.parts][0]

    def push(self, learner, grad: np.ndarray):
        list(self.pool.map(lambda part: part[2].push(learner, grad[part[0]:part[1]]), self.parts))

    def assert_state_equals(self, w: np.ndarray, v: np.ndarray):
        for a, b, r in self.parts:
            wr, vr = r.state()
            assert same_bits(w[a:b], wr), "weights differ in [%d, %d)" % (a, b)
            assert same_bits(v[a:b], vr), "momentum differs in [%d, %d)" % (a, b)

    def close(self):
        self.pool.shutdown()
        for _, _, r in self.parts:
            r.close()


@pytest.mark.parametrize("cfg,updates,layers", [
    (configs.LARGE_SOFTSYNC, 16, False), (configs.LARGE_STALE_BF16, 32, False), (configs.LARGE_SOFTSYNC, 4, True)],
    ids=["large_softsync", "large_stale_bf16", "large_softsync_layer_multipliers"])
def test_every_element_at_full_size(cfg, updates, layers):
    """Configs 3 and 4 on the whole 60,965,224-element vector in the launch mode bench.py times
    (programmatic dependent launches, T = 8 for the bf16 case), an even number of launches so that both
    traversal directions and overlapped pairs occur: EVERY element of theta and v bit-equal to the fp32
    reference, the log equal.  Third case: the same with Caffe-style per-layer multipliers."""
    import os
    from tests.test_gpu_parity import caffe_style_multipliers
    dev = torch.device("cuda", 0)
    layout = cfg.layout()
    n = layout.num_params
    tdt = TORCH_DTYPE[cfg.grad_dtype]
    pushes = updates * cfg.c
    table = caffe_style_multipliers(layout) if layers else None
    kinds, learners = R.simulate_arrivals(cfg.arrival_model, cfg.num_learners, pushes, cfg.seed)
    w0 = G.initial_weights(layout, cfg.seed, cfg.weight_std, device=dev)
    ref = PartitionedReference(cfg, w0.cpu().numpy(), max(1, min(32, os.cpu_count() or 1)), table)
    ps = P.ParameterServer(n, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                           cfg.modulation, cfg.grad_dtype, cfg.fuse_t, device=dev)
    if table:
        ps.set_layer_multipliers(*table)
    ps.init_weights(w0)
    ps.set_option(P.PS_OPT_OVERLAP_LAUNCH, 1)
    pulled, counts, ready, held = {}, {}, 0, []
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            pulled[l] = ps.pull_weights()
            assert ref.pull(l) == pulled[l]
            continue
        p = counts.get(l, 0)
        counts[l] = p + 1
        g = G.gradient(cfg.seed, l, p, n, cfg.grad_std, dtype=tdt, device=dev)
        ref.push(l, as_reference_grad(g))                  # the device-to-host copy also completes the gradient
        ready += ps.push_gradient(l, g, pulled[l])
        if ready >= cfg.fuse_t:
            ready -= ps.apply_update()                     # back-to-back launches overlap when the next group is ready
    ps.flush(); ps.synchronize()
    launches = ps.get_option(P.PS_OPT_LAUNCHES_VECTOR)
    assert launches == updates // cfg.fuse_t and launches % 2 == 0 and ps.get_option(P.PS_OPT_LAUNCHES_SCALAR) == 0
    ref.assert_state_equals(ps.w.cpu().numpy(), ps.v.cpu().numpy())
    assert_logs_equal(ps.update_log(), ref.parts[0][2].log())
    print("PARITY | %s%s | %d | %d | all elements, %d launches | theta, v and log bit-equal to the fp32 reference |"
          % (cfg.name, " + layer multipliers" if layers else "", n, updates, launches))
    ps.destroy()
    ref.close()


@pytest.mark.parametrize("align", [4, 0], ids=["starts_8_byte_aligned", "starts_16_byte_aligned"])
def test_eight_shards_of_the_bf16_config_keep_the_vector_kernel(align):
    """Config 4 (bf16 gradients, T = 8) cut into the eight contiguous shards an 8-GPU server would use, all
    on this GPU: every shard's pointers satisfy the vector kernel (bf16 gradient slices are only 8-byte
    aligned at some shard starts), every launch reports the vector kernel, and the shards together equal
    the unsharded server on every element and the reference on sampled ones."""
    from paper_1511_05950_b200.sharded import shard_bounds
    cfg = configs.LARGE_STALE_BF16
    dev = torch.device("cuda", 0)
    layout = cfg.layout()
    n = layout.num_params
    bounds = shard_bounds(n, 8, align=align, grad_dtype="bf16")
    if align == 4:                                          # the split an fp32 server would use
        assert any((2 * b) % 16 == 8 for b in bounds[1:-1])
    else:                                                   # the split the sharded server picks for bf16 gradients
        assert all((2 * b) % 16 == 0 for b in bounds[1:-1])
    pushes = 16
    idx = sample_indices(layout, 4000, 2)
    idx_dev = idx.to(dev)
    kinds, learners = R.simulate_arrivals(cfg.arrival_model, cfg.num_learners, pushes, cfg.seed)
    ref = R.ReferencePS(idx.numel(), cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                        P.binding.MODULATIONS[cfg.modulation], 32)
    ref.set_weights(G.initial_weights_at(layout, cfg.seed, idx, cfg.weight_std).numpy())
    w0 = G.initial_weights(layout, cfg.seed, cfg.weight_std, device=dev)
    whole = P.ParameterServer(n, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                              cfg.modulation, "bf16", 8, device=dev)
    whole.init_weights(w0)
    wbuf, vbuf = torch.empty(n, device=dev), torch.empty(n, device=dev)
    shards = []
    for a, b in zip(bounds[:-1], bounds[1:]):
        sh = P.ParameterServer(b - a, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                               cfg.modulation, "bf16", 8, device=dev, state=(wbuf[a:b], vbuf[a:b]))
        sh.set_option(P.PS_OPT_KERNEL, P.PS_KERNEL_VECTOR)          # a scalar fallback would be an error
        sh.init_weights(w0[a:b])
        shards.append((a, b, sh))
    pulled, counts = {}, {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            pulled[l] = whole.pull_weights()
            assert ref.pull(l) == pulled[l]
            assert all(sh.pull_weights() == pulled[l] for _, _, sh in shards)
            continue
        p = counts.get(l, 0); counts[l] = p + 1
        g = G.gradient(cfg.seed, l, p, n, cfg.grad_std, dtype=torch.bfloat16, device=dev)
        ref.push(l, as_reference_grad(G.gradient_at(cfg.seed, l, p, idx, cfg.grad_std, dtype=torch.bfloat16)))
        whole.push_gradient(l, g, pulled[l])
        for a, b, sh in shards:
            sh.push_gradient(l, g[a:b], pulled[l])
    assert whole.flush() == 16
    for a, b, sh in shards:
        assert sh.flush() == 16
        assert sh.get_option(P.PS_OPT_LAST_KERNEL) == P.PS_KERNEL_VECTOR
        assert sh.get_option(P.PS_OPT_LAUNCHES_VECTOR) == 2 and sh.get_option(P.PS_OPT_LAUNCHES_SCALAR) == 0
    torch.cuda.synchronize()
    assert torch.equal(whole.w, wbuf) and torch.equal(whole.v, vbuf)
    w32, v32 = ref.state()
    assert np.array_equal(wbuf[idx_dev].cpu().numpy(), w32.astype(np.float32))
    assert np.array_equal(vbuf[idx_dev].cpu().numpy(), v32.astype(np.float32))
    for _, _, sh in shards:
        sh.destroy()
    whole.destroy()


@pytest.mark.parametrize("grad_dtype", ["fp32", "bf16"])
def test_more_than_two_to_the_thirty_elements(grad_dtype):
    """A ragged vector of 2^30 + 3 elements (the sweep's largest size): byte offsets beyond 2^32, the
    scalar tail after the last full fragment, both traversal directions.  Sampled parity over 3 updates."""
    from workloads import layouts
    dev = torch.device("cuda", 0)
    n = (1 << 30) + 3
    need = n * (8 + 2 * 4) + (6 << 30)
    free, _ = torch.cuda.mem_get_info(dev)
    if free < need:
        pytest.skip("not enough free device memory for the 2^30-element case")
    tdt = TORCH_DTYPE[grad_dtype]
    layout = layouts.flat(n)
    rng = np.random.default_rng(5)
    picks = set(rng.integers(0, n, size=3000).tolist())
    for centre in (0, 1 << 29, (1 << 30) - 64, 1 << 30, n - 1):
        picks.update(k for k in range(centre - 40, centre + 40) if 0 <= k < n)
    idx = torch.tensor(sorted(picks), dtype=torch.int64)
    idx_dev = idx.to(dev)
    lam, c = 2, 2
    ref = R.ReferencePS(idx.numel(), lam, 1, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(G.initial_weights_at(layout, 3, idx).numpy())
    ps = P.ParameterServer(n, lam, 1, 0.01, 0.9, 5e-4, grad_dtype=grad_dtype, device=dev)
    G.normal_like(G.stream_key(3, G.STREAM_WEIGHTS), 0, n, 0.01, out=ps.w)
    ps.v.zero_()
    for u in range(3):
        grads = []
        for l in range(lam):
            ts = ps.pull_weights()
            assert ref.pull(l) == ts
        for l in range(lam):
            g = torch.empty(n, dtype=tdt, device=dev)
            G.gradient(3, l, u, n, 1e-3, dtype=tdt, device=dev, out=g)
            grads.append(g)
            ref.push(l, as_reference_grad(G.gradient_at(3, l, u, idx, 1e-3, dtype=tdt)))
            ps.push_gradient(l, g, u)
        assert ps.apply_update() == 1
        ps.synchronize()
        del grads
    w32, v32 = ref.state()
    assert np.array_equal(ps.w[idx_dev].cpu().numpy(), w32.astype(np.float32))
    assert np.array_equal(ps.v[idx_dev].cpu().numpy(), v32.astype(np.float32))
    assert ps.timestamps() == (3, 3)
    ps.destroy()
