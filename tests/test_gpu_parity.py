"""Parity of the CUDA path (through the C ABI) with the CPU reference, element by element.

Tolerances: the benchmark's — relative L2 <= 1e-5 on final weights and momentum against the
fp64 reference (<= 1e-3 with bf16 gradients) — and, stricter, bit equality with the fp32
reference, because the kernel performs the same separately rounded fp32 operations in the
same order.  Timestamps, staleness and group membership must be bit-exact.
"""
import numpy as np
import pytest
import torch

import paper_1511_05950_b200 as P
from oracle import reference as R
from tests.gpu_harness import run_pair, assert_parity, parity_line
from tests.helpers import PULL
from workloads import configs, generators as G, layouts

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5
TOL_BF16 = 1e-3


def run_config(cfg, num_pushes=None, layout=None, **kw):
    layout = layout or cfg.layout()
    pushes = num_pushes or cfg.num_pushes
    kinds, learners = R.simulate_arrivals(cfg.arrival_model, cfg.num_learners, pushes, cfg.seed)
    w0 = G.initial_weights(layout, cfg.seed, cfg.weight_std)
    w, v, log, refs = run_pair(layout.num_params, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum,
                               cfg.weight_decay, cfg.modulation, cfg.grad_dtype, cfg.grad_std,
                               kinds, learners, w0, cfg.seed, **kw)
    tol = TOL_BF16 if cfg.grad_dtype == "bf16" else TOL_FP32
    worst = assert_parity(w, v, log, refs, tol, layout)
    parity_line(cfg.name, layout.num_params, pushes // cfg.c, "all elements", w, v, refs[32][0], refs[32][1],
                refs[64][0], refs[64][1])
    return worst, log


def test_tiny_softsync_full():
    """Config 1 in full: lambda=4, n=1, 89,578 elements, 200 updates; state compared at every tenth of the run."""
    cfg = configs.TINY_SOFTSYNC
    worst, log = run_config(cfg, checkpoints=10)
    assert log["update"][-1] == 199 and (log["sigma"] == 1).all()


def test_pure_async_full():
    """Config 2 in full: lambda=30, n=30, 10,000 pushes with Exp(1) compute times."""
    cfg = configs.PURE_ASYNC
    worst, log = run_config(cfg, checkpoints=10)
    assert len(log) == 10000 and log["sigma"].max() > 60


def test_large_softsync_scaled_down():
    """Config 3's protocol (lambda=18, n=4, uniform arrivals) on a ragged vector of several tiles."""
    cfg = configs.LARGE_SOFTSYNC
    run_config(cfg, num_pushes=600, layout=layouts.flat(5 * 65536 + 4099))


@pytest.mark.parametrize("lazy", [False, True])
def test_large_stale_bf16_scaled_down(lazy):
    """Config 4's protocol (lambda=54, n=54, bf16 gradients, T=8) on a ragged vector."""
    cfg = configs.LARGE_STALE_BF16
    worst, log = run_config(cfg, num_pushes=400, layout=layouts.flat(3 * 65536 + 2053), fuse_t=8, lazy=lazy)
    assert log["sigma"].max() > 20


def _simple(num_params, lam, n, pushes, grad_dtype="fp32", model="exp", seed=77, **kw):
    """Random arrivals on a flat vector with the usual hyper-parameters, compared with both references."""
    kinds, learners = R.simulate_arrivals(model, lam, pushes, seed)
    w0 = G.initial_weights(layouts.flat(num_params), seed) if num_params else torch.zeros(0)
    w, v, log, refs = run_pair(num_params, lam, n, 0.01, 0.9, 5e-4, "inv_staleness", grad_dtype, 1e-3,
                               kinds, learners, w0, seed, **kw)
    assert_parity(w, v, log, refs, TOL_BF16 if grad_dtype == "bf16" else TOL_FP32)
    return w, v, log


@pytest.mark.parametrize("grad_dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("num_params", [1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 31, 33, 1023, 1025,
                                        16384, 16385, 16386, 16387, 16388, 16389, 16390, 16391])
def test_ragged_sizes(num_params, grad_dtype):
    _simple(num_params, 6, 3, 24, grad_dtype)


@pytest.mark.parametrize("grad_dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("misalign", [1, 2, 3])
def test_pointers_not_16_byte_aligned_take_the_scalar_path(misalign, grad_dtype):
    _simple(10007, 5, 2, 30, grad_dtype, misalign=misalign)


@pytest.mark.parametrize("grad_dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("lam,n", [(1, 1), (2, 1), (3, 1), (7, 1), (8, 1), (9, 1), (16, 1), (17, 1), (64, 1), (100, 1), (256, 1)])
def test_group_sizes(lam, n, grad_dtype):
    _simple(4099, lam, n, 3 * lam, grad_dtype, model="uniform")


@pytest.mark.parametrize("grad_dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("fuse_t", [2, 3, 8, 16])
@pytest.mark.parametrize("lam,n", [(4, 4), (6, 2), (40, 2)])
def test_temporal_fusion_is_invisible(lam, n, fuse_t, grad_dtype):
    """T groups per pass give the same bits as one group per pass."""
    pushes = 20 * (lam // n) + (lam // n) // 2
    a = _simple(8 * 1024 + 5, lam, n, pushes, grad_dtype, model="lognormal", fuse_t=fuse_t, lazy=True)
    b = _simple(8 * 1024 + 5, lam, n, pushes, grad_dtype, model="lognormal", fuse_t=1, lazy=False)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert np.array_equal(a[2], b[2])


@pytest.mark.parametrize("options", [
    {P.PS_OPT_KERNEL: P.PS_KERNEL_SCALAR}, {P.PS_OPT_KERNEL: P.PS_KERNEL_VECTOR},
    {P.PS_OPT_BLOCK_THREADS: 128}, {P.PS_OPT_BLOCK_THREADS: 256}, {P.PS_OPT_BLOCK_THREADS: 512},
    {P.PS_OPT_KERNEL: P.PS_KERNEL_SCALAR, P.PS_OPT_BLOCK_THREADS: 512},
    {P.PS_OPT_ZIGZAG: 0}, {P.PS_OPT_ZIGZAG: 0, P.PS_OPT_OVERLAP_LAUNCH: 1},
    {P.PS_OPT_KERNEL: P.PS_KERNEL_BULK},
    {P.PS_OPT_KERNEL: P.PS_KERNEL_BULK, P.PS_OPT_BULK_TILE: 256, P.PS_OPT_BULK_STAGES: 2},
    {P.PS_OPT_KERNEL: P.PS_KERNEL_BULK, P.PS_OPT_BULK_TILE: 512, P.PS_OPT_BULK_STAGES: 8, P.PS_OPT_BLOCK_THREADS: 128},
    {P.PS_OPT_KERNEL: P.PS_KERNEL_BULK, P.PS_OPT_BULK_TILE: 1024, P.PS_OPT_BULK_STAGES: 3, P.PS_OPT_OVERLAP_LAUNCH: 1},
])
def test_launch_shape_does_not_change_the_bits(options):
    want = {P.PS_KERNEL_SCALAR: "scalar", P.PS_KERNEL_BULK: "bulk"}.get(options.get(P.PS_OPT_KERNEL), "vector")
    for grad_dtype in ("fp32", "bf16"):
        _simple(70001, 8, 2, 40, grad_dtype, options=options)
        launches = run_pair.launches
        assert launches[want] == 10 and sum(launches.values()) == 10        # the kernel asked for is the one that ran
        assert run_pair.last_kernel == P.binding.KERNELS[want]


@pytest.mark.parametrize("grad_dtype,fuse_t,lam,n", [("fp32", 1, 8, 2), ("bf16", 8, 6, 6), ("fp32", 4, 8, 2), ("bf16", 1, 16, 1)])
def test_bulk_copy_kernel_matches_reference(grad_dtype, fuse_t, lam, n):
    """The shared-memory staged kernel on a vector of many tiles and a ragged end, both traversal directions
    (launches alternate), with temporal fusion, the bf16 mirror and a layer table whose boundaries cut
    fragments and tiles."""
    n_el = 37 * 4096 + 1234 + 3
    bounds = [0, 4096, 4097, 4097, 10001, 3 * 4096 + 2, 20 * 4096, n_el - 5, n_el]
    layers = (bounds, [1.0, 2.0, 3.0, 0.5, 1.0, 2.0, 0.25, 1.5], [1.0, 0.0, 1.0, 2.0, 1.0, 0.0, 1.0, 3.0])
    for use_layers in (None, layers):
        _simple(n_el, lam, n, 12 * (lam // n) * fuse_t, grad_dtype, model="lognormal", fuse_t=fuse_t, lazy=fuse_t > 1,
                options={P.PS_OPT_KERNEL: P.PS_KERNEL_BULK, P.PS_OPT_BULK_TILE: 2048 if fuse_t < 8 else 0},
                layers=use_layers, mirror=True)
        assert run_pair.launches["bulk"] == 12 and run_pair.launches["vector"] == 0


def test_bulk_copy_kernel_refuses_what_it_cannot_stage():
    """More than 16 gradients per launch, or a pointer that is not 16-byte aligned: an error, not a fallback."""
    dev = torch.device("cuda", 0)
    ps = P.ParameterServer(8192, 17, 1, 0.01, device=dev)
    ps.set_option(P.PS_OPT_KERNEL, P.PS_KERNEL_BULK)
    ps.init_weights(torch.zeros(8192))
    g = torch.zeros(8192, device=dev)
    for l in range(17):
        ps.push_gradient(l, g, 0)
    with pytest.raises(P.SoftsyncError) as e:
        ps.apply_update()
    assert e.value.status == P.PS_ERR_INVALID_ARG and ps.timestamps() == (0, 1)
    ps.set_option(P.PS_OPT_KERNEL, P.PS_KERNEL_AUTO)
    assert ps.apply_update() == 1
    ps.destroy()
    ps = P.ParameterServer(8192, 1, 1, 0.01, grad_dtype="bf16", device=dev)
    ps.set_option(P.PS_OPT_KERNEL, P.PS_KERNEL_BULK)
    ps.init_weights(torch.zeros(8192))
    buf = torch.zeros(8192 + 8, dtype=torch.bfloat16, device=dev)
    ps.push_gradient(0, buf[4:4 + 8192], 0)                 # 8-byte aligned: fine for the vector kernel only
    with pytest.raises(P.SoftsyncError):
        ps.apply_update()
    ps.set_option(P.PS_OPT_KERNEL, P.PS_KERNEL_VECTOR)
    assert ps.apply_update() == 1 and ps.get_option(P.PS_OPT_LAST_KERNEL) == P.PS_KERNEL_VECTOR
    ps.destroy()


def test_bulk_copy_kernel_wait_runs_out_and_is_reported():
    """A copy barrier that never completes (one block is told to expect 16 bytes that nothing sends): the
    block's bounded wait runs out, the kernel returns by itself, the host reads the status record, and
    the context stays usable: after re-initialising, the same server matches the reference."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    n_el, lam = 64 * 1024 + 7, 2
    w0 = G.initial_weights(layouts.flat(n_el), 51)
    ps = P.ParameterServer(n_el, lam, 1, 0.01, 0.9, 5e-4, device=dev)
    ps.set_option(P.PS_OPT_KERNEL, P.PS_KERNEL_BULK)
    ps.set_option(P.PS_OPT_BULK_TILE, 1024)
    ps.set_option(P.PS_OPT_BULK_WAIT_LIMIT, 2000)
    ps.init_weights(w0.to(dev))
    grads = [G.gradient(51, l, 0, n_el, 1e-3, device=dev) for l in range(lam)]
    ps.set_option(P.PS_OPT_BULK_SELFTEST, 1)
    for l in range(lam):
        ps.push_gradient(l, grads[l], 0)
    assert ps.apply_update() == 1                          # the launch itself is fine
    with pytest.raises(P.SoftsyncError) as e:
        ps.synchronize()
    assert e.value.status == P.PS_ERR_DEVICE_WAIT
    code, block, tile, stage = ps.kernel_status()
    assert (code, block, tile, stage) == (1, 0, 0, 0)
    assert ps.get_option(P.PS_OPT_BULK_SELFTEST) == 0      # one launch only
    torch.cuda.synchronize()                               # the context is intact
    ps.init_weights(w0.to(dev))                            # theta and v were partly updated: start again
    ps.synchronize()
    assert ps.kernel_status()[0] == 0
    ref = R.ReferencePS(n_el, lam, 1, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    for u in range(3):
        ts = ps.pull_weights()
        for l in range(lam):
            ref.pull(l)
        for l in range(lam):
            g = G.gradient(51, l, u, n_el, 1e-3, device=dev)
            ref.push(l, as_reference_grad(g))
            ps.push_gradient(l, g, ts)
        assert ps.apply_update() == 1
    ps.synchronize()
    assert np.array_equal(ps.w.cpu().numpy(), ref.state()[0].astype(np.float32))
    assert np.array_equal(ps.v.cpu().numpy(), ref.state()[1].astype(np.float32))
    ps.destroy()


@pytest.mark.parametrize("rho", [0.5, 0.9])
@pytest.mark.parametrize("grad_dtype,fuse_t", [("fp32", 1), ("bf16", 4)])
def test_exponential_penalty_matches_reference(rho, grad_dtype, fuse_t):
    """alpha = alpha0 * rho^tau (the rule Section 1 contrasts with Eq. 3) on an Exp(1) arrival trace with
    staleness up to several tens."""
    kinds, learners = R.simulate_arrivals("exp", 12, 240, 61)
    n_el = 50001
    w0 = G.initial_weights(layouts.flat(n_el), 61)
    w, v, log, refs = run_pair(n_el, 12, 6, 0.02, 0.9, 5e-4, "exp_staleness", grad_dtype, 1e-3, kinds, learners, w0, 61,
                               fuse_t=fuse_t, lazy=fuse_t > 1, penalty_base=rho)
    assert_parity(w, v, log, refs, TOL_BF16 if grad_dtype == "bf16" else TOL_FP32)
    assert log["tau"].max() >= 5 and np.array_equal(log["sigma"], log["tau"])
    assert len(np.unique(log["scale"])) >= 5


@pytest.mark.parametrize("grad_dtype,options,misalign", [
    ("fp32", None, 0), ("bf16", None, 0), ("fp32", None, 1), ("fp32", {P.PS_OPT_KERNEL: P.PS_KERNEL_BULK}, 0)])
def test_vanishing_scales_keep_their_denormals(grad_dtype, options, misalign):
    """The degenerate end of the exponential penalty: a learner that never pulls again pushes gradients whose
    staleness runs from 118 to 152, so that 0.5^tau passes through the smallest normal fp32 numbers, the
    denormals and zero.  With momentum 0, decay 0 and theta_0 = 0 the state is made of nothing but those
    products, and the momentum right after such an update is the bare product s*g: it must not be flushed to
    zero on the GPU (packed and scalar multiplies alike).  The state is compared after every single update."""
    from tests.helpers import PUSH
    lam, n_el = 2, 8197
    kinds, learners = [PULL, PULL], [0, 1]
    for u in range(153):
        if u >= 118 and u % 2 == 0:                     # the stale learner: timestamp 0 for ever
            kinds.append(PUSH); learners.append(1)
        kinds += [PUSH, PULL]; learners += [0, 0]
    kinds, learners = np.asarray(kinds, dtype=np.int32), np.asarray(learners, dtype=np.int32)
    w0 = torch.zeros(n_el)
    w, v, log, refs = run_pair(n_el, lam, lam, 1.0, 0.0, 0.0, "exp_staleness", grad_dtype, 1.0, kinds, learners, w0, 97,
                               penalty_base=0.5, options=options, misalign=misalign, precisions=(32,),
                               checkpoints=1000)      # v after EVERY update: the stale ones leave it denormal
    assert_parity(w, v, log, refs, TOL_FP32)
    stale = log[log["learner"] == 1]
    tiny = np.finfo(np.float32).tiny
    assert stale["tau"].min() >= 118 and stale["tau"].max() >= 150
    assert ((stale["scale"] > 0) & (stale["scale"] < tiny)).any() and (stale["scale"] == 0).any()    # denormal and zero scales
    assert (stale["scale"] >= tiny).any()


@pytest.mark.parametrize("grad_dtype,fuse_t,kernel", [("fp32", 1, "auto"), ("bf16", 2, "auto"), ("fp32", 2, "scalar"),
                                                     ("fp32", 1, "bulk"), ("bf16", 1, "bulk")])
def test_special_values_propagate_like_the_reference(grad_dtype, fuse_t, kernel):
    """Infinities, NaNs, signed zeros, denormals and the largest finite values in gradients and weights: the
    same elements become NaN or infinite on both sides, every other element agrees bit for bit (signed zeros
    included: the comparison is on the bit patterns, NaN payloads excepted)."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    tdt = torch.bfloat16 if grad_dtype == "bf16" else torch.float32
    n_el, lam = 4096 + 5, 2
    specials = torch.tensor([float("inf"), float("-inf"), float("nan"), -0.0, 0.0, 1e-42, -1e-42, 3.0e38, -3.0e38,
                             1.17549435e-38, 1.0, -1.0])
    w0 = G.initial_weights(layouts.flat(n_el), 5)
    w0[100:100 + specials.numel()] = specials
    w0[n_el - 3:] = torch.tensor([-0.0, 3.0e38, 1e-42])                        # the ragged tail too
    ps = P.ParameterServer(n_el, lam, 1, 0.5, 0.9, 5e-4, grad_dtype=grad_dtype, fuse_t=fuse_t, device=dev)
    ps.set_option(P.PS_OPT_KERNEL, P.binding.KERNELS[kernel])
    ps.init_weights(w0.to(dev))
    ref = R.ReferencePS(n_el, lam, 1, 0.5, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    pending = 0
    for u in range(4):
        ts = ps.pull_weights()
        for l in range(lam):
            ref.pull(l)
            g = G.gradient(5, l, u, n_el, 1e-2, dtype=torch.float32, device=dev)
            g[(7 + 13 * u) % 64: (7 + 13 * u) % 64 + specials.numel()] = specials.to(dev)     # over ordinary weights
            g[100 + u: 100 + u + 4] = specials[u: u + 4].to(dev)                           # over special weights
            g[n_el - 2] = float("inf") if u == 2 else -0.0
            if u == 3:
                g[200], g[201] = float("inf"), float("-inf")                                 # still infinite at the end
            g = g.to(tdt)
            ref.push(l, as_reference_grad(g))
            pending += ps.push_gradient(l, g, ts)
        if pending >= fuse_t:
            pending -= ps.apply_update()
    ps.flush(); ps.synchronize()
    for got, want in zip((ps.w.cpu().numpy(), ps.v.cpu().numpy()), ref.state()):
        want = want.astype(np.float32)
        assert np.array_equal(np.isnan(got), np.isnan(want))
        ok = ~np.isnan(want)
        assert np.array_equal(got.view(np.uint32)[ok], want.view(np.uint32)[ok])
        assert np.isnan(want).any() and np.isinf(want[ok]).any()                 # the case did what it is for
    ps.destroy()


def caffe_style_multipliers(layout):
    """Rate x1 / decay x1 for weights, rate x2 / decay x0 for biases (the usual setting of the Caffe models
    that Section 4.1's networks follow)."""
    bounds = [seg.offset for seg in layout.segments] + [layout.num_params]
    return (bounds, [2.0 if seg.is_bias else 1.0 for seg in layout.segments],
            [0.0 if seg.is_bias else 1.0 for seg in layout.segments])


@pytest.mark.parametrize("kernel", ["vector", "scalar", "bulk"])
def test_layer_multipliers_on_the_small_network(kernel):
    """Config 1 (89,578 elements, N mod 4 = 2, layer boundaries at every residue mod 4) with per-layer
    multipliers, every element compared."""
    cfg = configs.TINY_SOFTSYNC
    layout = cfg.layout()
    worst, log = run_config(cfg, num_pushes=160, layers=caffe_style_multipliers(layout),
                            options={P.PS_OPT_KERNEL: P.binding.KERNELS[kernel], P.PS_OPT_BULK_TILE: 512})
    assert run_pair.launches[kernel] == 40
    worst, log = run_config(configs.PURE_ASYNC, num_pushes=300, layers=caffe_style_multipliers(layout), fuse_t=8, lazy=True,
                            options={P.PS_OPT_KERNEL: P.binding.KERNELS[kernel]})


@pytest.mark.parametrize("grad_dtype,fuse_t,lam,n", [("fp32", 1, 6, 2), ("bf16", 3, 4, 4), ("fp32", 16, 40, 2), ("bf16", 1, 20, 1)])
def test_layer_boundaries_anywhere(grad_dtype, fuse_t, lam, n):
    """Boundaries inside fragments, empty layers, a one-element layer, a frozen layer (rate x0), layers that
    end in the ragged tail; all-ones multipliers give the bits of a server without a table."""
    n_el = 20003
    bounds = [0, 1, 1, 6, 7, 4098, 4099, 4099, 9001, 15002, 20000, 20002, n_el]
    lm = [1.0, 3.0, 0.5, 2.0, 1.0, 0.0, 1.0, 2.0, 0.125, 1.0, 4.0, 1.5]
    dm = [1.0, 1.0, 0.0, 2.0, 1.0, 1.0, 5.0, 0.0, 1.0, 0.5, 1.0, 0.0]
    pushes = 10 * (lam // n) * min(fuse_t, 4)
    a = _simple(n_el, lam, n, pushes, grad_dtype, model="lognormal", fuse_t=fuse_t, lazy=fuse_t > 1, layers=(bounds, lm, dm), mirror=True)
    assert run_pair.launches["vector"] > 0 and run_pair.launches["scalar"] == 0
    ones = _simple(n_el, lam, n, pushes, grad_dtype, model="lognormal", fuse_t=fuse_t, lazy=fuse_t > 1,
                   layers=([0, 5, n_el], [1.0, 1.0], [1.0, 1.0]))
    none = _simple(n_el, lam, n, pushes, grad_dtype, model="lognormal", fuse_t=fuse_t, lazy=fuse_t > 1)
    assert np.array_equal(ones[0], none[0]) and np.array_equal(ones[1], none[1])
    assert not np.array_equal(a[0], none[0])
    w0 = G.initial_weights(layouts.flat(n_el), 77).numpy()
    assert np.array_equal(a[0][4098:4099], w0[4098:4099])          # the frozen layer did not move


@pytest.mark.parametrize("grad_dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("c", [1, 4, 16, 64])
def test_sweep_point_with_uniform_staleness(c, grad_dtype):
    """The bandwidth sweep's smallest size (2^20 flat elements): c gradients per update, each pushed with
    a timestamp that makes its staleness uniform in [1, 2c] (clamped while the clock is still young)."""
    from tests.gpu_harness import as_reference_grad, assert_logs_equal
    dev = torch.device("cuda", 0)
    n_el, updates = 1 << 20, 6
    tdt = torch.bfloat16 if grad_dtype == "bf16" else torch.float32
    rng = np.random.default_rng(c)
    w0 = G.initial_weights(layouts.flat(n_el), 11)
    ps = P.ParameterServer(n_el, c, 1, 0.01, 0.9, 5e-4, "inv_staleness", grad_dtype, device=dev)
    ps.init_weights(w0.to(dev))
    refs = {prec: R.ReferencePS(n_el, c, 1, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, prec) for prec in (32, 64)}
    for r in refs.values():
        r.set_weights(w0.numpy())
    for u in range(updates):
        now = ps.pull_weights()
        assert now == u == refs[32].timestamp
        for l in range(c):
            ts = max(0, now - int(rng.integers(1, 2 * c + 1)))
            g = G.gradient(11, l, u, n_el, 1e-4, dtype=tdt, device=dev)
            ps.push_gradient(l, g, ts)
            for r in refs.values():
                r.push(l, as_reference_grad(g), timestamp=ts)
        assert ps.apply_update() == 1
    ps.synchronize()
    w, v, log = ps.w.cpu().numpy(), ps.v.cpu().numpy(), ps.update_log()
    ps.destroy()
    out = {prec: (*r.state(), r.log()) for prec, r in refs.items()}
    assert_parity(w, v, log, out, TOL_BF16 if grad_dtype == "bf16" else TOL_FP32)
    assert log["sigma"].max() > 1 or c == 1


def test_rate_schedule_matches_reference():
    """alpha0 lowered in steps while gradients are in flight (Section 4.3): a gradient keeps the rate
    that was in force when it was pushed, also across fused passes."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    n_el, lam, n = 50003, 6, 2
    kinds, learners = R.simulate_arrivals("lognormal", lam, 90, 6)
    w0 = G.initial_weights(layouts.flat(n_el), 6)
    ps = P.ParameterServer(n_el, lam, n, 0.04, 0.9, 5e-4, fuse_t=4, device=dev)
    ps.init_weights(w0.to(dev))
    refs = {prec: R.ReferencePS(n_el, lam, n, 0.04, 0.9, 5e-4, R.MOD_INV_STALENESS, prec) for prec in (32, 64)}
    for r in refs.values():
        r.set_weights(w0.numpy())
    pulled, counts, pushes, rate = {}, {}, 0, 0.04
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = ps.pull_weights()
            for r in refs.values():
                assert r.pull(l) == pulled[l]
            continue
        if pushes % 11 == 5:
            rate = rate * 0.5
            ps.set_alpha0(rate)
            for r in refs.values():
                r.set_alpha0(rate)
        b = counts.get(l, 0); counts[l] = b + 1
        g = G.gradient(6, l, b, n_el, 1e-3, device=dev)
        for r in refs.values():
            r.push(l, as_reference_grad(g))
        ps.push_gradient(l, g, pulled[l])
        pushes += 1
        if ps.timestamps()[1] - ps.timestamps()[0] >= 4:
            ps.apply_update()
    ps.flush(); ps.synchronize()
    w, v, log = ps.w.cpu().numpy(), ps.v.cpu().numpy(), ps.update_log()
    ps.destroy()
    assert_parity(w, v, log, {prec: (*r.state(), r.log()) for prec, r in refs.items()}, TOL_FP32)
    assert len(np.unique(log["scale"] * log["sigma"])) > 3


@pytest.mark.parametrize("grad_dtype,fuse_t", [("fp32", 1), ("bf16", 4)])
def test_overlapped_launch_gives_the_same_bits(grad_dtype, fuse_t):
    """Update kernels launched as programmatic dependents (each may start while the previous one drains)
    produce exactly what ordinary launches produce.  All gradients exist before the first update."""
    dev = torch.device("cuda", 0)
    n_el, lam, n, pushes = 2_000_003, 4, 2, 48
    tdt = torch.bfloat16 if grad_dtype == "bf16" else torch.float32
    kinds, learners = R.simulate_arrivals("exp", lam, pushes, 12)
    w0 = G.initial_weights(layouts.flat(n_el), 12)
    grads = {}
    counts = {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 1:
            b = counts.get(l, 0); counts[l] = b + 1
            grads[(l, b)] = G.gradient(12, l, b, n_el, 1e-3, dtype=tdt, device=dev)
    torch.cuda.synchronize()
    results = []
    for overlap in (0, 1):
        ps = P.ParameterServer(n_el, lam, n, 0.01, 0.9, 5e-4, grad_dtype=grad_dtype, fuse_t=fuse_t, device=dev)
        ps.set_option(P.PS_OPT_OVERLAP_LAUNCH, overlap)
        assert ps.get_option(P.PS_OPT_OVERLAP_LAUNCH) == overlap
        ps.init_weights(w0.to(dev))
        torch.cuda.synchronize()
        pulled, counts, ready = {}, {}, 0
        for k, l in zip(kinds.tolist(), learners.tolist()):
            if k == 0:
                pulled[l] = ps.pull_weights()
                continue
            b = counts.get(l, 0); counts[l] = b + 1
            ready += ps.push_gradient(l, grads[(l, b)], pulled[l])
            if ready >= fuse_t:
                ready -= ps.apply_update()
        ps.flush(); ps.synchronize()
        results.append((ps.w.cpu().numpy().copy(), ps.v.cpu().numpy().copy(), ps.update_log()))
        ps.destroy()
    assert np.array_equal(results[0][0], results[1][0]) and np.array_equal(results[0][1], results[1][1])
    assert np.array_equal(results[0][2], results[1][2])
    ref = R.ReferencePS(n_el, lam, n, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    from tests.gpu_harness import as_reference_grad
    from tests.helpers import replay_reference
    replay_reference(ref, kinds, learners, lambda l, b: as_reference_grad(grads[(l, b)]))
    from tests.gpu_harness import assert_logs_equal
    for w, v, log in results:
        assert np.array_equal(w, ref.state()[0].astype(np.float32)) and np.array_equal(v, ref.state()[1].astype(np.float32))
        assert_logs_equal(log, ref.log())


@pytest.mark.parametrize("grad_dtype,fuse_t", [("fp32", 1), ("bf16", 2)])
def test_overlapped_launch_with_host_gradients_in_recycled_slots(grad_dtype, fuse_t):
    """The arrangement the benchmark's end-to-end leg runs: programmatic dependent launches while every
    gradient arrives from pinned host memory into 2*c*T staging slots that are reused generation after
    generation, the copy of the next gradients enqueued right behind the kernel that still reads the
    previous ones.  Against the reference, every element."""
    from tests.gpu_harness import as_reference_grad, assert_logs_equal
    dev = torch.device("cuda", 0)
    n_el, lam, n = 2_000_003, 6, 2
    c = lam // n
    tdt = torch.bfloat16 if grad_dtype == "bf16" else torch.float32
    pushes = 2 * c * fuse_t * 5                              # five generations of every slot
    kinds, learners = R.simulate_arrivals("uniform", lam, pushes, 33)
    w0 = G.initial_weights(layouts.flat(n_el), 33)
    ref = R.ReferencePS(n_el, lam, n, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    ps = P.ParameterServer(n_el, lam, n, 0.01, 0.9, 5e-4, grad_dtype=grad_dtype, fuse_t=fuse_t, device=dev)
    ps.set_option(P.PS_OPT_OVERLAP_LAUNCH, 1)
    ps.bind_staging(2 * c * fuse_t)
    ps.init_weights(w0.to(dev))
    w_host = torch.empty(n_el).pin_memory()
    pulled, counts, ready = {}, {}, 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = ps.pull_weights()
            assert ref.pull(l) == pulled[l]
            continue
        b = counts.get(l, 0); counts[l] = b + 1
        g = G.gradient(33, l, b, n_el, 1e-3, dtype=tdt).pin_memory()
        ref.push(l, as_reference_grad(g))
        ready += ps.push_gradient(l, g, pulled[l])           # host tensor: cudaMemcpyAsync into a staging slot
        if ready >= fuse_t:
            ready -= ps.apply_update()
            ps.pull_weights(w_host, non_blocking=True)       # the read-back of the e2e leg, overlapping the next uploads
    ps.flush(); ps.synchronize()
    assert ps.get_option(P.PS_OPT_LAUNCHES_VECTOR) == pushes // c // fuse_t
    assert np.array_equal(ps.w.cpu().numpy(), ref.state()[0].astype(np.float32))
    assert np.array_equal(ps.v.cpu().numpy(), ref.state()[1].astype(np.float32))
    assert np.array_equal(w_host.numpy(), ps.w.cpu().numpy())
    assert_logs_equal(ps.update_log(), ref.log())
    ps.destroy()


@pytest.mark.parametrize("grad_dtype,fuse_t,n_el,misalign", [
    ("fp32", 1, 70003, 0), ("bf16", 4, 70005, 0), ("fp32", 3, 9999, 1), ("bf16", 1, 4097, 3), ("fp32", 1, 3, 0)])
def test_bf16_weight_mirror_tracks_the_weights(grad_dtype, fuse_t, n_el, misalign):
    """The bf16 copy written by the update pass equals the reference's weights rounded to bf16, bit for bit,
    after set-up, after every update (fused or not, vector or scalar kernel) and through the bf16 pull."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    tdt = torch.bfloat16 if grad_dtype == "bf16" else torch.float32
    lam, n = 6, 3
    kinds, learners = R.simulate_arrivals("exp", lam, 30, 8)
    w0 = G.initial_weights(layouts.flat(n_el), 8)
    ref = R.ReferencePS(n_el, lam, n, 0.05, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    ps = P.ParameterServer(n_el, lam, n, 0.05, 0.9, 5e-4, grad_dtype=grad_dtype, fuse_t=fuse_t, device=dev)
    ps.init_weights(w0.to(dev))
    guard = torch.full((n_el + misalign + 64,), 7.0, dtype=torch.bfloat16, device=dev)
    mirror = ps.bind_weight_mirror(guard[misalign:misalign + n_el])

    def bits(t):
        return t.cpu().view(torch.int16).numpy().view(np.uint16)

    assert np.array_equal(bits(mirror), ref.weights_bf16())               # filled when bound
    pulled, counts, ready = {}, {}, 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = ps.pull_weights()
            ref.pull(l)
            continue
        b = counts.get(l, 0); counts[l] = b + 1
        g = G.gradient(8, l, b, n_el, 1e-2, dtype=tdt, device=dev)
        fired = ref.push(l, as_reference_grad(g))
        ready += ps.push_gradient(l, g, pulled[l])
        if ready >= fuse_t:
            ready -= ps.apply_update()
            if ready == 0:
                assert np.array_equal(bits(mirror), ref.weights_bf16())
    out = torch.empty(n_el, dtype=torch.bfloat16, device=dev)
    assert ps.pull_weights(out) == ref.timestamp                              # flushes, then copies the mirror
    assert np.array_equal(bits(out), ref.weights_bf16())
    assert np.array_equal(ps.w[:n_el].cpu().numpy(), ref.state()[0].astype(np.float32))
    assert (guard[:misalign] == 7.0).all() and (guard[misalign + n_el:] == 7.0).all()
    ps.init_weights(w0.to(dev))                                               # re-initialising refreshes it
    ref2 = R.round_to_bf16(w0.numpy())
    assert np.array_equal(bits(mirror), ref2)
    ps.destroy()


@pytest.mark.parametrize("grad_dtype,fuse_t,kernel,misalign", [
    ("fp32", 1, "auto", 0), ("bf16", 8, "auto", 0), ("fp32", 2, "auto", 1), ("fp32", 1, "bulk", 0), ("bf16", 4, "scalar", 0)])
def test_weight_replicas_are_written_by_the_update_pass(grad_dtype, fuse_t, kernel, misalign):
    """ps_bind_weight_replicas: three further fp32 buffers hold theta after set-up and after every update,
    bit for bit the reference's weights; nothing outside them is touched; a misaligned replica takes the
    scalar kernel; unbinding stops the writes."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    tdt = torch.bfloat16 if grad_dtype == "bf16" else torch.float32
    lam, n, n_el = 8, 8, 9 * 4096 + 77
    kinds, learners = R.simulate_arrivals("exp", lam, 48, 23)
    w0 = G.initial_weights(layouts.flat(n_el), 23)
    ref = R.ReferencePS(n_el, lam, n, 0.05, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    ps = P.ParameterServer(n_el, lam, n, 0.05, 0.9, 5e-4, grad_dtype=grad_dtype, fuse_t=fuse_t, device=dev)
    ps.set_option(P.PS_OPT_KERNEL, P.binding.KERNELS[kernel])
    ps.init_weights(w0.to(dev))
    guards = [torch.full((n_el + 72,), 7.0, device=dev) for _ in range(3)]
    offs = [8, 8 + misalign, 8]
    reps = [gd[o:o + n_el] for gd, o in zip(guards, offs)]
    ps.bind_weight_replicas(reps)
    want = lambda: ref.state()[0].astype(np.float32)
    for r in reps:
        assert np.array_equal(r.cpu().numpy(), want())                       # filled when bound
    pulled, counts, ready = {}, {}, 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = ps.pull_weights(); ref.pull(l)
            continue
        b = counts.get(l, 0); counts[l] = b + 1
        g = G.gradient(23, l, b, n_el, 1e-2, dtype=tdt, device=dev)
        ref.push(l, as_reference_grad(g))
        ready += ps.push_gradient(l, g, pulled[l])
        if ready >= fuse_t:
            ready -= ps.apply_update()
            if ready == 0:
                for r in reps:
                    assert np.array_equal(r.cpu().numpy(), want())
    ps.flush(); ps.synchronize()
    assert ps.get_option(P.PS_OPT_LAST_KERNEL) == (P.PS_KERNEL_SCALAR if misalign or kernel == "scalar" else
                                                   P.binding.KERNELS[kernel] or P.PS_KERNEL_VECTOR)
    assert np.array_equal(ps.w.cpu().numpy(), want())
    for gd, o, r in zip(guards, offs, reps):
        assert np.array_equal(r.cpu().numpy(), want())
        assert (gd[:o] == 7.0).all() and (gd[o + n_el:] == 7.0).all()
    big = torch.zeros(2 * n_el + 8, device=dev)
    for bad in ([big[:n_el], big[4:4 + n_el]], [big[:n_el], big[:n_el]], [ps.w], [big[:n_el], ps.v]):
        with pytest.raises(P.SoftsyncError) as e:                            # overlapping one another, theta or v
            ps.bind_weight_replicas(bad)
        assert e.value.status == P.PS_ERR_INVALID_ARG
    ps.bind_weight_replicas([])                                              # unbound: later updates leave them alone
    before = reps[0].clone()
    ts = ps.pull_weights()
    for l in range(lam):
        ps.push_gradient(l, G.gradient(23, l, 99, n_el, 1e-2, dtype=tdt, device=dev), ts)
    ps.flush(); ps.synchronize()
    assert torch.equal(reps[0], before) and not torch.equal(ps.w, before)
    ps.destroy()


def test_shards_assemble_the_weights_in_every_replica_buffer():
    """The all-gather of the sharded server, fused into the update: three shards over contiguous ranges, and two
    full-length buffers standing for two GPUs' copies of the weights.  Every shard's update kernel stores its
    range into both; after the updates both buffers hold the reference's whole weight vector, without any copy
    or gather at pull time."""
    from paper_1511_05950_b200.sharded import shard_bounds
    from tests.gpu_harness import as_reference_grad
    from tests.helpers import replay_reference
    dev = torch.device("cuda", 0)
    n_el, lam, n, world = 100003, 6, 2, 3
    bounds = shard_bounds(n_el, world)
    kinds, learners = R.simulate_arrivals("lognormal", lam, 60, 31)
    w0 = G.initial_weights(layouts.flat(n_el), 31).to(dev)
    buffers = [torch.zeros(n_el, device=dev) for _ in range(2)]
    shards = []
    for a, b in zip(bounds[:-1], bounds[1:]):
        sh = P.ParameterServer(b - a, lam, n, 0.02, 0.9, 5e-4, fuse_t=2, device=dev)
        sh.init_weights(w0[a:b].contiguous())
        sh.bind_weight_replicas([buf[a:b] for buf in buffers])
        shards.append((a, b, sh))
    assert all(torch.equal(buf, w0) for buf in buffers)
    ref = R.ReferencePS(n_el, lam, n, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.cpu().numpy())
    pulled, counts = {}, {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = shards[0][2].pull_weights()
            assert all(sh.pull_weights() == pulled[l] for _, _, sh in shards) and ref.pull(l) == pulled[l]
            continue
        c_ = counts.get(l, 0); counts[l] = c_ + 1
        g = G.gradient(31, l, c_, n_el, 1e-3, device=dev)
        ref.push(l, as_reference_grad(g))
        for a, b, sh in shards:
            if sh.push_gradient(l, g[a:b], pulled[l]):
                sh.apply_update()
        if ref.timestamp % 5 == 0:
            torch.cuda.synchronize()
            if all(sh.timestamps()[0] == ref.timestamp for _, _, sh in shards):
                for buf in buffers:
                    assert np.array_equal(buf.cpu().numpy(), ref.state()[0].astype(np.float32))
    for _, _, sh in shards:
        sh.flush()
    torch.cuda.synchronize()
    for buf in buffers:
        assert np.array_equal(buf.cpu().numpy(), ref.state()[0].astype(np.float32))
    for _, _, sh in shards:
        sh.destroy()


def test_bf16_pull_needs_a_mirror():
    dev = torch.device("cuda", 0)
    ps = P.ParameterServer(64, 1, 1, 0.1, device=dev)
    ps.init_weights(torch.zeros(64))
    out = torch.empty(64, dtype=torch.bfloat16, device=dev)
    with pytest.raises(P.SoftsyncError) as e:
        ps.pull_weights(out)
    assert e.value.status == P.PS_ERR_NO_STATE
    ps.destroy()


def test_contiguous_shards_need_no_synchronisation():
    """The paper shards its parameter server and the shards never talk to each other (Section 2.3).
    Three servers over contiguous ranges of one vector, fed the same pushes, give bit for bit the
    state of one server over the whole vector, and their clocks and logs stay in lock-step."""
    dev = torch.device("cuda", 0)
    n_el, lam, n = 100003, 6, 2
    bounds = [0, 33336, 70004, n_el]                       # ragged, differently aligned shard starts
    kinds, learners = R.simulate_arrivals("lognormal", lam, 60, 14)
    w0 = G.initial_weights(layouts.flat(n_el), 14).to(dev)
    whole = P.ParameterServer(n_el, lam, n, 0.02, 0.9, 5e-4, fuse_t=2, device=dev)
    whole.init_weights(w0)
    wbuf, vbuf = torch.empty(n_el, device=dev), torch.empty(n_el, device=dev)
    shards = []
    for a, b in zip(bounds[:-1], bounds[1:]):
        sh = P.ParameterServer(b - a, lam, n, 0.02, 0.9, 5e-4, fuse_t=2, device=dev, state=(wbuf[a:b], vbuf[a:b]))
        sh.init_weights(w0[a:b].contiguous())
        shards.append((a, b, sh))
    shards[1][2].bind_staging(2 * (lam // n) * 2)          # the middle shard receives into its own slots
    pulled, counts = {}, {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = whole.pull_weights()
            assert all(sh.pull_weights() == pulled[l] for _, _, sh in shards)
            continue
        c_ = counts.get(l, 0); counts[l] = c_ + 1
        g = G.gradient(14, l, c_, n_el, 1e-3, device=dev)
        whole.push_gradient(l, g, pulled[l])
        for a, b, sh in shards:
            if sh is shards[1][2]:                         # scattered push: the learner writes its slice straight
                sid, slot = sh.acquire_slot()              # into a receive slot of the shard that owns the range
                slot.copy_(g[a:b])
                sh.push_slot(l, sid, pulled[l])
            else:
                sh.push_gradient(l, g[a:b], pulled[l])     # slice a of the same gradient goes to shard a
        if whole.timestamps()[1] - whole.timestamps()[0] >= 2:
            whole.apply_update()
            for _, _, sh in shards:
                sh.apply_update()
    whole.flush()
    for _, _, sh in shards:
        sh.flush()
    torch.cuda.synchronize()
    assert torch.equal(whole.w, wbuf) and torch.equal(whole.v, vbuf)
    for _, _, sh in shards:
        assert sh.timestamps() == whole.timestamps()
        assert np.array_equal(sh.update_log(), whole.update_log())
    # and both are what the reference computes on the whole vector
    from tests.gpu_harness import as_reference_grad, assert_logs_equal
    from tests.helpers import replay_reference
    ref = R.ReferencePS(n_el, lam, n, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.cpu().numpy())
    replay_reference(ref, kinds, learners, lambda l, p: as_reference_grad(G.gradient(14, l, p, n_el, 1e-3, device=dev)))
    assert np.array_equal(wbuf.cpu().numpy(), ref.state()[0].astype(np.float32))
    assert np.array_equal(vbuf.cpu().numpy(), ref.state()[1].astype(np.float32))
    assert_logs_equal(whole.update_log(), ref.log())
    for _, _, sh in shards:
        sh.destroy()
    whole.destroy()


def test_checkpoint_and_resume_reproduce_the_uninterrupted_run():
    """Save theta, v and the exported protocol state on a group boundary, restore them into a fresh server,
    carry on: the final state equals the reference's uninterrupted run bit for bit."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    n_el, lam, n = 40009, 4, 2
    kinds, learners = R.simulate_arrivals("exp", lam, 64, 21)
    w0 = G.initial_weights(layouts.flat(n_el), 21)
    ref = R.ReferencePS(n_el, lam, n, 0.03, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    ps = P.ParameterServer(n_el, lam, n, 0.03, 0.9, 5e-4, device=dev)
    ps.init_weights(w0.to(dev))
    pulled, counts, pushes, resumed = {}, {}, 0, False
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == 0:
            pulled[l] = ps.pull_weights()
            assert ref.pull(l) == pulled[l]
            continue
        b = counts.get(l, 0); counts[l] = b + 1
        g = G.gradient(21, l, b, n_el, 1e-3, device=dev)
        ref.push(l, as_reference_grad(g))
        if ps.push_gradient(l, g, pulled[l]):
            ps.apply_update()
        pushes += 1
        if pushes == 30 and not resumed:
            ps.synchronize()
            saved = (ps.w.clone(), ps.v.clone(), ps.export_state())
            ps.destroy()
            ps = P.ParameterServer(n_el, lam, n, 0.03, 0.9, 5e-4, device=dev)
            ps.w.copy_(saved[0]); ps.v.copy_(saved[1])
            ps.import_state(saved[2])
            assert ps.timestamps() == (15, 15)
            resumed = True
    ps.flush(); ps.synchronize()
    w, v = ref.state()
    assert np.array_equal(ps.w.cpu().numpy(), w.astype(np.float32)) and np.array_equal(ps.v.cpu().numpy(), v.astype(np.float32))
    assert np.array_equal(ps.update_log(15)["tau"], ref.log()["tau"][30:])
    ps.destroy()


def test_hardsync_protocol_matches_reference():
    """Eq. 1 through the C ABI: rounds of one gradient per learner on the current weights."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    n_el, lam = 33333, 6
    w0 = G.initial_weights(layouts.flat(n_el), 16)
    ps = P.ParameterServer(n_el, lam, 1, 0.02, 0.9, 5e-4, device=dev)
    ps.set_option(P.PS_OPT_PROTOCOL, P.PS_PROTOCOL_HARDSYNC)
    ps.init_weights(w0.to(dev))
    refs = {prec: R.ReferencePS(n_el, lam, 1, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, prec) for prec in (32, 64)}
    for r in refs.values():
        r.set_weights(w0.numpy())
        r.set_hardsync()
    for rnd in range(8):
        ts = ps.pull_weights()
        assert ts == rnd
        for r in refs.values():
            for l in range(lam):
                r.pull(l)
        for l in np.random.default_rng(rnd).permutation(lam):
            g = G.gradient(16, int(l), rnd, n_el, 1e-3, device=dev)
            for r in refs.values():
                r.push(int(l), as_reference_grad(g))
            if ps.push_gradient(int(l), g, ts):
                ps.apply_update()
            elif l % 2 == 0:
                with pytest.raises(P.SoftsyncError) as e:
                    ps.push_gradient(int(l), g, ts)
                assert e.value.status == P.PS_ERR_BARRIER
    ps.synchronize()
    w, v, log = ps.w.cpu().numpy(), ps.v.cpu().numpy(), ps.update_log()
    ps.destroy()
    assert_parity(w, v, log, {prec: (*r.state(), r.log()) for prec, r in refs.items()}, TOL_FP32)
    assert (log["tau"] == 0).all()


def test_two_servers_on_their_own_streams():
    """Each server enqueues on the stream it was given; two servers on two streams run concurrently
    and independently, and each matches the reference."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    n_el, lam = 600011, 3
    streams = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    servers, refs, grads = [], [], []
    w0 = G.initial_weights(layouts.flat(n_el), 31)
    for k, st in enumerate(streams):
        with torch.cuda.stream(st):
            ps = P.ParameterServer(n_el, lam, 1, 0.01 * (k + 1), 0.9, 5e-4, device=dev)
            assert ps.get_option(P.PS_OPT_STREAM) == st.cuda_stream
            ps.init_weights(w0.to(dev))
            gs = [[G.gradient(31 + k, l, u, n_el, 1e-3, device=dev) for l in range(lam)] for u in range(6)]
        ref = R.ReferencePS(n_el, lam, 1, 0.01 * (k + 1), 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
        ref.set_weights(w0.numpy())
        servers.append(ps); refs.append(ref); grads.append(gs)
    torch.cuda.synchronize()
    for u in range(6):                                   # interleave the two servers' launches
        for k, st in enumerate(streams):
            with torch.cuda.stream(st):
                ts = servers[k].pull_weights()
                for l in range(lam):
                    servers[k].push_gradient(l, grads[k][u][l], ts)
                assert servers[k].apply_update() == 1
    for k, st in enumerate(streams):
        for u in range(6):
            for l in range(lam):
                refs[k].pull(l)
            for l in range(lam):
                refs[k].push(l, as_reference_grad(grads[k][u][l]))
        servers[k].synchronize()
        assert np.array_equal(servers[k].w.cpu().numpy(), refs[k].state()[0].astype(np.float32))
        assert np.array_equal(servers[k].v.cpu().numpy(), refs[k].state()[1].astype(np.float32))
        servers[k].destroy()


@pytest.mark.parametrize("grad_dtype", ["fp32", "bf16"])
def test_largest_launch_512_entries(grad_dtype):
    """c = 256 (the largest group) with two groups fused: 512 gradient pointers in one launch."""
    _simple(2051, 256, 1, 4 * 256, grad_dtype, model="uniform", fuse_t=16, lazy=True)


def test_zero_parameters():
    _simple(0, 4, 2, 12)


def test_constant_modulation_and_plain_rule():
    kinds, learners = R.simulate_arrivals("exp", 10, 60, 5)
    w0 = G.initial_weights(layouts.flat(5000), 5)
    for mod, m, wd in (("constant", 0.9, 5e-4), ("inv_staleness", 0.0, 0.0)):
        w, v, log, refs = run_pair(5000, 10, 5, 0.02, m, wd, mod, "fp32", 1e-3, kinds, learners, w0, 5)
        assert_parity(w, v, log, refs, TOL_FP32)


def test_guard_bands_stay_untouched():
    """State and gradients sit between poisoned guard regions; nothing outside [0, N) is written,
    and gradients are never written at all."""
    dev = torch.device("cuda", 0)
    for grad_dtype, tdt in (("fp32", torch.float32), ("bf16", torch.bfloat16)):
        for n_el in (16384 + 3, 999):
            pad = 1024
            wbuf = torch.full((n_el + 2 * pad,), 7.25, device=dev)
            vbuf = torch.full((n_el + 2 * pad,), -3.5, device=dev)
            ps = P.ParameterServer(n_el, 3, 1, 0.01, 0.9, 5e-4, grad_dtype=grad_dtype, device=dev,
                                   state=(wbuf[pad:pad + n_el], vbuf[pad:pad + n_el]))
            ps.init_weights(G.initial_weights(layouts.flat(n_el), 3).to(dev))
            grads = []
            for l in range(3):
                gb = torch.full((n_el + 2 * pad,), 1.5, dtype=tdt, device=dev)
                G.gradient(3, l, 0, n_el, 1e-3, dtype=tdt, device=dev, out=gb[pad:pad + n_el])
                grads.append((gb, gb.clone()))
                ps.push_gradient(l, gb[pad:pad + n_el], ps.pull_weights())
            assert ps.apply_update() == 1
            ps.synchronize()
            for buf, val in ((wbuf, 7.25), (vbuf, -3.5)):
                assert (buf[:pad] == val).all() and (buf[pad + n_el:] == val).all()
            for gb, before in grads:
                assert torch.equal(gb, before)
            ps.destroy()


def test_weight_pull_flushes_pending_groups_and_host_paths():
    """A pull that returns weights applies every complete group first; host push/pull agree with device ones."""
    dev = torch.device("cuda", 0)
    n_el, lam = 30011, 4
    w0 = G.initial_weights(layouts.flat(n_el), 9)
    results = []
    for host in (False, True):
        ps = P.ParameterServer(n_el, lam, 2, 0.01, 0.9, 5e-4, fuse_t=4, device=dev)
        ps.init_weights(w0 if host else w0.to(dev))
        if host:
            ps.bind_staging(2 * 3)
        ts = {l: ps.pull_weights() for l in range(lam)}
        for p in range(3):
            for l in range(2):
                g = G.gradient(9, l, p, n_el, 1e-3, device="cpu" if host else dev)
                if host:
                    g = g.pin_memory()
                ps.push_gradient(l, g, ts[l])
        assert ps.timestamps() == (0, 3)
        out = torch.empty(n_el, device="cpu" if host else dev)
        assert ps.pull_weights(out) == 3
        assert ps.timestamps() == (3, 3)
        ps.synchronize()
        results.append(out.cpu().numpy().copy())
        assert np.array_equal(results[-1], ps.w.cpu().numpy())
        ps.destroy()
    assert np.array_equal(results[0], results[1])
    ref = R.ReferencePS(n_el, lam, 2, 0.01, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    for l in range(lam):
        ref.pull(l)
    for p in range(3):
        for l in range(2):
            ref.push(l, G.gradient(9, l, p, n_el, 1e-3).numpy())
    assert np.array_equal(results[0], ref.state()[0].astype(np.float32))


def test_null_and_misaligned_gradient_pointers_are_rejected():
    import ctypes as C
    dev = torch.device("cuda", 0)
    ps = P.ParameterServer(64, 2, 1, 0.01, device=dev)
    assert P.ps_push_gradient(ps._h, 0, None, 0) == P.PS_ERR_INVALID_ARG
    g = torch.ones(66, device=dev)
    assert P.ps_push_gradient(ps._h, 0, g.data_ptr() + 2, 0) == P.PS_ERR_INVALID_ARG
    host = torch.ones(64)
    assert P.ps_push_gradient_host(ps._h, 0, host.data_ptr(), 0) == P.PS_ERR_NO_STATE     # no staging slots bound
    assert ps.timestamps() == (0, 0)
    ps.destroy()


def test_asynchronous_host_pull_orders_with_later_updates():
    """The non-blocking read-back returns the weights of its own timestamp even when more updates
    are enqueued right behind it."""
    dev = torch.device("cuda", 0)
    n_el = 3_000_017
    ps = P.ParameterServer(n_el, 1, 1, 0.05, 0.9, 5e-4, device=dev)
    ps.init_weights(G.initial_weights(layouts.flat(n_el), 4).to(dev))
    ps.bind_staging(4)
    snaps, expect = [], []
    for step in range(4):
        g = G.gradient(4, 0, step, n_el, 1e-3).pin_memory()
        ps.push_gradient(0, g, ps.pull_weights())
        ps.apply_update()
        expect.append(ps.w.clone())                     # stream-ordered device copy of theta_{step+1}
        out = torch.empty(n_el).pin_memory()
        assert ps.pull_weights(out, non_blocking=True) == step + 1
        snaps.append(out)
    ps.synchronize()
    for out, want in zip(snaps, expect):
        assert torch.equal(out, want.cpu())
    assert not torch.equal(snaps[0], snaps[3])
    ps.destroy()


def test_learners_write_into_server_owned_slots():
    """Gradients produced straight into receive slots (acquire, write, push) give the same bits as borrowed buffers."""
    dev = torch.device("cuda", 0)
    n_el, lam = 20011, 3
    w0 = G.initial_weights(layouts.flat(n_el), 41)
    out = []
    for use_slots in (False, True):
        ps = P.ParameterServer(n_el, lam, 1, 0.02, 0.9, 5e-4, device=dev)
        ps.init_weights(w0.to(dev))
        if use_slots:
            ps.bind_staging(lam + 1)
        for u in range(5):
            ts = ps.pull_weights()
            for l in range(lam):
                if use_slots:
                    sid, view = ps.acquire_slot()
                    G.gradient(41, l, u, n_el, 1e-3, device=dev, out=view)
                    if l == 0 and u == 0:                                   # a slot can be handed back unused
                        spare, _ = ps.acquire_slot()
                        ps.release_slot(spare)
                    fired = ps.push_slot(l, sid, ts)
                else:
                    fired = ps.push_gradient(l, G.gradient(41, l, u, n_el, 1e-3, device=dev), ts)
            assert fired and ps.apply_update() == 1
        ps.synchronize()
        out.append((ps.w.cpu().numpy().copy(), ps.v.cpu().numpy().copy()))
        ps.destroy()
    assert np.array_equal(out[0][0], out[1][0]) and np.array_equal(out[0][1], out[1][1])
    ref = R.ReferencePS(n_el, lam, 1, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    for u in range(5):
        for l in range(lam):
            ref.pull(l)
        for l in range(lam):
            ref.push(l, G.gradient(41, l, u, n_el, 1e-3).numpy())
    assert np.array_equal(out[1][0], ref.state()[0].astype(np.float32))
    assert np.array_equal(out[1][1], ref.state()[1].astype(np.float32))


@pytest.mark.parametrize("overlap", [0, 1])
def test_learner_fills_recycled_slots_from_its_own_stream(overlap):
    """A learner with its own stream and its own kernels writes gradients straight into receive slots.  With
    only c + 1 slots every slot is recycled update after update, so a write can meet the update kernel that is still
    reading the slot's previous gradient unless the learner's stream waits for that kernel (ps_slot_wait),
    and the update must wait for the learner's kernels (ps_slot_written).  PS_OPT_OVERLAP_LAUNCH is on in
    one variant: launches that consume learner-written slots must not fetch their gradients early."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    n_el, lam = 4_000_001, 2
    updates = 8                                              # 16 pushes through 3 slots: 5+ generations each
    w0 = G.initial_weights(layouts.flat(n_el), 43)
    ref = R.ReferencePS(n_el, lam, 1, 0.02, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    ps = P.ParameterServer(n_el, lam, 1, 0.02, 0.9, 5e-4, device=dev)
    ps.set_option(P.PS_OPT_OVERLAP_LAUNCH, overlap)
    ps.bind_staging(lam + 1)
    ps.init_weights(w0.to(dev))
    learner_stream = torch.cuda.Stream(dev)
    seen = set()
    for u in range(updates):
        ts = ps.pull_weights()
        for l in range(lam):
            assert ref.pull(l) == ts
        for l in range(lam):
            sid, view = ps.acquire_slot()
            seen.add(sid)
            ps.slot_wait(sid, learner_stream)                # after the kernel that read this slot last
            with torch.cuda.stream(learner_stream):
                G.gradient(43, l, u, n_el, 1e-3, device=dev, out=view)      # a chain of the learner's kernels
            ps.slot_written(sid, learner_stream)             # the server's stream waits for them
            fired = ps.push_slot(l, sid, ts)
            ref.push(l, G.gradient(43, l, u, n_el, 1e-3).numpy())
        assert fired and ps.apply_update() == 1              # no host synchronisation anywhere in the loop
    ps.synchronize()
    learner_stream.synchronize()
    assert lam <= len(seen) <= lam + 1                       # the pool hands back the slot freed last: each one
                                                             # is rewritten right behind the kernel that read it
    assert np.array_equal(ps.w.cpu().numpy(), ref.state()[0].astype(np.float32))
    assert np.array_equal(ps.v.cpu().numpy(), ref.state()[1].astype(np.float32))
    ps.destroy()


def test_stream_change_orders_after_work_on_the_old_stream():
    """Updates enqueued on the first stream finish before anything enqueued after PS_OPT_STREAM moves the
    server to another stream; weights and momentum overlapping in memory are refused."""
    from tests.gpu_harness import as_reference_grad
    dev = torch.device("cuda", 0)
    n_el = 3_000_001
    w0 = G.initial_weights(layouts.flat(n_el), 47)
    ref = R.ReferencePS(n_el, 1, 1, 0.05, 0.9, 5e-4, R.MOD_INV_STALENESS, 32)
    ref.set_weights(w0.numpy())
    ps = P.ParameterServer(n_el, 1, 1, 0.05, 0.9, 5e-4, device=dev)
    ps.init_weights(w0.to(dev))
    grads = [G.gradient(47, 0, u, n_el, 1e-3, device=dev) for u in range(8)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    for u in range(8):
        ps.set_option(P.PS_OPT_STREAM, streams[u % 2].cuda_stream)          # hop between two streams, no host sync
        ref.pull(0)
        ref.push(0, as_reference_grad(grads[u]))
        ps.push_gradient(0, grads[u], ps.pull_weights())
        assert ps.apply_update() == 1
    ps.synchronize()
    torch.cuda.synchronize()
    assert np.array_equal(ps.w.cpu().numpy(), ref.state()[0].astype(np.float32))
    assert np.array_equal(ps.v.cpu().numpy(), ref.state()[1].astype(np.float32))
    ps.destroy()
    buf = torch.zeros(100, device=dev)
    with pytest.raises(P.SoftsyncError):
        P.ParameterServer(64, 1, 1, 0.1, device=dev, state=(buf[:64], buf[32:96]))


def test_staging_slots_run_out():
    dev = torch.device("cuda", 0)
    ps = P.ParameterServer(64, 4, 1, 0.01, device=dev)
    ps.init_weights(torch.zeros(64))
    ps.bind_staging(2)
    g = torch.ones(64)
    ps.push_gradient(0, g, 0)
    ps.push_gradient(1, g, 0)
    with pytest.raises(P.SoftsyncError) as e:
        ps.push_gradient(2, g, 0)
    assert e.value.status == P.PS_ERR_QUEUE_FULL
    ps.destroy()


def test_kernel_timing_option_counts_launches():
    dev = torch.device("cuda", 0)
    ps = P.ParameterServer(1 << 16, 1, 1, 0.01, device=dev)
    ps.init_weights(torch.zeros(1 << 16))
    ps.set_option(P.PS_OPT_TIMING, 1)
    g = torch.ones(1 << 16, device=dev)
    for i in range(5):
        ps.push_gradient(0, g, i)
        ps.apply_update()
    ms, launches = ps.kernel_time()
    assert launches == 5 and ms > 0
    assert ps.kernel_time() == (0.0, 0)
    ps.destroy()
