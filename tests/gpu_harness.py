"""Drive the CUDA library and the reference with the same seeded inputs (GPU tests only)."""
from __future__ import annotations

import numpy as np
import torch

import paper_1511_05950_b200 as P
from oracle import reference as R
from tests.helpers import PULL, rel_l2
from workloads import generators as G

TORCH_DTYPE = {"fp32": torch.float32, "bf16": torch.bfloat16}


def as_reference_grad(g: torch.Tensor) -> np.ndarray:
    """Device gradient -> what the reference's push takes (fp32 values or bf16 bit patterns)."""
    g = g.detach().cpu()
    if g.dtype == torch.bfloat16:
        return g.view(torch.int16).numpy().view(np.uint16)
    return g.numpy()


def replay_gpu(ps: P.ParameterServer, kinds, learners, grad_fn, lazy: bool = False, fuse_t: int = 1):
    """grad_fn(learner, push_index) -> device tensor.  Applies eagerly, or T groups at a time."""
    pulled, counts = {}, {}
    ready = 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            pulled[l] = ps.pull_weights()
        else:
            p = counts.get(l, 0)
            counts[l] = p + 1
            ready += ps.push_gradient(l, grad_fn(l, p), pulled[l])
            if ready and (not lazy or ready >= fuse_t):
                ready -= ps.apply_update()
    ps.flush()
    ps.synchronize()


def run_pair(num_params, lam, n, alpha0, momentum, wd, modulation, grad_dtype, grad_std, kinds, learners,
             w0: torch.Tensor, seed: int, fuse_t: int = 1, lazy: bool = False, precisions=(32, 64),
             options=None, misalign: int = 0, checkpoints: int = 0, tol: float = 1e-5,
             penalty_base=None, layers=None, mirror: bool = False):
    """Returns (gpu_w, gpu_v, gpu_log, {precision: (w, v, log)}).  layers = (bounds, lr_mult, wd_mult);
    mirror: also keep the bf16 weight mirror and compare it with the reference's rounding at the end."""
    dev = torch.device("cuda", 0)
    tdt = TORCH_DTYPE[grad_dtype]
    mod = P.binding.MODULATIONS[modulation]
    refs = {}
    for prec in precisions:
        r = R.ReferencePS(num_params, lam, n, alpha0, momentum, wd, mod, prec)
        r.set_weights(w0.numpy())
        if penalty_base is not None:
            r.set_penalty_base(penalty_base)
        if layers is not None:
            r.set_layer_multipliers(*layers)
        refs[prec] = r

    state = None
    if misalign:                      # state carved out at an odd element offset: scalar kernel path
        wbuf = torch.zeros(num_params + misalign + 8, dtype=torch.float32, device=dev)
        vbuf = torch.zeros(num_params + misalign + 8, dtype=torch.float32, device=dev)
        state = (wbuf[misalign:misalign + num_params], vbuf[misalign:misalign + num_params])
    ps = P.ParameterServer(num_params, lam, n, alpha0, momentum, wd, modulation, grad_dtype, fuse_t,
                           device=dev, state=state)
    for key, val in (options or {}).items():
        ps.set_option(key, val)
    if penalty_base is not None:
        ps.set_penalty_base(penalty_base)
    if layers is not None:
        ps.set_layer_multipliers(*layers)
    ps.init_weights(w0.to(dev))
    mirror_t = ps.bind_weight_mirror() if mirror else None

    def grad_fn(l, p):
        if misalign:
            buf = torch.empty(num_params + misalign, dtype=tdt, device=dev)
            g = buf[misalign:]
            G.gradient(seed, l, p, num_params, grad_std, dtype=tdt, device=dev, out=g)
        else:
            g = G.gradient(seed, l, p, num_params, grad_std, dtype=tdt, device=dev)
        host = as_reference_grad(g)
        for r in refs.values():
            r_fired = r.push(l, host)
        return g

    # the reference consumes pulls too: interleave by wrapping the replay
    pulled, counts = {}, {}
    ready = 0
    total_updates = int((kinds != PULL).sum()) // (lam // n)
    every = max(1, total_updates // checkpoints) if checkpoints else 0
    next_check = every
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            pulled[l] = ps.pull_weights()
            for r in refs.values():
                assert r.pull(l) == pulled[l]          # timestamps agree call by call
        else:
            p = counts.get(l, 0)
            counts[l] = p + 1
            ready += ps.push_gradient(l, grad_fn(l, p), pulled[l])
            if ready and (not lazy or ready >= fuse_t):
                ready -= ps.apply_update()
            applied = ps.timestamps()[0]
            if every and ready == 0 and applied >= next_check:       # intermediate states, not only the final one
                next_check = applied + every
                ps.synchronize()
                wc, vc = ps.w[:num_params].cpu().numpy(), ps.v[:num_params].cpu().numpy()
                for prec, r in refs.items():
                    assert r.timestamp == applied
                    wr, vr = r.state()
                    if prec == 32:
                        assert same_bits(wc, wr) and same_bits(vc, vr)
                    else:
                        assert rel_l2(wc, wr) <= tol and rel_l2(vc, vr) <= tol
    ps.flush()
    ps.synchronize()
    out = {prec: (*r.state(), r.log()) for prec, r in refs.items()}
    empty = np.zeros(0, np.float32)
    w = ps.w[:num_params].cpu().numpy().copy() if num_params else empty
    v = ps.v[:num_params].cpu().numpy().copy() if num_params else empty
    log = ps.update_log()
    if mirror and 32 in refs and num_params:
        got = mirror_t[:num_params].cpu().view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(got, refs[32].weights_bf16()), "bf16 mirror differs from the reference's rounding"
    run_pair.last_kernel = ps.get_option(P.PS_OPT_LAST_KERNEL)
    run_pair.launches = {k: ps.get_option(o) for k, o in (("scalar", P.PS_OPT_LAUNCHES_SCALAR),
                                                          ("vector", P.PS_OPT_LAUNCHES_VECTOR),
                                                          ("bulk", P.PS_OPT_LAUNCHES_BULK))}
    ps.destroy()
    return w, v, log, out


def same_bits(x, ref) -> bool:
    """fp32 arrays equal as bit patterns (so +0 and -0 differ); NaNs must sit in the same places, their
    payloads may differ."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    ref = np.ascontiguousarray(np.asarray(ref).astype(np.float32))
    if x.shape != ref.shape or not np.array_equal(np.isnan(x), np.isnan(ref)):
        return False
    ok = ~np.isnan(ref)
    return bool(np.array_equal(x.view(np.uint32)[ok], ref.view(np.uint32)[ok]))


def assert_logs_equal(log, rlog):
    for f in ("update", "push_index", "ts_grad", "tau", "sigma", "learner", "position"):
        assert np.array_equal(log[f], rlog[f]), f
    assert np.array_equal(log["scale"], rlog["scale"].astype(np.float32))
    assert np.array_equal(log["decay"], rlog["decay"].astype(np.float32))


def assert_parity(w, v, log, refs, tol, layout=None):
    """Bit-exact against the fp32 reference, within `tol` relative L2 against the fp64 one."""
    if 32 in refs:
        w32, v32, log32 = refs[32]
        assert_logs_equal(log, log32)
        assert same_bits(w, w32), "weights differ from the fp32 reference"
        assert same_bits(v, v32), "momentum differs from the fp32 reference"
    if 64 in refs:
        w64, v64, log64 = refs[64]
        worst = max(rel_l2(w, w64), rel_l2(v, v64))
        if layout is not None:
            for seg in layout.segments:
                sl = slice(seg.offset, seg.offset + seg.count)
                if np.linalg.norm(w64[sl]) > 0:
                    worst = max(worst, rel_l2(w[sl], w64[sl]))
                if np.linalg.norm(v64[sl]) > 0:
                    worst = max(worst, rel_l2(v[sl], v64[sl]))
        assert worst <= tol, "relative L2 error %.3e above %.1e" % (worst, tol)
        return worst
    return 0.0


def parity_line(name, elements, updates, compared, w, v, w32, v32, w64, v64):
    """One row of the parity table (printed by the configuration tests; shown with pytest -s): distance of
    the GPU state from the fp64 reference, distance of the fp32 reference from the fp64 one (what keeping the
    state in fp32 costs by itself), and whether GPU and fp32 reference agree bit for bit."""
    same = same_bits(w, w32) and same_bits(v, v32)
    line = "PARITY | %s | %d | %d | %s | %.2e | %.2e | %.2e | %.2e | %s |" % (
        name, elements, updates, compared, rel_l2(w, w64), rel_l2(v, v64), rel_l2(w32, w64), rel_l2(v32, v64),
        "yes" if same else "NO")
    print(line)
    return line
