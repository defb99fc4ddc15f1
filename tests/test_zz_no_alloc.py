"""ps_fused_update_static: the update for callers that may not allocate.

A learner framework whose caching allocator owns the whole device, or a steady-state loop that must stay
free of the device-wide synchronisation an allocation brings, cannot use a code path that obtains memory
at run time; the bulk-copy kernel of the ordinary path does (a pinned status record, on its first launch).
The static entry point runs the same kernel with its status records in the library's static device memory.
Here it is called through the C ABI twice in a row and compared, bit for bit, with what ps_apply_update
(the existing entry point) leaves in theta and v for the same gradients and the same scales.

Collected last on purpose (the file name sorts behind every other test file): a run that stops at the first
failure has then already run everything else.  Passes alone in a fresh process and after the other tests.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_1511_05950_b200 as P
from workloads import generators as G, layouts

pytestmark = pytest.mark.gpu


def _served_and_static(n_el, lam, grad_dtype, seed, blocks):
    """Two consecutive updates through a ParameterServer (ps_apply_update) and through the static entry
    point, on separate copies of the same theta_0; yields both states after each update."""
    dev = torch.device("cuda", 0)
    tdt = P.binding.TORCH_DTYPE[grad_dtype]
    momentum, wd = 0.9, 5e-4
    w0 = G.initial_weights(layouts.flat(n_el), seed).to(dev)
    ps = P.ParameterServer(n_el, lam, 1, 0.01, momentum, wd, "exp_staleness", grad_dtype, device=dev)
    ps.init_weights(w0)
    w, v = w0.clone(), torch.zeros_like(w0)
    stale = [0, 0]                                  # learner 0 keeps its first timestamp: staleness 1, half the rate, in update 1
    for u in range(2):
        now = ps.pull_weights()
        grads = [G.gradient(seed, l, u, n_el, 1e-3, dtype=tdt, device=dev) for l in range(lam)]
        for l in range(lam):
            ps.push_gradient(l, grads[l], stale[0] if l == 0 else now)
        assert ps.apply_update() == 1
        ps.synchronize()
        log = ps.update_log(u, 1)
        order = [int(x) for x in log["learner"]]    # the summation order the server used
        gave_up = P.fused_update_static(w, v, [grads[l] for l in order], [float(s) for s in log["scale"]],
                                        float(log["decay"][0]), momentum, blocks=blocks)
        assert gave_up == 0
        yield (ps.w.cpu().numpy(), ps.v.cpu().numpy()), (w.cpu().numpy(), v.cpu().numpy())
    ps.destroy()


@pytest.mark.parametrize("grad_dtype,lam,n_el,blocks", [
    ("fp32", 4, 37 * 4096 + 1234 + 3, 0),           # many tiles, a ragged end
    ("bf16", 3, 5 * 8192 + 77, 0),
    ("fp32", 16, 300007, 5),                         # the largest group, a capped grid
    ("bf16", 1, 200, 0),                             # shorter than one tile: the element path alone
])
def test_static_entry_point_matches_apply_update_twice_in_a_row(grad_dtype, lam, n_el, blocks):
    calls = 0
    for (w_ref, v_ref), (w, v) in _served_and_static(n_el, lam, grad_dtype, 77, blocks):
        assert np.array_equal(w, w_ref) and np.array_equal(v, v_ref)       # same bits as the existing entry point
        calls += 1
    assert calls == 2


def test_static_entry_point_refuses_what_its_status_area_cannot_hold():
    dev = torch.device("cuda", 0)
    n_el = 4096
    w = torch.zeros(n_el, device=dev)
    v = torch.zeros(n_el, device=dev)
    g = torch.ones(n_el, device=dev)
    with pytest.raises(P.SoftsyncError) as e:
        P.fused_update_static(w, v, [g] * (P.PS_STATIC_MAX_GRADS + 1), [1.0] * (P.PS_STATIC_MAX_GRADS + 1), 0.0, 0.0)
    assert e.value.status == P.PS_ERR_STATIC_LIMIT
    with pytest.raises(P.SoftsyncError) as e:
        P.fused_update_static(w, v, [g], [1.0], 0.0, 0.0, blocks=P.PS_STATIC_MAX_BLOCKS + 1)
    assert e.value.status == P.PS_ERR_STATIC_LIMIT
    ptrs = (C.c_void_p * 1)(g.data_ptr() + 4)        # a gradient that is not 16-byte aligned
    sc = (C.c_float * 1)(1.0)
    assert P.ps_fused_update_static(w.data_ptr(), v.data_ptr(), n_el - 4, ptrs, sc, 1, 0.0, 0.0, P.PS_GRAD_FP32, 0,
                                    None, None) == P.PS_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert float(w.abs().sum()) == 0.0 and float(v.abs().sum()) == 0.0     # refused calls did nothing
    # and the plain case right after: v = g, theta = -g
    assert P.fused_update_static(w, v, [g], [1.0], 0.0, 0.0) == 0
    assert torch.equal(v, g) and torch.equal(w, -g)
