"""What the method is for, on a problem small enough to reason about.

The paper's experimental claim (Section 4.3): with many asynchronous learners a constant learning rate alpha0
stops converging, dividing it by the staleness restores convergence.  Gradient descent with gradients that
are tau updates old is unstable on a quadratic of curvature L once alpha*L exceeds about pi/(2*tau + 1).
Here lambda = 30 learners run 30-softsync (c = 1, average staleness about 29) on f(theta) = 1/2 sum h_k theta_k^2
with alpha0 * max(h) = 0.5: far beyond the stable range for a constant rate, well inside it after division by
the staleness (0.5/29 = 0.017 < pi/59 = 0.053).  Learners really pull weights and compute their gradient from them.
This is a qualitative check of behaviour; the arithmetic itself is pinned elsewhere.
"""
import numpy as np
import pytest
import torch

from oracle import reference as R
from tests.helpers import PULL

LAM, PUSHES, N_EL, ALPHA0 = 30, 1500, 64, 0.5


def curvatures(n):
    return np.linspace(0.1, 1.0, n)


def run_reference(modulation):
    kinds, learners = R.simulate_arrivals("uniform", LAM, PUSHES, 4)
    h = curvatures(N_EL)
    ps = R.ReferencePS(N_EL, LAM, LAM, ALPHA0, 0.0, 0.0, modulation, 64)
    ps.set_weights(np.ones(N_EL, np.float32))
    held = {}
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == PULL:
            ps.pull(l)
            held[l] = ps.state()[0].copy()                    # the weights this learner will differentiate
        else:
            ps.push(l, (h * held[l]).astype(np.float32))      # gradient of the quadratic at the pulled weights
    return np.linalg.norm(ps.state()[0]) / np.sqrt(N_EL), ps.log()


def test_reference_diverges_with_a_constant_rate_and_converges_with_modulation():
    const, log_c = run_reference(R.MOD_CONSTANT)
    modulated, log_m = run_reference(R.MOD_INV_STALENESS)
    assert 25 < log_m["tau"][200:].mean() < 33                # <tau> close to n = 30 (Section 2.4)
    assert modulated < 0.05                                   # started at 1
    assert not np.isfinite(const) or const > 1e3


@pytest.mark.gpu
def test_library_shows_the_same_behaviour_with_real_weight_pulls():
    import paper_1511_05950_b200 as P
    dev = torch.device("cuda", 0)
    kinds, learners = R.simulate_arrivals("uniform", LAM, PUSHES, 4)
    h = torch.tensor(curvatures(N_EL), dtype=torch.float32, device=dev)
    out = {}
    for modulation in ("constant", "inv_staleness"):
        ps = P.ParameterServer(N_EL, LAM, LAM, ALPHA0, 0.0, 0.0, modulation, device=dev)
        ps.init_weights(torch.ones(N_EL))
        held, stamp = {}, {}
        for k, l in zip(kinds.tolist(), learners.tolist()):
            if k == PULL:
                held[l] = torch.empty(N_EL, device=dev)
                stamp[l] = ps.pull_weights(held[l])           # pullWeights: theta_i and its timestamp
            else:
                if ps.push_gradient(l, h * held[l], stamp[l]):
                    ps.apply_update()
        ps.synchronize()
        out[modulation] = float(torch.linalg.vector_norm(ps.w.double()) / np.sqrt(N_EL))
        ps.destroy()
    ref_const, _ = run_reference(R.MOD_CONSTANT)
    ref_mod, _ = run_reference(R.MOD_INV_STALENESS)
    assert out["inv_staleness"] < 0.05
    assert not np.isfinite(out["constant"]) or out["constant"] > 1e3
    assert abs(out["inv_staleness"] - ref_mod) <= 1e-3 * ref_mod + 1e-6      # fp32 server vs fp64 reference
