"""The paper's accuracy experiment in miniature (Section 4.3), with synthetic images.

Thirty simulated learners train the 89,578-parameter CIFAR-shaped CNN (three 5x5 convolutions with pooling and
a 10-way linear layer: the layout of workloads.layouts.cifar_cnn) through the parameter server with the
30-softsync protocol: each pulls the weights, computes a mini-batch gradient with autograd, pushes it with the
timestamp it pulled.  Images are class templates plus noise (CIFAR10 itself is not available).  What the paper
reports, and this checks: alpha0 is a good rate for one learner; with 30 asynchronous learners the same constant
alpha0 does not train at all, and dividing it by the staleness trains to high accuracy.
The learners use PyTorch; everything the server does runs in the library under test.

Every gradient the learners push (real autograd gradients: a large dynamic range, exact zeros from dead
units, values growing without bound in the run that diverges) is also pushed, with the same timestamp, into
the CPU reference; the final weights, momentum and the whole log must equal the reference's bit for bit.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

pytestmark = pytest.mark.gpu

ALPHA0 = 0.003


def _forward(layout, flat, x):
    seg = {s.name: (s.offset, s.count) for s in layout.segments}

    def p(name, shape):
        o, c = seg[name]
        return flat[o:o + c].view(shape)

    h = F.max_pool2d(F.relu(F.conv2d(x, p("conv1.weight", (32, 3, 5, 5)), p("conv1.bias", (32,)), padding=2)), 2)
    h = F.max_pool2d(F.relu(F.conv2d(h, p("conv2.weight", (32, 32, 5, 5)), p("conv2.bias", (32,)), padding=2)), 2)
    h = F.max_pool2d(F.relu(F.conv2d(h, p("conv3.weight", (64, 32, 5, 5)), p("conv3.bias", (64,)), padding=2)), 2)
    return F.linear(h.flatten(1), p("fc.weight", (10, 1024)), p("fc.bias", (10,)))


def _train(num_learners, n, modulation, pushes, mu=8):
    import paper_1511_05950_b200 as P
    from oracle import reference as R
    from tests.gpu_harness import assert_logs_equal
    from workloads import arrivals, generators as G, layouts

    dev = torch.device("cuda", 0)
    torch.backends.cudnn.deterministic = True          # same convolution algorithms from run to run
    torch.backends.cudnn.benchmark = False
    layout = layouts.cifar_cnn()
    num_params = layout.num_params
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    templates = torch.randn(10, 3, 32, 32, device=dev, generator=gen)

    def batch(count, g):
        y = torch.randint(0, 10, (count,), device=dev, generator=g)
        return templates[y] + torch.randn(count, 3, 32, 32, device=dev, generator=g), y

    held_out = torch.Generator(device=dev)
    held_out.manual_seed(123)
    xv, yv = batch(512, held_out)

    kinds, learners = arrivals.make_trace("uniform", num_learners, pushes, 5)
    ps = P.ParameterServer(num_params, num_learners, n, ALPHA0, 0.9, 5e-4, modulation, device=dev)
    w0 = G.initial_weights(layout, 3, 0.05, device=dev)
    ps.init_weights(w0)
    ref = R.ReferencePS(num_params, num_learners, n, ALPHA0, 0.9, 5e-4, P.binding.MODULATIONS[modulation], 32)
    ref.set_weights(w0.cpu().numpy())
    held = {l: torch.empty(num_params, device=dev) for l in range(num_learners)}
    stamp = {}
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    for k, l in zip(kinds.tolist(), learners.tolist()):
        if k == arrivals.PULL:
            stamp[l] = ps.pull_weights(held[l])                       # pullWeights
        else:
            w_l = held[l].clone().requires_grad_(True)
            x, y = batch(mu, g)
            grad, = torch.autograd.grad(F.cross_entropy(_forward(layout, w_l, x), y), w_l)    # calcGradient
            grad = grad.contiguous()
            ref.push(l, grad.cpu().numpy(), timestamp=stamp[l])
            if ps.push_gradient(l, grad, stamp[l]):                   # pushGradient
                ps.apply_update()
    ps.synchronize()
    w32, v32 = ref.state()
    w_gpu, v_gpu = ps.w.cpu().numpy(), ps.v.cpu().numpy()
    # exact equality of every value; a run that has diverged must have its inf / nan in the same places
    # (the payload bits of a nan are the one thing CPU and GPU arithmetic may legitimately choose differently)
    assert np.array_equal(w_gpu, w32.astype(np.float32), equal_nan=True)
    assert np.array_equal(v_gpu, v32.astype(np.float32), equal_nan=True)
    assert_logs_equal(ps.update_log(), ref.log())
    with torch.no_grad():
        accuracy = (_forward(layout, ps.w, xv).argmax(1) == yv).float().mean().item()
    tau = ps.update_log()["tau"]
    ps.destroy()
    return accuracy, float(tau.mean())


def test_single_learner_trains_with_alpha0():
    accuracy, tau = _train(1, 1, "inv_staleness", 1500)
    assert accuracy > 0.95 and tau == 0.0


def test_thirty_learners_need_the_staleness_dependent_rate():
    acc_constant, tau_c = _train(30, 30, "constant", 8000)
    acc_modulated, tau_m = _train(30, 30, "inv_staleness", 8000)
    assert 25 < tau_m < 33 and tau_c == tau_m                         # <tau> close to n = 30 (Section 2.4)
    assert acc_constant < 0.3                                         # no better than chance: does not train
    assert acc_modulated > 0.6                                        # typically 0.95-0.99; training is chaotic,
    assert acc_modulated > acc_constant + 0.4                         # so the bar is far below the usual outcome
