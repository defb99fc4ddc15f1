"""The seeded input generators: shapes, determinism, CPU/GPU-agnostic bits, distribution."""
import numpy as np
import pytest
import torch

from workloads import arrivals, configs, generators as G, layouts


def test_layout_sizes():
    small = layouts.cifar_cnn()
    assert small.num_params == 89578
    assert [s.offset for s in small.segments] == [0, 2400, 2432, 28032, 28064, 79264, 79328, 89568]
    large = layouts.alexnet_like()
    assert large.num_params == 60965224
    assert large.num_params % 8 == 0 and small.num_params % 4 == 2
    assert layouts.flat(1 << 20).num_params == 1 << 20


def test_splitmix64_known_answer():
    # first output of SplitMix64 seeded with 0 (published test vector)
    assert G.mix64_int(0x9E3779B97F4A7C15) == 0xE220A8397B1DCDAF
    t = G.mix64(torch.tensor([G._s64(0x9E3779B97F4A7C15)]))
    assert int(t[0]) & ((1 << 64) - 1) == 0xE220A8397B1DCDAF


def test_subset_equals_full_and_deterministic():
    n = 50000
    full = G.gradient(123, 3, 7, n, 1e-3)
    again = G.gradient(123, 3, 7, n, 1e-3)
    assert torch.equal(full, again)
    idx = torch.tensor([0, 1, 17, 4095, 4096, n - 1])
    assert torch.equal(G.gradient_at(123, 3, 7, idx, 1e-3), full[idx])
    other = G.gradient(123, 3, 8, n, 1e-3)
    assert not torch.equal(full, other)
    assert not torch.equal(full, G.gradient(123, 4, 7, n, 1e-3))


def test_distribution_is_normal_like():
    x = G.gradient(9, 0, 0, 1 << 21, 1e-4).double() / 1e-4
    assert abs(x.mean().item()) < 5e-3
    assert abs(x.std().item() - 1.0) < 5e-3
    assert abs((x ** 4).mean().item() - 2.9) < 0.05          # Irwin-Hall(12): kurtosis 3 - 0.1
    assert abs((x.abs() < 1).double().mean().item() - 0.6827) < 5e-3
    assert x.abs().max().item() <= 6.0


def test_integers_exact_in_fp32():
    x = G.centred_integers(G.stream_key(1, G.STREAM_GRADIENT, 0, 0), torch.arange(100000))
    assert x.abs().max().item() < (1 << 24)


def test_bf16_is_round_to_nearest_even_of_fp32():
    f = G.gradient(5, 1, 2, 4096, 1e-4)
    b = G.gradient(5, 1, 2, 4096, 1e-4, dtype=torch.bfloat16)
    assert torch.equal(b, f.to(torch.bfloat16))
    bits = f.view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    rne = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) & 0xFFFF
    assert torch.equal(b.view(torch.int16).to(torch.int64) & 0xFFFF, rne)


def test_initial_weights_biases_zero():
    lay = layouts.cifar_cnn()
    w = G.initial_weights(lay, 77)
    for seg in lay.segments:
        part = w[seg.offset:seg.offset + seg.count]
        if seg.is_bias:
            assert torch.count_nonzero(part) == 0
        else:
            assert abs(part.std().item() - 0.01) < 1.5e-3
    idx = torch.tensor([0, 2399, 2400, 2431, 2432, 89567, 89568, 89577])
    assert torch.equal(G.initial_weights_at(lay, 77, idx), w[idx])


@pytest.mark.parametrize("model", arrivals.MODELS)
def test_trace_structure(model):
    lam, pushes = 6, 200
    k, l = arrivals.make_trace(model, lam, pushes, seed=4)
    k2, l2 = arrivals.make_trace(model, lam, pushes, seed=4)
    assert np.array_equal(k, k2) and np.array_equal(l, l2)
    assert (k == arrivals.PUSH).sum() == pushes
    assert np.array_equal(l[:lam], np.arange(lam)) and (k[:lam] == arrivals.PULL).all()
    # every push is by a learner that pulled since its previous push, and is followed by its pull
    ready = set()
    for kind, who in zip(k.tolist(), l.tolist()):
        if kind == arrivals.PULL:
            ready.add(who)
        else:
            assert who in ready
            ready.remove(who)
    if model == "rounds":
        pl = l[k == arrivals.PUSH]
        for r in range(pushes // lam):
            assert sorted(pl[r * lam:(r + 1) * lam].tolist()) == list(range(lam))


def test_configs_match_the_benchmark_list():
    c1, c2, c3, c4 = configs.ALL
    assert (c1.c, c1.num_updates) == (4, 200)
    assert (c2.c, c2.num_updates) == (1, 10000)
    assert (c3.c, c3.num_updates) == (4, 500)
    assert (c4.c, c4.num_updates, c4.fuse_t) == (1, 2000, 8)
    assert c3.layout().num_params == 60965224
