"""GPU parity of the knapsack allocation of Section 3.4: range curves bit-exact against the checker's greedy
loop, allocations identical to the checker's dynamic programme (both sides take every comparison in double
with the same single operations), total reward equal."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs, prng
from oracle import oracle as orc

from gpu_util import dev, host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,S_max", [((33, 20), 7), ((16, 12, 3, 3), 30), ((9, 1), 4), ((5, 6), 0), ((130, 2051), 300),
                                         ((64, 3136), 400)])
def test_range_curve_matches_checker(shape, S_max):
    W = prng.laplace(19, 0, shape, 0.02)
    W.reshape(-1)[prng.distinct_positions(19, 1, W.size, min(5, W.size))] *= 25
    st = ocs.new_status()
    curve = host(ocs.ocs_range_curve(dev(W), S_max, dev_status=st))
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(curve.view(np.uint32), orc.range_curve(W, S_max).view(np.uint32))


def test_range_curve_ties_and_zero():
    c3 = configs.config3(O=64, C=3136, M=4)["W"]              # thousands of equal outliers: the curve stays flat
    np.testing.assert_array_equal(host(ocs.ocs_range_curve(dev(c3), 314)), orc.range_curve(c3, 314))
    Z = np.zeros((4, 8), np.float32)
    np.testing.assert_array_equal(host(ocs.ocs_range_curve(dev(Z), 5)), np.zeros(6, np.float32))


def test_knapsack_small_layers_match_checker():
    rng = np.random.default_rng(47)
    for trial in range(5):
        n_layers = int(rng.integers(3, 9))
        Ws, cost = [], []
        for l in range(n_layers):
            O, Cn, R = int(rng.integers(2, 9)) * 4, int(rng.integers(3, 40)), int(rng.choice([1, 9]))
            W = prng.laplace(50 + trial, l, (O, Cn, R), 0.02)
            W.reshape(-1)[prng.distinct_positions(50 + trial, 100 + l, W.size, 3)] *= float(rng.uniform(3, 30))
            Ws.append(W)
            cost.append(O * R)
        smax = [int(rng.integers(1, 12)) for _ in Ws]
        o_curves = [orc.range_curve(W, s) for W, s in zip(Ws, smax)]
        budget = int(sum(c * s for c, s in zip(cost, smax)) * rng.uniform(0.15, 0.8))
        S_o, tot_o = orc.knapsack(o_curves, cost, budget)
        g_curves = [ocs.ocs_range_curve(dev(W), s) for W, s in zip(Ws, smax)]
        S_g, tot_g = ocs.ocs_knapsack_allocate(g_curves, cost, budget)
        np.testing.assert_array_equal(host(S_g), S_o)
        assert float(host(tot_g)[0]) == tot_o
        assert sum(int(s) * c for s, c in zip(host(S_g), cost)) <= budget


def test_knapsack_resnet50_at_the_simple_rules_budget():
    """Config 4's layers with the memory the ceil(r*C) rule spends at r = 0.01 as the budget: the allocation equals
    the checker's, stays within the budget and earns at least the simple rule's reward."""
    cfg = configs.config4(batch=1, image=32)
    specs = cfg["layers"] + [cfg["fc"]]
    Ws = [cfg["params"][s.name][0].reshape(s.O, s.C, s.k * s.k) for s in specs]
    cost = [s.O * s.k * s.k for s in specs]
    simple = [orc.num_splits(s.C, 0.01) for s in specs]
    budget = sum(c * n for c, n in zip(cost, simple))
    smax = [min(s.C, 4 * n + 4) for s, n in zip(specs, simple)]
    o_curves = [orc.range_curve(W, m) for W, m in zip(Ws, smax)]
    S_o, tot_o = orc.knapsack(o_curves, cost, budget)
    g_curves = [ocs.ocs_range_curve(dev(W), m) for W, m in zip(Ws, smax)]
    for gc, oc in zip(g_curves, o_curves):
        np.testing.assert_array_equal(host(gc), oc)
    S_g, tot_g = ocs.ocs_knapsack_allocate(g_curves, cost, budget)
    np.testing.assert_array_equal(host(S_g), S_o)
    assert float(host(tot_g)[0]) == tot_o
    assert sum(int(s) * c for s, c in zip(S_o, cost)) <= budget
    simple_reward = sum((float(c[0]) - float(c[n])) / float(c[0]) for c, n in zip(o_curves, simple))
    assert tot_o >= simple_reward - 1e-12


def test_knapsack_rejects_bad_arguments():
    c = [ocs.ocs_range_curve(dev(prng.laplace(3, 0, (8, 8), 0.1)), 2)]
    with pytest.raises(ocs.OcsError):
        ocs.ocs_knapsack_allocate(c, [0], 10)
    with pytest.raises(ocs.OcsError):
        ocs.ocs_knapsack_allocate(c, [1], 1 << 40)
