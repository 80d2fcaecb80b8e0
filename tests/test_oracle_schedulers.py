"""Pins for the oracle's workload-ratio schedulers (Algorithms 1 and 2 of the paper)."""
import itertools

import numpy as np
import pytest

from oracle import halo_ref as R


def test_comp_greedy_fills_fastest_first_and_leaves_the_rest_empty():
    # c descending order is devices 2, 0, 1; budgets 4, 5, 3; model 6 -> device 2 full (3), device 0 takes 3
    r = R.comp_greedy([4, 5, 3], [2.0, 1.0, 3.0], 6.0)
    assert np.allclose(r, [0.5, 0.0, 0.5])
    assert np.isclose(r.sum(), 1.0)
    # model exactly fills the fastest device -> only that one
    assert np.allclose(R.comp_greedy([4, 5, 3], [2.0, 1.0, 3.0], 3.0), [0, 0, 1])
    # model needs everything -> ratios proportional to the budgets
    assert np.allclose(R.comp_greedy([4, 5, 3], [2.0, 1.0, 3.0], 12.0), np.array([4, 5, 3]) / 12)
    # equal computing power: lower index first
    assert np.allclose(R.comp_greedy([2, 2], [1.0, 1.0], 2.0), [1, 0])


def test_comp_greedy_brute_force_small():
    rng = np.random.default_rng(0)
    for _ in range(200):
        n = int(rng.integers(1, 6))
        m = rng.integers(1, 10, n).astype(float)
        c = rng.permutation(n).astype(float) + 1.0   # distinct
        Mt = float(rng.uniform(0.1, m.sum()))
        r = R.comp_greedy(m, c, Mt)
        order = sorted(range(n), key=lambda i: -c[i])
        u = np.zeros(n); left = Mt
        for i in order:
            take = min(m[i], left); u[i] = take; left -= take
            if left <= 0: break
        assert np.allclose(r, u / u.sum(), atol=1e-12)


def test_min_max_memory_unbounded_is_proportional_to_computing_power():
    c = np.array([1.0, 2.0, 0.5, 4.0])
    m = np.full(4, 1e6)
    r = R.min_max(m, c, 100.0, 1e-6)
    assert np.allclose(r, c / c.sum(), rtol=1e-6)


def test_min_max_water_filling_properties():
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(2, 7))
        m = rng.uniform(1, 10, n)
        c = rng.uniform(0.5, 2.0, n)
        Mt = float(rng.uniform(0.2, 0.95) * m.sum())
        eps = 1e-6
        r = R.min_max(m, c, Mt, eps)
        assert np.isclose(r.sum(), 1.0)
        # the allocation holds the model; scaled back to Mt, nobody exceeds its budget by more than the slack
        # every device is either memory-capped or shares one utilisation level T = load / c
        load = r * Mt
        util = load / c
        T = util.max()
        capped = util < T * (1 - 1e-4)
        assert np.all(load[capped] <= m[capped] * (1 + 1e-6))
        # capped devices sit at (their share of) the full budget: load_i / m_i is the same for all of them
        if capped.sum() > 1:
            frac = load[capped] / m[capped]
            assert np.allclose(frac, frac[0], rtol=1e-4)
        # optimality against a brute-force search over T on a fine grid
        Ts = np.linspace(0, m.max() / c.min(), 20001)
        used = np.minimum(m[None, :], Ts[:, None] * c[None, :]).sum(1)
        T_best = Ts[np.argmax(used >= Mt)]
        u = np.minimum(m, T_best * c)
        assert np.allclose(r, u / u.sum(), atol=2e-3)


def test_min_max_beats_or_equals_greedy_on_makespan():
    rng = np.random.default_rng(2)
    for _ in range(100):
        n = int(rng.integers(2, 7))
        m = rng.uniform(1, 10, n); c = rng.uniform(0.5, 2.0, n)
        Mt = float(rng.uniform(0.2, 0.9) * m.sum())
        mk = lambda r: (r * Mt / c).max()
        assert mk(R.min_max(m, c, Mt, 1e-6)) <= mk(R.comp_greedy(m, c, Mt)) * (1 + 1e-5)


def test_schedulers_reject_models_that_do_not_fit():
    with pytest.raises(RuntimeError):
        R.comp_greedy([1, 1], [1.0, 1.0], 3.0)
    with pytest.raises(RuntimeError):
        R.min_max([1, 1], [1.0, 1.0], 3.0)
    with pytest.raises(RuntimeError):
        R.min_max([1, 1], [1.0, 0.0], 1.0)
