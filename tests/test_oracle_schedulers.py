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


# ---- late devices (Sec. III-B.3 timeout, Eq. 1 cost model) ------------------------------------------------------

def test_late_devices_hand_computed():
    # tau = 2 ms per group; capacities 1, 2, 4 (relative speed); T_c = 0.5 ms; timeout 10 ms
    #   device 0: 4 groups -> 8.0 + 0.5 = 8.5  on time
    #   device 1: 10 groups -> 10.0 + 0.5 = 10.5 late
    #   device 2: 19 groups -> 9.5 + 0.5 = 10.0 exactly the timeout: still merged (late means later than)
    #   device 3: nothing assigned: never late, whatever its speed
    late = R.late_devices([4, 10, 19, 0], [1.0, 2.0, 4.0, 1e-9], 2.0, 0.5, 10.0)
    assert late.tolist() == [0, 1, 0, 0]


def test_late_devices_is_monotone_and_matches_brute_force():
    rng = np.random.default_rng(3)
    for _ in range(200):
        n = int(rng.integers(1, 7))
        units = rng.integers(0, 40, size=n)
        comp = rng.uniform(0.2, 5.0, size=n)
        tau, tc, to = rng.uniform(0.1, 3.0), rng.uniform(0.0, 1.0), rng.uniform(1.0, 30.0)
        late = R.late_devices(units, comp, tau, tc, to)
        brute = [(1 if (u > 0 and tau * u / c + tc > to) else 0) for u, c in zip(units.tolist(), comp.tolist())]
        assert late.tolist() == brute
        assert (R.late_devices(units, comp * 2, tau, tc, to) <= late).all()        # faster devices: never later
        assert (R.late_devices(units + 1, comp, tau, tc, to) >= late).all()        # more work: never earlier
    # a min-max schedule equalises tau*W_i/c_i, so either everybody is late or nobody (memory not binding)
    c = np.array([1.0, 2.0, 5.0])
    r = R.min_max([1e9] * 3, c, 100.0)
    units = np.round(r * 800).astype(np.int32)
    t = 0.1 * units / c
    assert t.max() - t.min() <= 0.1 * 2 / c.min()
    assert len(set(R.late_devices(units, c, 0.1, 0.0, float(t.max()) + 1e-9).tolist())) == 1


def test_late_devices_rejects_bad_arguments():
    with pytest.raises(Exception):
        R.late_devices([1, 2], [1.0, 0.0], 1.0, 0.0, 1.0)
    with pytest.raises(Exception):
        R.late_devices([1, -2], [1.0, 1.0], 1.0, 0.0, 1.0)
