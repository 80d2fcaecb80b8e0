"""Pins for the oracle's counter-based generator, arrival draw and Algorithm 3."""
import os

import numpy as np
import pytest

from oracle import halo_ref as R


def _read(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_philox_known_answers(golden_dir):
    rows = _read(golden_dir, "philox4x32_10_kat.txt")
    assert len(rows) == 3
    for row in rows:
        v = [int(t, 16) for t in row]
        assert R.philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_loss_threshold_endpoints_and_rounding():
    assert R.loss_threshold(0.0) == 0
    assert R.loss_threshold(1.0) == 1 << 32
    assert R.loss_threshold(0.5) == 1 << 31
    assert R.loss_threshold(0.25) == 1 << 30
    # round-half-up of rho * 2^32
    assert R.loss_threshold(0.3) == int(np.floor(0.3 * 2**32 + 0.5))


def test_arrival_extremes_never_random():
    for step in range(50):
        for layer in range(4):
            for dev in range(4):
                assert R.arrival(7, step, layer, dev, 0.0) == 1
                assert R.arrival(7, step, layer, dev, 1.0) == 0


def test_arrival_is_word0_of_philox_against_threshold():
    # the draw is defined by counter (step, layer, device, 0), key = seed halves
    seed = (0x12345678 << 32) | 0x9ABCDEF0
    for step, layer, dev, rho in [(0, 0, 0, 0.3), (5, 9, 2, 0.9), (1000, 31, 7, 0.05)]:
        w0 = R.philox4x32_10([step, layer, dev, 0], [seed & 0xFFFFFFFF, seed >> 32])[0]
        assert R.arrival(seed, step, layer, dev, rho) == int(w0 >= R.loss_threshold(rho))


@pytest.mark.parametrize("rho", [0.01, 0.05, 0.3, 0.5])
def test_arrival_frequency_within_three_sigma(rho):
    n = 40000
    lost = sum(1 - R.arrival(0, s, s % 32, s % 4, rho) for s in range(n))
    sigma = np.sqrt(n * rho * (1 - rho))
    assert abs(lost - n * rho) <= 3.5 * sigma


def test_arrival_streams_differ_across_step_layer_device():
    base = [R.arrival(3, s, 0, 0, 0.5) for s in range(256)]
    assert base != [R.arrival(3, s, 1, 0, 0.5) for s in range(256)]
    assert base != [R.arrival(3, s, 0, 1, 0.5) for s in range(256)]
    assert base != [R.arrival(4, s, 0, 0, 0.5) for s in range(256)]
    # pairwise independence (rough): joint loss of two devices ~ product
    n = 20000
    both = sum((1 - R.arrival(1, s, 2, 0, 0.5)) * (1 - R.arrival(1, s, 2, 1, 0.5)) for s in range(n))
    assert abs(both - n * 0.25) <= 4 * np.sqrt(n * 0.25 * 0.75)


def test_algorithm3_paper_example(golden_dir):
    rows = {r[0]: r[1:] for r in _read(golden_dir, "alg3_worked_example.txt")}
    G = int(rows["n_groups"][0])
    rho = [float(v) for v in rows["rho"]]
    ratio = [float(v) for v in rows["ratio"]]
    weights = [int(round(v * 10)) for v in ratio]
    order, thr, bnd = R.plan(rho, weights, G)
    got = {}
    for j, dev in enumerate(order):
        got[int(dev)] = list(range(bnd[j] + 1, bnd[j + 1] + 1))  # 1-based priority indices
    for dev in range(3):
        assert got[dev] == [int(v) for v in rows[f"device{dev}"]]
    # and through select(): scores descending in group id => priority index = group id + 1
    scores = np.arange(G, 0, -1, dtype=np.float32)
    sel = R.select(scores, rho, weights, R.SEL_TOPK, 0, 0.0, seed=0, step=0, layer=1, force_all=True)
    for dev in range(3):
        held = [g + 1 for g in range(G) if sel["dev_of_group"][g] == dev]
        assert held == [int(v) for v in rows[f"device{dev}"]]


def test_group_count_arithmetic_from_paper():
    # Sec. II-A: an MLP of width 6144 with group size 256 has 24 groups
    from paper_2601_11676_b200 import synth
    wl = synth.Workload("x", 1, 64, 6144, 256, 8, "f32", (0.0,), (1,), 500, 1)
    assert wl.n_groups == 24


@pytest.mark.parametrize("n", [2, 3, 4, 8])
def test_equal_shares_leave_one_nth_on_the_reliable_device(n):
    # Sec. V robustness study: with n equal devices of which n-1 are lossy, NGLR = 1 - 1/n
    G = 24 * n
    rho = [0.0] + [0.2] * (n - 1)
    order, thr, bnd = R.plan(rho, [1] * n, G)
    assert order[0] == 0
    assert bnd[1] - bnd[0] == G // n
    exposed = G - (bnd[1] - bnd[0])
    assert exposed / G == pytest.approx(1 - 1 / n)


def test_partition_invariants_random():
    rng = np.random.default_rng(0)
    for _ in range(300):
        n = int(rng.integers(1, 9))
        M = int(rng.integers(0, 200))
        rho = rng.uniform(0, 1, n).round(2)  # rounding creates ties
        w = rng.integers(0, 5, n).astype(np.uint32)
        if w.sum() == 0:
            w[0] = 1
        order, thr, bnd = R.plan(rho, w, M)
        assert sorted(order.tolist()) == list(range(n))
        # ascending loss, ties by index
        keys = [(rho[i], i) for i in order]
        assert keys == sorted(keys)
        assert bnd[0] == 0 and bnd[n] == M
        assert all(bnd[j] <= bnd[j + 1] for j in range(n))
        W = int(w.sum())
        cum = 0
        for j in range(n):
            cum += int(w[order[j]])
            exact = M * cum / W
            assert abs(bnd[j + 1] - exact) <= 0.5 + 1e-9
            if w[order[j]] == 0:
                assert bnd[j + 1] == bnd[j]  # zero share => empty chunk


def test_plan_rejects_bad_input():
    with pytest.raises(RuntimeError):
        R.plan([0.1, 1.5], [1, 1], 4)
    with pytest.raises(RuntimeError):
        R.plan([0.1, 0.2], [0, 0], 4)
