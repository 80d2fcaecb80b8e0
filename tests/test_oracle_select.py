"""Pins for the oracle's ranking, critical choice, assignment and keep mask (steps a2..a5)."""
import itertools

import numpy as np
import pytest

from oracle import halo_ref as R


def _brute_order(scores):
    s = [(-np.inf if np.isnan(v) else float(v)) for v in scores]
    return sorted(range(len(s)), key=lambda g: (-s[g], g))


def _sel(scores, rho=(0.0, 0.3), w=(1, 1), mode=R.SEL_TOPK, k=0, theta=0.0, seed=0, step=0, layer=1, force=False):
    return R.select(np.asarray(scores, dtype=np.float32), list(rho), list(w), mode, k, theta, seed, step, layer, force)


def test_order_all_permutations_small():
    for G in range(1, 7):
        base = np.linspace(-1.0, 1.0, G).astype(np.float32)
        for perm in itertools.permutations(range(G)):
            s = base[list(perm)]
            out = _sel(s, k=0)
            assert out["order"].tolist() == _brute_order(s)
            assert [out["rank"][g] for g in out["order"]] == list(range(G))


def test_order_random_with_duplicates():
    rng = np.random.default_rng(1)
    for _ in range(200):
        G = int(rng.integers(1, 65))
        s = rng.integers(-3, 4, G).astype(np.float32)  # many ties
        out = _sel(s, k=int(rng.integers(0, G + 1)))
        assert out["order"].tolist() == _brute_order(s)


def test_all_equal_scores_identity_order():
    out = _sel(np.full(17, 2.5, dtype=np.float32), k=5)
    assert out["order"].tolist() == list(range(17))


def test_nan_is_lowest_and_flagged_and_negative_zero_ties_with_zero():
    s = np.array([1.0, np.nan, -0.0, 0.0, -5.0], dtype=np.float32)
    out = _sel(s, k=2)
    assert out["order"].tolist() == [0, 2, 3, 4, 1]
    assert out["status"] & R.STATUS_NONFINITE
    assert _sel([1.0, 2.0], k=1)["status"] == 0


def test_topk_critical_are_master_and_always_kept():
    rng = np.random.default_rng(2)
    for trial in range(100):
        G = int(rng.integers(2, 100))
        k = int(rng.integers(0, G + 1))
        s = rng.normal(size=G).astype(np.float32)
        out = _sel(s, rho=(1.0, 1.0), w=(3, 2), k=k, step=trial)
        order = _brute_order(s)
        crit = set(order[:k])
        assert {g for g in range(G) if out["dev_of_group"][g] == -1} == crit
        # every device always lost => exactly the critical groups survive
        assert out["n_keep"] == k
        assert out["keep_list"][:k].tolist() == sorted(crit)
        assert (out["keep_list"][k:] == -1).all()
        assert out["keep"].sum() == k


def test_threshold_mode_is_prefix_of_order():
    rng = np.random.default_rng(3)
    for _ in range(100):
        G = int(rng.integers(1, 80))
        s = rng.normal(size=G).astype(np.float32)
        theta = float(np.float32(rng.normal()))
        out = _sel(s, rho=(1.0,), w=(1,), mode=R.SEL_THRESHOLD, theta=theta)
        crit = [g for g in range(G) if s[g] >= np.float32(theta)]
        assert out["keep_list"][: out["n_keep"]].tolist() == crit
        assert all(out["rank"][g] < len(crit) for g in crit)


def test_assignment_follows_plan_in_priority_order():
    rng = np.random.default_rng(4)
    for _ in range(100):
        G = int(rng.integers(4, 120))
        n = int(rng.integers(1, 6))
        k = int(rng.integers(0, G))
        rho = rng.uniform(0, 1, n)
        w = rng.integers(1, 10, n)
        s = rng.normal(size=G).astype(np.float32)
        out = _sel(s, rho=rho, w=w, k=k, force=True)
        order_dev, thr, bnd = R.plan(rho, w, G - k)
        order = _brute_order(s)
        for p, g in enumerate(order[k:]):
            j = next(j for j in range(n) if bnd[j] <= p < bnd[j + 1])
            assert out["dev_of_group"][g] == order_dev[j]
        assert out["n_keep"] == G and out["arrived"].all()


def test_keep_is_critical_or_arrived_and_list_is_ascending():
    rho, w = (0.0, 0.5, 0.9), (2, 1, 1)
    s = np.random.default_rng(5).normal(size=40).astype(np.float32)
    seen_partial = False
    for step in range(40):
        out = _sel(s, rho=rho, w=w, k=10, seed=11, step=step, layer=3)
        arr = [R.arrival(11, step, 3, i, rho[i]) for i in range(3)]
        assert out["arrived"].tolist() == arr
        for g in range(40):
            dev = out["dev_of_group"][g]
            assert out["keep"][g] == (1 if dev < 0 else arr[dev])
        kl = out["keep_list"][: out["n_keep"]].tolist()
        assert kl == [g for g in range(40) if out["keep"][g]]
        seen_partial |= 10 < out["n_keep"] < 40
    assert seen_partial


def test_first_layer_rule_force_all_ignores_loss():
    out = _sel(np.arange(8, dtype=np.float32), rho=(1.0, 1.0), w=(1, 1), k=0, force=True)
    assert out["n_keep"] == 8 and out["arrived"].tolist() == [1, 1]


def test_everything_exposed_and_lost_gives_empty_keep_set():
    # 100 % of groups on lossy devices and all of them lost: the block is skipped
    out = _sel(np.arange(8, dtype=np.float32), rho=(1.0,), w=(1,), k=0)
    assert out["n_keep"] == 0 and (out["keep_list"] == -1).all()


def test_no_devices_means_master_holds_all():
    out = R.select(np.arange(5, dtype=np.float32), [], [], R.SEL_TOPK, 2, 0.0, 0, 0, 1)
    assert out["n_keep"] == 5 and (out["dev_of_group"] == -1).all()
