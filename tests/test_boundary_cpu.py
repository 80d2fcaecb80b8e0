"""CPU-side checks of the C-ABI library: it loads, exports what include/halo.h declares, validates arguments on
the host, and its host-only Assignment phase agrees with the oracle's Algorithm 3."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import build as halo_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    halo_build.build()
    return B.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "halo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(halo_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in halo.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_status_strings(lib):
    assert B.status_string(0) == "ok"
    assert "aligned" in B.status_string(-3)
    assert "index" in B.status_message(B.DEV_BAD_INDEX)
    assert B.status_message(0) == "clean"


def test_plan_matches_oracle_algorithm3(lib):
    rng = np.random.default_rng(0)
    for _ in range(200):
        n = int(rng.integers(0, 9))
        G = int(rng.integers(1, 300))
        M = int(rng.integers(0, G + 1))
        rho = rng.uniform(0, 1, n).round(2)
        w = rng.integers(0, 6, n)
        if n and w.sum() == 0:
            w[0] = 1
        plan = B.Plan(G, rho, w, B.SEL_TOPK, G - M, 0.0, 5)
        order, thr, bnd = plan.describe(M)
        o_ref, t_ref, b_ref = R.plan(rho, w, M)
        assert order == o_ref.tolist() and thr == [int(v) for v in t_ref] and bnd == b_ref.tolist()
        plan.close()


def test_plan_paper_example(lib):
    plan = B.Plan(8, [0.0, 0.5, 0.1], [4, 4, 2], B.SEL_TOPK, 0, 0.0, 0)
    order, thr, bnd = plan.describe(8)
    assert order == [0, 2, 1] and bnd == [0, 3, 5, 8]


def test_plan_rejects_bad_arguments(lib):
    for args in [
        (8, [1.5], [1]), (8, [-0.1], [1]), (8, [0.1, 0.2], [0, 0]), (0, [0.1], [1]), (B.MAX_GROUPS + 1, [0.1], [1]),
        (8, [0.0] * (B.MAX_DEVICES + 1), [1] * (B.MAX_DEVICES + 1)),
    ]:
        with pytest.raises(B.HaloError):
            B.Plan(*args)
    with pytest.raises(B.HaloError):
        B.Plan(8, [0.1], [1], B.SEL_TOPK, 9)
    with pytest.raises(B.HaloError):
        B.Plan(8, [0.1], [1], B.SEL_THRESHOLD, 0, float("nan"))


def test_host_side_argument_checks_launch_nothing(lib):
    # NULL pointers / bad shapes are rejected before any CUDA call, so this runs without a GPU
    sh = B.ffn_shape(256, 688, 16, B.F32)
    rc = lib.halo_group_ffn(ctypes.byref(sh), None, None, 1, None, None, None, 0, None, None, 0, None, None)
    assert rc == -1
    bad = B.ffn_shape(250, 688, 16, B.F32)
    rc = lib.halo_group_ffn(ctypes.byref(bad), 16, 16, 1, 16, 16, None, 0, 16, None, 0, None, None)
    assert rc == -2
    bad = B.ffn_shape(256, 690, 16, B.F32)
    assert lib.halo_pack_weights(ctypes.byref(bad), 16, 16, 16, 16, None) == -2
    bad = B.ffn_shape(256, 688, 16, 7)
    assert lib.halo_pack_weights(ctypes.byref(bad), 16, 16, 16, 16, None) == -4
    rc = lib.halo_group_ffn(ctypes.byref(sh), 24, 16, 1, 16, 16, None, 0, 16, None, 0, None, None)
    assert rc == -3  # W_packed not 16-byte aligned
    ps = B.pred_shape(256, 32, 43, B.F32)
    assert B.halo_predict_workspace_bytes(ps, 1) == 4 * (32 + 43)
    rc = lib.halo_predict_groups(ctypes.byref(ps), 16, 16, 16, 1, 0, 16, 16, 8, None, None)
    assert rc == -8  # workspace too small
    assert lib.halo_merge_partials(None, None, 1, 1, 8, None, None) == -1
    assert lib.halo_select_groups(None, None, 0, 0, 0, None, None, None, None, None, None, None, None) == -1


def test_int4_entry_points_check_their_arguments_on_the_host(lib):
    """The int4 calls reject NULL pointers, shapes outside the format (d_model % 128), misaligned arrays and other
    element types before anything is launched."""
    sh = B.ffn_shape(256, 688, 16, B.BF16)
    assert lib.halo_quantize_rows_i4(256, 10, B.BF16, None, 16, 16, None) == -1
    assert lib.halo_quantize_rows_i4(200, 10, B.BF16, 16, 16, 16, None) == -2          # not a multiple of 128
    assert lib.halo_quantize_rows_i4(256, 0, B.BF16, 16, 16, 16, None) == -2
    assert lib.halo_quantize_rows_i4(256, 10, 5, 16, 16, 16, None) == -4
    assert lib.halo_quantize_rows_i4(256, 10, B.BF16, 16, 24, 16, None) == -3
    assert lib.halo_dequantize_weights_i4(ctypes.byref(sh), None, 16, None, None, 16, None, None) == -1
    assert lib.halo_dequantize_weights_i4(ctypes.byref(sh), 16, 16, 16, None, 16, None, None) == -1   # list without a count
    assert lib.halo_dequantize_weights_i4(ctypes.byref(sh), 16, 16, None, None, 24, None, None) == -3
    bad = B.ffn_shape(192, 688, 16, B.BF16)
    assert lib.halo_dequantize_weights_i4(ctypes.byref(bad), 16, 16, None, None, 16, None, None) == -2
    lm = B.lm_shape(256, 100, 16, B.BF16)
    assert lib.halo_group_lm_head_i4(ctypes.byref(lm), 16, 16, 16, 1, None, None, 16, None, None) == -1   # no status word
    assert lib.halo_group_lm_head_i4(ctypes.byref(lm), 16, 16, 16, 1, 16, None, 16, 16, None) == -1       # list without a count
    assert lib.halo_group_lm_head_i4(ctypes.byref(B.lm_shape(200, 100, 16, B.BF16)), 16, 16, 16, 1, None, None, 16, 16, None) == -2
    assert lib.halo_group_lm_head_i4(ctypes.byref(lm), 16, 24, 16, 1, None, None, 16, 16, None) == -3
    mh = B.mha_shape(256, 4, 32, 64, B.BF16)
    ptrs = [16] * 9
    assert lib.halo_mha_block_i4(ctypes.byref(mh), None, *ptrs[1:], 0, 16, 16, None, 0, 16, None, None) == -1
    assert lib.halo_mha_block_i4(ctypes.byref(mh), *ptrs, 64, 16, 16, None, 0, 16, None, None) == -1       # pos beyond the cache
    assert lib.halo_mha_block_i4(ctypes.byref(B.mha_shape(256, 4, 32, 64, B.F32)), *ptrs, 0, 16, 16, None, 0, 16, None, None) == -4
    assert lib.halo_mha_block_i4(ctypes.byref(B.mha_shape(192, 4, 32, 64, B.BF16)), *ptrs, 0, 16, 16, None, 0, 16, None, None) == -2
    assert lib.halo_mha_block_i4(ctypes.byref(mh), 16, 24, *ptrs[2:], 0, 16, 16, None, 0, 16, None, None) == -3
    big = B.ffn_shape(512, 1024, 128, B.BF16)
    assert B.halo_group_ffn_i4_workspace_bytes(big, 8) == 0                      # too few tokens for the tensor cores
    need = B.halo_group_ffn_i4_workspace_bytes(big, 64)
    assert need >= 3 * 1024 * 512 * 2                                             # one bf16 block + the FFN's own
    assert B.halo_group_ffn_i4_workspace_bytes(B.ffn_shape(512, 1024, 32, B.BF16), 64) == 0   # group size not taken
    assert lib.halo_group_ffn_i4_prompt(ctypes.byref(big), 16, 16, 16, 64, 16, 16, None, 0, 16, None, 0, None, None) == -8
    assert lib.halo_group_ffn_i4_prompt(ctypes.byref(big), 16, 16, 16, 64, 16, 16, None, 0, 16, 16, need - 1, None, None) == -8
    assert lib.halo_group_ffn_i4_prompt(ctypes.byref(big), None, 16, 16, 64, 16, 16, None, 0, 16, 16, need, None, None) == -1
    assert lib.halo_group_ffn_i4_prompt(ctypes.byref(big), 16, 16, 16, 64, 16, 16, None, 0, 16, 24, need, None, None) == -3
    out = ctypes.c_void_p()
    assert lib.halo_block_stack_create_i4(ctypes.byref(out), ctypes.byref(sh), ctypes.byref(mh), None, None, None, 1, None,
                                          None, None, None) == -1


def test_schedulers_match_oracle_and_feed_the_plan(lib):
    rng = np.random.default_rng(3)
    for _ in range(200):
        n = int(rng.integers(1, 9))
        m = rng.uniform(0.3, 6.3, n).round(1)
        c = rng.uniform(0.6, 1.8, n).round(1)
        Mt = float(rng.uniform(0.2, 1.0) * m.sum())
        assert np.allclose(B.halo_schedule_comp_greedy(m, c, Mt), R.comp_greedy(m, c, Mt), atol=1e-12)
        # the library solves the min-max problem exactly, the oracle bisects as Algorithm 2 does: two different
        # routes, which must meet as the oracle's tolerance shrinks
        r_lib = np.array(B.halo_schedule_min_max(m, c, Mt, 1e-3))
        assert np.allclose(r_lib, R.min_max(m, c, Mt, 1e-10), atol=1e-7)
        assert np.abs(r_lib - R.min_max(m, c, Mt, 1e-3)).max() <= 2e-3
        # invariants of the problem itself: ratios sum to 1, the loads r * Mt fit every budget (the allocation holds
        # the model exactly), and no choice of "full" devices gives a smaller slowest-device time
        assert abs(r_lib.sum() - 1.0) <= 1e-12
        load = r_lib * Mt
        assert (load <= m * (1 + 1e-9)).all()
        best = np.inf
        for mask in range(1 << n):                       # brute force: which devices are filled to their budget
            full = np.array([(mask >> i) & 1 for i in range(n)], dtype=bool)
            if full.all():
                T = (m / c).max() if abs(m.sum() - Mt) <= 1e-9 * Mt else np.inf
            else:
                T = (Mt - m[full].sum()) / c[~full].sum()
            if T < 0 or not np.isfinite(T):
                continue
            if (T * c[~full] <= m[~full] * (1 + 1e-12)).all() and (m[full] <= T * c[full] * (1 + 1e-12)).all():
                best = min(best, T)
        assert np.isclose((load / c).max(), best, rtol=1e-9)
    # ratios -> integer share weights -> Algorithm 3: a device with ratio 0 gets an empty chunk
    r = B.halo_schedule_comp_greedy([4, 5, 3], [2.0, 1.0, 3.0], 6.0)
    w = B.halo_ratios_to_share_weights(r)
    assert w == [32768, 0, 32768]
    plan = B.Plan(20, [0.1, 0.0, 0.3], w, B.SEL_TOPK, 4, 0.0, 0)
    order, _, bnd = plan.describe(16)
    assert order == [1, 0, 2] and bnd == [0, 0, 8, 16]
    for bad in [([1, 1], [1.0, 1.0], 3.0), ([1, -1], [1.0, 1.0], 0.5), ([1, 1], [1.0, 0.0], 0.5)]:
        with pytest.raises(B.HaloError):
            B.halo_schedule_min_max(*bad)
        with pytest.raises(B.HaloError):
            B.halo_schedule_comp_greedy(*bad)


def test_late_devices_match_the_oracle_and_feed_the_plan(lib):
    rng = np.random.default_rng(11)
    for _ in range(200):
        n = int(rng.integers(1, 9))
        units = rng.integers(0, 60, size=n)
        comp = rng.uniform(0.2, 4.0, size=n)
        tau, tc, to = float(rng.uniform(0.05, 2.0)), float(rng.uniform(0.0, 1.0)), float(rng.uniform(1.0, 20.0))
        assert B.halo_late_devices(units, comp, tau, tc, to) == R.late_devices(units, comp, tau, tc, to).tolist()
    # chunks of a plan -> late devices -> a plan in which they never arrive and hold the least critical groups
    loss, w = [0.0, 0.2, 0.1], [2, 1, 1]
    plan = B.Plan(40, loss, w, B.SEL_TOPK, 8, 0.0, 0)
    order, _, bnd = plan.describe(32)
    chunk = [0] * 3
    for pos, dev in enumerate(order):
        chunk[dev] = bnd[pos + 1] - bnd[pos]
    assert chunk == [16, 8, 8]
    late = B.halo_late_devices(chunk, [1.0, 2.0, 0.5], 1.0, 0.0, 10.0)   # busy 16, 4, 16 -> devices 0 and 2 are late
    assert late == [1, 0, 1]
    plan2 = B.Plan(40, [1.0 if l else r for l, r in zip(late, loss)], w, B.SEL_TOPK, 8, 0.0, 0)
    order2, thresh2, _ = plan2.describe(32)
    assert order2[0] == 1 and thresh2[0] == 1 << 32 and thresh2[2] == 1 << 32 and thresh2[1] < 1 << 32
    for bad in [([1, 2], [1.0, 0.0], 1.0, 0.0, 1.0), ([1, -1], [1.0, 1.0], 1.0, 0.0, 1.0), ([1], [1.0], -1.0, 0.0, 1.0)]:
        with pytest.raises(B.HaloError):
            B.halo_late_devices(*bad)
