"""Pins for the oracle's MHA neuron groups (one head + its output-projection slice)."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import synth


def _setup(dtype="f32", d=64, H=4, L=12, seed=0):
    wl = synth.Workload("a", 1, d, 64, 16, 8, dtype, (0.0, 0.3), (1, 1), 500, 1, seed=seed)
    Wq, Wk, Wv, Wo = (synth.host_bits(t) for t in synth.mha_matrices(wl, 0, H))
    dh = d // H
    cache_dt = np.float32 if dtype == "f32" else np.uint16
    K = np.zeros((H, L, dh), dtype=cache_dt)
    V = np.zeros((H, L, dh), dtype=cache_dt)
    xs = [synth.host_bits(synth.activation(wl, 100 + t))[0] for t in range(L)]
    for t in range(L):
        R.mha_kv_append(Wk, Wv, xs[t], t, K, V)
    return wl, (Wq, Wk, Wv, Wo), R.pack_mha(Wq, Wo, H), K, V, xs, H, dh


def _dense_mha(Wq, Wo, x, K, V, pos, H, dh):
    """Textbook multi-head attention for one query token with fp64 library routines."""
    q = (Wq @ x).reshape(H, dh)
    out = np.zeros(H * dh)
    for h in range(H):
        s = K[h, :pos + 1] @ q[h] / np.sqrt(dh)
        w = np.exp(s - s.max()); w /= w.sum()
        out[h * dh:(h + 1) * dh] = w @ V[h, :pos + 1]
    return Wo @ out


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_kv_append_is_the_projection_rounded_to_the_cache_dtype(dtype):
    wl, (Wq, Wk, Wv, Wo), Wp, K, V, xs, H, dh = _setup(dtype)
    x = R.to_f64(xs[3])
    k_ref = (R.to_f64(Wk) @ x).reshape(H, dh)
    if dtype == "f32":
        assert (K[:, 3] == k_ref.astype(np.float32)).all()
    else:
        lib_cast = synth.host_bits(torch.from_numpy(k_ref.astype(np.float32)).to(torch.bfloat16))
        assert (K[:, 3] == lib_cast).all()
    assert np.abs(R.to_f64(V[:, 3]) - (R.to_f64(Wv) @ x).reshape(H, dh)).max() <= 2 ** -8 * np.abs(k_ref).max() + 1e-6


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_all_heads_equal_dense_multi_head_attention(dtype):
    wl, (Wq, Wk, Wv, Wo), Wp, K, V, xs, H, dh = _setup(dtype)
    for pos in (0, 5, 11):
        y = R.group_mha(Wp, xs[pos], K, V, pos, list(range(H)))[0]
        ref = _dense_mha(R.to_f64(Wq), R.to_f64(Wo), R.to_f64(xs[pos]), R.to_f64(K), R.to_f64(V), pos, H, dh)
        assert np.abs(y - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())


def test_first_position_attends_to_itself_only():
    wl, (Wq, Wk, Wv, Wo), Wp, K, V, xs, H, dh = _setup("f32")
    y = R.group_mha(Wp, xs[0], K, V, 0, list(range(H)))[0]
    v0 = R.to_f64(V[:, 0]).reshape(-1)          # softmax over one position is 1: o = v_0
    assert np.abs(y - R.to_f64(Wo) @ v0).max() <= 1e-12


def test_identical_keys_give_the_mean_of_the_values():
    wl, (Wq, Wk, Wv, Wo), Wp, K, V, xs, H, dh = _setup("f32")
    K2 = np.repeat(K[:, :1], K.shape[1], axis=1).copy()
    y = R.group_mha(Wp, xs[7], K2, V, 7, [2])[0]
    o = R.to_f64(V[2, :8]).mean(axis=0)
    assert np.abs(y - R.to_f64(Wo)[:, 2 * dh:3 * dh] @ o).max() <= 1e-12


def test_heads_are_independent_groups_linearity_slots_and_empty():
    wl, (Wq, Wk, Wv, Wo), Wp, K, V, xs, H, dh = _setup("bf16")
    dev = np.array([-1, 0, 1, 0], dtype=np.int32)
    kept = [0, 1, 3]
    P, hp = R.group_mha(Wp, xs[9], K, V, 9, kept, dev, 2, want_head_partials=True)
    for i, h in enumerate(kept):
        alone = R.group_mha(Wp, xs[9], K, V, 9, [h])[0]
        assert np.abs(alone - hp[i]).max() <= 1e-14
    assert np.abs(P[0] - hp[0]).max() <= 1e-14 and np.abs(P[1] - (hp[1] + hp[2])).max() <= 1e-13 and (P[2] == 0).all()
    assert np.abs(R.merge(P[:, None, :])[0] - hp.sum(0)).max() <= 1e-13
    assert (R.group_mha(Wp, xs[9], K, V, 9, []) == 0).all()
    with pytest.raises(RuntimeError):
        R.group_mha(Wp, xs[9], K, V, 9, [H])


def test_permuting_head_storage_leaves_output_unchanged():
    wl, (Wq, Wk, Wv, Wo), Wp, K, V, xs, H, dh = _setup("f32")
    perm = np.array([2, 0, 3, 1])
    y0 = R.group_mha(Wp, xs[4], K, V, 4, [1, 2])[0]
    inv = np.argsort(perm)
    y1 = R.group_mha(Wp[perm], xs[4], K[perm].copy(), V[perm].copy(), 4, sorted(int(inv[h]) for h in (1, 2)))[0]
    assert np.abs(y0 - y1).max() <= 1e-13
