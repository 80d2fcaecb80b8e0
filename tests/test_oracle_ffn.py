"""Pins for the oracle's layout, predictor, group FFN, merge and glue (steps a1, a6..a9)."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import synth


def _silu(a):
    return a / (1.0 + np.exp(-a))


def _dense_swiglu(wg, wu, wd, x):
    """Textbook SwiGLU FFN with fp64 library matmuls on the conventional matrices."""
    a = x @ wg.T
    b = x @ wu.T
    return (_silu(a) * b) @ wd.T


def _small(dtype="f32", d=64, F=96, S=16, r=8, n_dev=3):
    return synth.Workload("small", 2, d, F, S, r, dtype, (0.0, 0.2, 0.5)[:n_dev], (3, 2, 1)[:n_dev], 500, 4)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_pack_roundtrip_and_group_byte_range(dtype):
    wl = _small(dtype)
    wg, wu, wd = (synth.host_bits(t) for t in synth.ffn_matrices(wl, 0))
    P = R.pack_weights(wg, wu, wd, wl.group_size)
    assert P.shape == (wl.n_groups, 3, wl.group_size, wl.d_model)
    ug, uu, ud = R.unpack_weights(P)
    assert (ug == wg).all() and (uu == wu).all() and (ud == wd).all()
    # a group is one contiguous block: [g*3*S*d, (g+1)*3*S*d) elements
    S, d = wl.group_size, wl.d_model
    flat = P.reshape(-1)
    for g in (0, wl.n_groups - 1):
        blk = flat[g * 3 * S * d:(g + 1) * 3 * S * d].reshape(3, S, d)
        assert (blk[0] == wg[g * S:(g + 1) * S]).all()
        assert (blk[1] == wu[g * S:(g + 1) * S]).all()
        assert (blk[2] == wd[:, g * S:(g + 1) * S].T).all()
    assert P.nbytes // wl.n_groups == wl.group_bytes


def test_bf16_widening_is_exact():
    t = torch.randn(1000, generator=torch.Generator().manual_seed(0)).to(torch.bfloat16)
    assert (R.to_f64(synth.host_bits(t)) == t.to(torch.float64).numpy()).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n_tok", [1, 3])
def test_all_groups_kept_equals_dense_swiglu(dtype, n_tok):
    wl = _small(dtype)
    mats = [synth.host_bits(t) for t in synth.ffn_matrices(wl, 1)]
    x = synth.host_bits(synth.activation(wl, 1, n_tok=n_tok))
    P = R.pack_weights(*mats, wl.group_size)
    part = R.group_ffn(P, x, list(range(wl.n_groups)))
    y = R.merge(part)
    ref = _dense_swiglu(*(R.to_f64(m) for m in mats), R.to_f64(x))
    assert np.abs(y - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())


def test_masked_output_is_sum_of_isolated_group_partials():
    wl = _small("bf16")
    mats = [synth.host_bits(t) for t in synth.ffn_matrices(wl, 0)]
    x = synth.host_bits(synth.activation(wl, 2, n_tok=2))
    P = R.pack_weights(*mats, wl.group_size)
    G = wl.n_groups
    dev = np.array([-1, 0, 1, 2, 0, -1], dtype=np.int32)[:G]
    kept = [0, 2, 3, 5]
    part, gp = R.group_ffn(P, x, kept, dev, wl.n_dev, want_group_partials=True)
    # each p_g computed alone
    for i, g in enumerate(kept):
        alone = R.merge(R.group_ffn(P, x, [g]))
        assert np.abs(alone - gp[i]).max() <= 1e-14
        # and against the dense formula restricted to the group's neurons
        S = wl.group_size
        sl = slice(g * S, (g + 1) * S)
        wg, wu, wd = (R.to_f64(m) for m in mats)
        ref = _dense_swiglu(wg[sl], wu[sl], wd[:, sl], R.to_f64(x))
        assert np.abs(alone - ref).max() <= 1e-12
    y = R.merge(part)
    assert np.abs(y - gp.sum(axis=0)).max() <= 1e-12 * max(1.0, np.abs(y).max())
    # slots hold their devices' groups
    for slot in range(wl.n_dev + 1):
        want = sum((gp[i] for i, g in enumerate(kept) if dev[g] + 1 == slot), np.zeros_like(gp[0]))
        assert np.abs(part[slot] - want).max() <= 1e-13


def test_permuting_group_storage_leaves_output_unchanged():
    wl = _small("f32")
    mats = [synth.host_bits(t) for t in synth.ffn_matrices(wl, 0)]
    x = synth.host_bits(synth.activation(wl, 3))
    P = R.pack_weights(*mats, wl.group_size)
    perm = np.random.default_rng(0).permutation(wl.n_groups)
    kept = [1, 4, 5]
    y0 = R.merge(R.group_ffn(P, x, kept))
    inv = np.argsort(perm)
    y1 = R.merge(R.group_ffn(P[perm], x, sorted(int(inv[g]) for g in kept)))
    assert np.abs(y0 - y1).max() <= 1e-13


def test_zero_input_empty_list_and_closed_forms():
    wl = _small("f32")
    mats = [synth.host_bits(t) for t in synth.ffn_matrices(wl, 0)]
    P = R.pack_weights(*mats, wl.group_size)
    x0 = np.zeros((1, wl.d_model), dtype=np.float32)
    assert (R.merge(R.group_ffn(P, x0, list(range(wl.n_groups)))) == 0).all()  # silu(0) = 0
    x = synth.host_bits(synth.activation(wl, 4))
    assert (R.merge(R.group_ffn(P, x, [])) == 0).all()  # skipped block
    # one neuron, d = 2: gate=(2,0) up=(0,3) down col=(1,-1); x=(1.5,0.5): a=3, b=1.5
    Wp = np.zeros((1, 3, 1, 2), dtype=np.float32)
    Wp[0, 0, 0] = [2, 0]
    Wp[0, 1, 0] = [0, 3]
    Wp[0, 2, 0] = [1, -1]
    y = R.merge(R.group_ffn(Wp, np.array([[1.5, 0.5]], dtype=np.float32), [0]))
    h = 3.0 / (1.0 + np.exp(-3.0)) * 1.5
    assert np.allclose(y, [[h, -h]], rtol=1e-15)
    # large positive gate pre-activation: silu(a) -> a
    Wp[0, 0, 0] = [40, 0]
    y = R.merge(R.group_ffn(Wp, np.array([[1.0, 1.0]], dtype=np.float32), [0]))
    assert np.allclose(y, [[120.0, -120.0]], rtol=1e-12)
    # transposed-operand check: gate and up are not interchangeable
    Wp[0, 0, 0] = [2, 0]
    Wq = Wp.copy()
    Wq[0, 0, 0], Wq[0, 1, 0] = Wp[0, 1, 0].copy(), Wp[0, 0, 0].copy()
    ya = R.merge(R.group_ffn(Wp, np.array([[1.5, 0.5]], dtype=np.float32), [0]))
    yb = R.merge(R.group_ffn(Wq, np.array([[1.5, 0.5]], dtype=np.float32), [0]))
    assert not np.allclose(ya, yb)


def test_group_ffn_rejects_bad_group_index():
    wl = _small("f32")
    P = R.pack_weights(*[synth.host_bits(t) for t in synth.ffn_matrices(wl, 0)], wl.group_size)
    with pytest.raises(RuntimeError):
        R.group_ffn(P, np.zeros((1, wl.d_model), np.float32), [wl.n_groups])


def test_merge_flip_identity_and_all_arrived():
    rng = np.random.default_rng(0)
    P = rng.normal(size=(4, 2, 8))
    assert np.allclose(R.merge(P), P.sum(axis=0), rtol=0, atol=1e-15)
    arr = np.array([1, 0, 1], dtype=np.uint8)
    y = R.merge(P, arr)
    assert np.allclose(y, P[0] + P[1] + P[3], atol=1e-15)
    for i in range(3):
        flipped = arr.copy()
        flipped[i] ^= 1
        sign = 1.0 if flipped[i] else -1.0
        assert np.allclose(R.merge(P, flipped) - y, sign * P[i + 1], atol=1e-15)
    assert np.allclose(R.merge(P, np.zeros(3, np.uint8)), P[0])  # the master's own part is never lost


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_predictor_against_library_matmul(dtype):
    wl = _small(dtype, r=12)
    w1, w2 = (synth.host_bits(t) for t in synth.predictor(wl, 0))
    f = synth.host_bits(synth.activation(wl, 5, n_tok=4))
    W1, W2, Fm = R.to_f64(w1), R.to_f64(w2), R.to_f64(f)
    s = R.predict(w1, w2, f, act=R.ACT_RELU)
    ref = np.maximum(Fm @ W1.T, 0.0) @ W2.T
    assert s.dtype == np.float32 and s.shape == (4, wl.n_groups)
    assert (s == ref.astype(np.float32)).mean() > 0.95 and np.abs(s - ref).max() <= 1e-6 * np.abs(ref).max()
    # no activation: collapses to the single matrix product (W2 W1) f
    s_lin = R.predict(w1, w2, f, act=R.ACT_NONE)
    ref_lin = Fm @ (W2 @ W1).T
    assert np.abs(s_lin - ref_lin).max() <= 1e-6 * np.abs(ref_lin).max()
    # relu is inactive when every hidden value is positive
    w1p = np.abs(W1).astype(np.float32)
    fp = np.abs(Fm).astype(np.float32)
    w2f = W2.astype(np.float32)
    assert (R.predict(w1p, w2f, fp, act=R.ACT_RELU) == R.predict(w1p, w2f, fp, act=R.ACT_NONE)).all()
    # relu matters otherwise
    assert not np.allclose(s, s_lin)
    # mean pooling = mean over tokens of the per-token scores; identical tokens = single token
    pooled = R.predict(w1, w2, f, mean_pool=True)
    assert np.abs(pooled - ref.mean(axis=0)).max() <= 1e-6 * np.abs(ref).max()
    same = np.repeat(f[:1], 5, axis=0)
    assert np.abs(R.predict(w1, w2, same, mean_pool=True) - R.predict(w1, w2, f[:1])).max() <= 1e-6


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_glue_residual_and_rmsnorm(dtype):
    rng = np.random.default_rng(1)
    h = rng.normal(size=(2, 64))
    y = rng.normal(size=(2, 64)) * 0.1
    code = R.F32 if dtype == "f32" else R.BF16
    h1, x = R.glue(h, y, code)
    assert np.allclose(h1, h + y, atol=1e-15)
    want = h1 / np.sqrt((h1 ** 2).mean(axis=1, keepdims=True) + 1e-5)
    if dtype == "f32":
        assert (x == want.astype(np.float32)).all()
    else:
        lib_cast = synth.host_bits(torch.from_numpy(want.astype(np.float32)).to(torch.bfloat16))  # library RNE cast
        assert (x == lib_cast).all()
    h2, x2 = R.glue(h, None, code)
    assert np.allclose(h2, h)


def test_layer_composition_matches_its_steps():
    wl = _small("bf16")
    P = R.pack_weights(*[synth.host_bits(t) for t in synth.ffn_matrices(wl, 1)], wl.group_size)
    w1, w2 = (synth.host_bits(t) for t in synth.predictor(wl, 1))
    feat = synth.host_bits(synth.activation(wl, 6))
    x = synth.host_bits(synth.activation(wl, 7))
    out = R.layer(P, w1, w2, feat, x, wl.loss_rate, wl.share_weight, R.SEL_TOPK, 2, 0.0, 9, 4, 1)
    s = R.predict(w1, w2, feat)
    sel = R.select(s, wl.loss_rate, wl.share_weight, R.SEL_TOPK, 2, 0.0, 9, 4, 1)
    y = R.merge(R.group_ffn(P, x, sel["keep_list"][: sel["n_keep"]], sel["dev_of_group"], wl.n_dev))
    assert (out["scores"] == s).all() and out["n_keep"] == sel["n_keep"]
    assert (out["keep_list"] == sel["keep_list"]).all()
    assert np.abs(out["y"] - y).max() <= 1e-15


def test_prefill_one_token_equals_decode():
    wl = _small("bf16")
    P = R.pack_weights(*[synth.host_bits(t) for t in synth.ffn_matrices(wl, 1)], wl.group_size)
    w1, w2 = (synth.host_bits(t) for t in synth.predictor(wl, 1))
    x = synth.host_bits(synth.activation(wl, 8, n_tok=3))
    multi = R.layer(P, w1, w2, x, x, wl.loss_rate, wl.share_weight, R.SEL_TOPK, 3, 0.0, 0, 0, 1)
    # one mask for the whole prompt; each token's output is the decode output under that mask
    for t in range(3):
        part = R.group_ffn(P, x[t:t + 1], multi["keep_list"][: multi["n_keep"]])
        assert np.abs(R.merge(part)[0] - multi["y"][t]).max() <= 1e-13
    single = R.layer(P, w1, w2, x[:1], x[:1], wl.loss_rate, wl.share_weight, R.SEL_TOPK, 3, 0.0, 0, 0, 1)
    assert (single["scores"] == R.predict(w1, w2, x[:1])).all()
