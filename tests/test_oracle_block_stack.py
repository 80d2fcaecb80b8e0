"""Pins of the oracle's transformer-block stack (MHA groups, FFN groups, LM-head groups chained per layer)."""
import numpy as np

from oracle import halo_ref as R


def _dense_reference(h0s, Wq, Wk, Wv, Wo, Wg, Wu, Wd, Wlm, H, dh):
    """A pre-norm transformer written the textbook way in numpy (fp64 arithmetic; activations and cached keys and
    values rounded to float32 where the path stores them), all heads and all neurons active."""
    L = len(Wq)
    d = h0s.shape[1]
    Kc = [np.zeros((0, H, dh)) for _ in range(L)]
    Vc = [np.zeros((0, H, dh)) for _ in range(L)]
    norm = lambda h: (h / np.sqrt(np.mean(h ** 2) + 1e-5)).astype(np.float32).astype(np.float64)
    outs, logits = [], []
    for h in h0s.astype(np.float64):
        for l in range(L):
            x = norm(h)
            q = (Wq[l] @ x).reshape(H, dh)
            k = (Wk[l] @ x).astype(np.float32).astype(np.float64).reshape(1, H, dh)
            v = (Wv[l] @ x).astype(np.float32).astype(np.float64).reshape(1, H, dh)
            Kc[l] = np.concatenate([Kc[l], k]); Vc[l] = np.concatenate([Vc[l], v])
            o = np.zeros((H, dh))
            for hd in range(H):
                sc = Kc[l][:, hd] @ q[hd] / np.sqrt(dh)
                w = np.exp(sc - sc.max()); w /= w.sum()
                o[hd] = w @ Vc[l][:, hd]
            h = h + Wo[l] @ o.reshape(-1)
            x = norm(h)
            a, b = Wg[l] @ x, Wu[l] @ x
            h = h + Wd[l] @ (a / (1 + np.exp(-a)) * b)
        outs.append(h)
        logits.append(Wlm @ norm(h))
    return np.array(outs), np.array(logits)


def _make(rng, L, d, H, dh, F, S, vocab, r=8):
    f32 = lambda *s: rng.normal(0, 0.3, size=s).astype(np.float32)
    Wq, Wk, Wv = [f32(H * dh, d) for _ in range(L)], [f32(H * dh, d) for _ in range(L)], [f32(H * dh, d) for _ in range(L)]
    Wo = [f32(d, H * dh) for _ in range(L)]
    Wg, Wu, Wd = [f32(F, d) for _ in range(L)], [f32(F, d) for _ in range(L)], [f32(d, F) for _ in range(L)]
    Wlm = f32(vocab, d)
    blocks = []
    for l in range(L):
        blocks.append(dict(W_mha=R.pack_mha(Wq[l], Wo[l], H), Wk=Wk[l], Wv=Wv[l],
                           K=np.zeros((H, 8, dh), dtype=np.float32), V=np.zeros((H, 8, dh), dtype=np.float32),
                           W_ffn=R.pack_weights(Wg[l], Wu[l], Wd[l], S),
                           W1_mha=f32(r, d), W2_mha=f32(H, r), W1_ffn=f32(r, d), W2_ffn=f32(F // S, r)))
    return (Wq, Wk, Wv, Wo, Wg, Wu, Wd, Wlm), blocks


def test_block_stack_with_everything_kept_is_a_dense_transformer():
    rng = np.random.default_rng(0)
    L, d, H, dh, F, S, vocab = 3, 64, 4, 16, 96, 16, 50
    mats, blocks = _make(rng, L, d, H, dh, F, S, vocab)
    none = dict(loss_rate=(), share_weight=(), mode=R.SEL_TOPK, k=0, threshold=0.0, seed=0)
    h0s = rng.normal(size=(3, d)).astype(np.float32)
    ref_h, ref_logits = _dense_reference(h0s, *mats, H, dh)
    for t in range(3):
        h, logits, recs = R.block_stack_token(h0s[t], t, t, blocks, mats[-1], 7, none, none, R.F32)
        assert np.allclose(h[0], ref_h[t], rtol=1e-9, atol=1e-9)
        assert np.allclose(logits[0], ref_logits[t], rtol=1e-9, atol=1e-9)
        assert all(r["sel_a"]["n_keep"] == H and r["sel_f"]["n_keep"] == F // S for r in recs)


def test_block_stack_first_layer_reliable_and_separate_draws_per_block():
    rng = np.random.default_rng(1)
    L, d, H, dh, F, S = 3, 64, 4, 16, 96, 16
    mats, blocks = _make(rng, L, d, H, dh, F, S, 10)
    lossy = dict(loss_rate=(0.5, 0.5), share_weight=(1, 1), mode=R.SEL_TOPK, k=1, threshold=0.0, seed=5)
    seen_diff = False
    for step in range(40):
        for b in blocks:
            b["K"][:] = 0; b["V"][:] = 0
        _, _, recs = R.block_stack_token(rng.normal(size=d), 0, step, blocks, None, 1, lossy, lossy, R.F32)
        assert recs[0]["sel_a"]["n_keep"] == H and recs[0]["sel_f"]["n_keep"] == F // S       # first layer: all arrive
        for l in range(1, L):
            # the arrival draws are those of (step, 2l) and (step, 2l+1)
            for i in range(2):
                assert recs[l]["sel_a"]["arrived"][i] == R.arrival(5, step, 2 * l, i, 0.5)
                assert recs[l]["sel_f"]["arrived"][i] == R.arrival(5, step, 2 * l + 1, i, 0.5)
            seen_diff |= (recs[l]["sel_a"]["arrived"] != recs[l]["sel_f"]["arrived"]).any()
    assert seen_diff


def test_block_stack_dropping_heads_and_groups_changes_only_their_contribution():
    """Linearity of the merge through the chain: with the scores fixed by the inputs, the residual update of each
    block equals the sum of the kept heads' / groups' isolated partials."""
    rng = np.random.default_rng(2)
    L, d, H, dh, F, S = 2, 64, 4, 16, 96, 16
    mats, blocks = _make(rng, L, d, H, dh, F, S, 10)
    plan = dict(loss_rate=(1.0,), share_weight=(1,), mode=R.SEL_TOPK, k=2, threshold=0.0, seed=0)   # one dead device
    h, _, recs = R.block_stack_token(rng.normal(size=d), 0, 0, blocks, None, 1, plan, plan, R.F32)
    r1 = recs[1]
    assert r1["sel_a"]["n_keep"] == 2 and r1["sel_f"]["n_keep"] == 2
    kept = r1["sel_a"]["keep_list"][:2]
    _, hp = R.group_mha(blocks[1]["W_mha"], r1["x_a"][0], blocks[1]["K"], blocks[1]["V"], 0, kept, want_head_partials=True)
    assert np.allclose(r1["y_a"][0], hp.sum(0), rtol=1e-12, atol=1e-12)
