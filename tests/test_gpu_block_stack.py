"""GPU parity of the transformer-block stack (MHA groups -> FFN groups per layer, LM-head groups at the end):
teacher-forced per block against the oracle through the recorded taps, and the free-running oracle chain for scale."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = U.DEV


def build(wl, H, dh, max_len, r_mha, vocab, lm_group, plan_mha_args):
    code = U.dtype_code(wl)
    L, d, G = wl.n_layers, wl.d_model, wl.n_groups
    mh = B.mha_shape(d, H, dh, max_len, code)
    blocks = []
    for l in range(L):
        Wq, Wk, Wv, Wo = synth.mha_matrices(wl, l, H, DEV)
        Wp = torch.empty((H, 2, dh, d), dtype=wl.torch_dtype, device=DEV)
        B.halo_pack_mha_weights(mh, Wq, Wo, Wp)
        blk = dict(W_ffn=synth.packed_layer(wl, l, DEV), W_mha=Wp, Wk=Wk, Wv=Wv,
                   K=torch.zeros((H, max_len, dh), dtype=wl.torch_dtype, device=DEV),
                   V=torch.zeros((H, max_len, dh), dtype=wl.torch_dtype, device=DEV))
        if l > 0:
            blk["W1_ffn"], blk["W2_ffn"] = synth.predictor(wl, l, DEV)
            mw = synth.Workload("m", L, d, H * 8, 8, r_mha, wl.dtype, (), (), 500, 1, seed=wl.seed + 1)
            blk["W1_mha"], blk["W2_mha"] = synth.predictor(mw, l, DEV)
        blocks.append(blk)
    g = torch.Generator(device="cpu").manual_seed(17)
    W_lm = (torch.randn((vocab, d), generator=g) / 8).to(wl.torch_dtype).to(DEV) if vocab else None
    plan_f = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    plan_a = B.Plan(H, plan_mha_args["loss_rate"], plan_mha_args["share_weight"], B.SEL_TOPK, plan_mha_args["k"], 0.0,
                    plan_mha_args["seed"])
    stack = B.BlockStack(B.ffn_shape(d, wl.d_ffn, wl.group_size, code), mh,
                         B.lm_shape(d, vocab, lm_group, code) if vocab else None,
                         B.pred_shape(d, wl.pred_rank, G, code), B.pred_shape(d, r_mha, H, code), plan_f, plan_a, blocks, W_lm)
    torch.cuda.synchronize()
    return stack, blocks, W_lm


def run(wl, stack, H, vocab, steps, pos0, step0):
    L, G, d, nf = wl.n_layers, wl.n_groups, wl.d_model, wl.n_dev
    h0 = torch.stack([synth.stream_input(wl, 100 + s, DEV)[0] for s in range(steps)])
    mk = lambda shape, dt: torch.zeros(shape, dtype=dt, device=DEV)
    def taps(Gx, n):
        t = dict(x=mk((steps, L, 1, d), wl.torch_dtype), scores=mk((steps, L, Gx), torch.float32),
                 dev_of_group=mk((steps, L, Gx), torch.int32), arrived=mk((steps, L, max(n, 1)), torch.uint8),
                 keep_list=mk((steps, L, Gx), torch.int32), n_keep=mk((steps, L), torch.int32),
                 y=mk((steps, L, 1, d), torch.float32))
        return t, B.Taps(*[t[k].data_ptr() for k in ("x", "scores", "dev_of_group", "arrived", "keep_list", "n_keep", "y")])
    ta, Ta = taps(H, stack.plan_mha.n_dev)
    tf, Tf = taps(G, nf)
    bt = B.BlockTaps(Ta, Tf)
    logits = mk((steps, vocab), torch.float32) if vocab else None
    h_out = mk((steps, d), torch.float32)
    stack.decode(h0, steps, pos0, step0, logits, h_out, bt)
    torch.cuda.synchronize()
    assert stack.status() == 0
    return h0, h_out, logits, ta, tf


@pytest.mark.parametrize("name,layers,H,dh,steps,pos0", [("tiny-f32", 3, 4, 16, 4, 0), ("tinyllama-1.1b-decode", 3, 32, 64, 3, 37),
                                                         ("llama2-7b-decode", 2, 32, 128, 2, 500)])
def test_block_stack_teacher_forced(name, layers, H, dh, steps, pos0):
    if name == "tiny-f32":
        wl = synth.Workload("t", layers, 64, 96, 16, 8, "f32", (0.0, 0.4), (1, 1), 500, steps)
        vocab, lm_group, r_mha, max_len = 50, 7, 8, 16
    else:
        wl = synth.small_variant(synth.workload(name), layers, steps)
        vocab, lm_group, r_mha, max_len = 1000, 256, 64, pos0 + steps + 3
    code = U.dtype_code(wl)
    tol = U.tol_for(wl)
    pm = dict(loss_rate=(0.0, 0.3, 0.6), share_weight=(2, 1, 1), k=max(1, H // 4), seed=11)
    stack, blocks, W_lm = build(wl, H, dh, max_len, r_mha, vocab, lm_group, pm)
    hb = synth.host_bits
    # a context to attend to: positions before pos0 hold random keys / values
    if pos0:
        g = torch.Generator(device=DEV).manual_seed(5)
        for b in blocks:
            b["K"][:, :pos0] = torch.randn((H, pos0, dh), generator=g, device=DEV).to(wl.torch_dtype)
            b["V"][:, :pos0] = torch.randn((H, pos0, dh), generator=g, device=DEV).to(wl.torch_dtype)
    K_start = [hb(b["K"]) for b in blocks]
    V_start = [hb(b["V"]) for b in blocks]
    step0 = 3
    h0, h_out, logits, ta, tf = run(wl, stack, H, vocab, steps, pos0, step0)
    assert stack.last_launches() >= steps * layers * 4             # one launch per step of the path
    L, G, d, nf, na = wl.n_layers, wl.n_groups, wl.d_model, wl.n_dev, 3
    Kc, Vc = [k.copy() for k in K_start], [v.copy() for v in V_start]
    lost_a = lost_f = 0
    for s in range(steps):
        pos = pos0 + s
        h = h0[s].cpu().numpy().astype(np.float64).reshape(1, d)
        _, x0 = R.glue(h, None, code)
        xa_all, xf_all = hb(ta["x"]), hb(tf["x"])
        assert np.abs(R.to_f64(x0) - R.to_f64(xa_all[s, 0])).max() <= 2 ** -7 * np.abs(R.to_f64(x0)).max()
        for l in range(L):
            b = blocks[l]
            x_a, x_f = xa_all[s, l], xf_all[s, l]
            # keys / values of this token, from the recorded input
            R.mha_kv_append(hb(b["Wk"]), hb(b["Wv"]), x_a[0], pos, Kc[l], Vc[l])
            Kg, Vg = hb(b["K"][:, pos]), hb(b["V"][:, pos])
            kk = R.to_f64(Kc[l][:, pos])
            rt = 1e-5 if wl.dtype == "f32" else 2 ** -7
            assert np.abs(R.to_f64(Kg) - kk).max() <= rt * np.abs(kk).max()
            assert np.abs(R.to_f64(Vg) - R.to_f64(Vc[l][:, pos])).max() <= rt * np.abs(kk).max()
            Kc[l][:, pos], Vc[l][:, pos] = Kg, Vg          # teacher forcing: go on from the GPU's own cache bytes
            # MHA scores, selection, outputs
            sa = ta["scores"][s, l].cpu().numpy()
            if l == 0:
                assert (sa == 0).all()
            else:
                ref = R.predict(hb(b["W1_mha"]), hb(b["W2_mha"]), xa_all[s, l - 1])
                assert U.rel_err(sa, ref.astype(np.float64)) <= tol
            sel = R.select(sa, pm["loss_rate"], pm["share_weight"], R.SEL_TOPK, pm["k"], 0.0, pm["seed"], step0 + s, 2 * l,
                           force_all=(l == 0))
            nk = int(ta["n_keep"][s, l].item())
            assert nk == sel["n_keep"] and (ta["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            assert (ta["dev_of_group"][s, l].cpu().numpy() == sel["dev_of_group"]).all()
            assert (ta["arrived"][s, l, :na].cpu().numpy() == sel["arrived"]).all()
            lost_a += int(nk < H)
            P = R.group_mha(hb(b["W_mha"]), x_a[0], Kc[l], Vc[l], pos, sel["keep_list"][:nk], sel["dev_of_group"], na)
            y_ref = P.sum(0)
            y = ta["y"][s, l, 0].cpu().numpy()
            assert U.rel_err(y, y_ref) <= tol, ("mha", s, l)
            h, x_next = R.glue(h, y.astype(np.float64).reshape(1, d), code)
            assert np.abs(R.to_f64(x_next) - R.to_f64(x_f)).max() <= 2 ** -7 * np.abs(R.to_f64(x_next)).max()
            # MLP scores, selection, outputs
            sf = tf["scores"][s, l].cpu().numpy()
            if l == 0:
                assert (sf == 0).all()
            else:
                ref = R.predict(hb(b["W1_ffn"]), hb(b["W2_ffn"]), xf_all[s, l - 1])
                assert U.rel_err(sf, ref.astype(np.float64)) <= tol
            sel = R.select(sf, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, step0 + s, 2 * l + 1,
                           force_all=(l == 0))
            nk = int(tf["n_keep"][s, l].item())
            assert nk == sel["n_keep"] and (tf["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            assert (tf["dev_of_group"][s, l].cpu().numpy() == sel["dev_of_group"]).all()
            if nf:
                assert (tf["arrived"][s, l, :nf].cpu().numpy() == sel["arrived"]).all()
            lost_f += int(nk < G)
            y_ref = R.merge(R.group_ffn(hb(b["W_ffn"]), x_f, sel["keep_list"][:nk], sel["dev_of_group"], nf))
            y = tf["y"][s, l].cpu().numpy()
            assert U.rel_err(y, y_ref) <= tol, ("ffn", s, l)
            h, x_next = R.glue(h, y.astype(np.float64), code)
            if l + 1 < L:
                xr, xg = R.to_f64(x_next), R.to_f64(xa_all[s, l + 1])
                assert np.abs(xr - xg).max() <= 2 ** -7 * np.abs(xr).max()
        assert np.abs(h_out[s].cpu().numpy() - h[0]).max() <= 1e-4 * np.abs(h).max()
        # LM head on the normalised final stream (from the GPU's own stream)
        _, x_o = R.glue(h_out[s].cpu().numpy().astype(np.float64).reshape(1, d), None, code)
        ref = R.group_lm_head(hb(W_lm), x_o, lm_group)
        got = logits[s].cpu().numpy()
        assert np.abs(got - ref[0]).max() <= tol * np.sqrt(np.mean(ref ** 2)) + 2 ** -6 * np.abs(ref).max()
    assert lost_a > 0 and lost_f > 0


def test_block_stack_argument_checks():
    wl = synth.Workload("t", 2, 64, 96, 16, 8, "f32", (0.0,), (1,), 500, 1)
    pm = dict(loss_rate=(0.0,), share_weight=(1,), k=1, seed=0)
    stack, blocks, W_lm = build(wl, 4, 16, 8, 8, 0, 1, pm)
    h0 = torch.zeros((1, 64), dtype=torch.float32, device=DEV)
    with pytest.raises(B.HaloError):
        stack.decode(h0, 1, 8, 0)                        # position beyond the cache
    with pytest.raises(B.HaloError):
        stack.decode(h0, 1, 0, 0, logits=torch.zeros((1, 10), dtype=torch.float32, device=DEV))   # no LM head given


def _qrows(W2d):
    rows, d = W2d.shape
    Q = torch.empty((rows, d // 2), dtype=torch.uint8, device=DEV)
    S = torch.empty((rows, d // 128), dtype=torch.bfloat16, device=DEV)
    B.halo_quantize_rows_i4(d, rows, B.BF16, W2d, Q, S)
    torch.cuda.synchronize()
    return Q, S


@pytest.mark.parametrize("name,layers,H,dh,steps,pos0,sample", [("tinyllama-1.1b-decode", 3, 32, 64, 3, 37, None),
                                                                ("llama2-7b-decode", 2, 32, 128, 2, 500, None),
                                                                ("llama2-7b-decode", 32, 32, 128, 2, 1024, (0, 1, 18, 31))])
def test_block_stack_on_int4_weights_teacher_forced(name, layers, H, dh, steps, pos0, sample):
    """halo_block_stack_create_i4: every weight matrix of the stack as int4 codes + scales (the paper's models are
    4-bit), activations, caches and predictors bf16.  Teacher-forced per block against the oracle's functions on the
    dequantised weights through the recorded taps; logits against the oracle's int4 LM head.  The last case is the
    configuration bench.py times (32 layers, 1024 cached positions, LM head of 32000 rows): selections and the
    residual chain of every block, the oracle's outputs on the sampled layers."""
    wl = synth.small_variant(synth.workload(name), layers, steps)
    vocab, lm_group, r_mha, max_len = (1000 if sample is None else 32000), 256, 64, pos0 + steps + 3
    L, G, d, nf, na = wl.n_layers, wl.n_groups, wl.d_model, wl.n_dev, 3
    tol = U.TOL_BF16
    pm = dict(loss_rate=(0.0, 0.3, 0.6), share_weight=(2, 1, 1), k=max(1, H // 4), seed=11)
    mh = B.mha_shape(d, H, dh, max_len, B.BF16)
    fsh = B.ffn_shape(d, wl.d_ffn, wl.group_size, B.BF16)
    hb = synth.host_bits
    blocks, host = [], []
    g = torch.Generator(device=DEV).manual_seed(5)
    for l in range(L):
        Wq, Wk, Wv, Wo = synth.mha_matrices(wl, l, H, DEV)
        Wp = torch.empty((H, 2, dh, d), dtype=torch.bfloat16, device=DEV)
        B.halo_pack_mha_weights(mh, Wq, Wo, Wp)
        Wf = synth.packed_layer(wl, l, DEV)
        Qf = torch.empty((G, 3, wl.group_size, d // 2), dtype=torch.uint8, device=DEV)
        Sf = torch.empty((G, 3, wl.group_size, d // 128), dtype=torch.bfloat16, device=DEV)
        B.halo_quantize_weights_i4(fsh, Wf, Qf, Sf)
        Qp, Sp = _qrows(Wp.view(H * 2 * dh, d))
        Qk, Sk = _qrows(Wk)
        Qv, Sv = _qrows(Wv)
        K = torch.zeros((H, max_len, dh), dtype=torch.bfloat16, device=DEV)
        V = torch.zeros((H, max_len, dh), dtype=torch.bfloat16, device=DEV)
        K[:, :pos0] = torch.randn((H, pos0, dh), generator=g, device=DEV).to(torch.bfloat16)
        V[:, :pos0] = torch.randn((H, pos0, dh), generator=g, device=DEV).to(torch.bfloat16)
        blk = dict(W_ffn=Qf, S_ffn=Sf, W_mha=Qp, S_mha=Sp, Wk=Qk, Sk=Sk, Wv=Qv, Sv=Sv, K=K, V=V)
        if l > 0:
            blk["W1_ffn"], blk["W2_ffn"] = synth.predictor(wl, l, DEV)
            mw = synth.Workload("m", L, d, H * 8, 8, r_mha, wl.dtype, (), (), 500, 1, seed=wl.seed + 1)
            blk["W1_mha"], blk["W2_mha"] = synth.predictor(mw, l, DEV)
        blocks.append(blk)
        host.append({k: (v.cpu().numpy() if v.dtype == torch.uint8 else hb(v)) for k, v in blk.items() if k not in ("K", "V")}
                    if sample is None or l in sample else None)
        del Wf, Wp, Wq, Wk, Wv, Wo
    gl = torch.Generator(device="cpu").manual_seed(17)
    W_lm = (torch.randn((vocab, d), generator=gl) / 8).to(torch.bfloat16).to(DEV)
    Q_lm, S_lm = _qrows(W_lm)
    plan_f = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    plan_a = B.Plan(H, pm["loss_rate"], pm["share_weight"], B.SEL_TOPK, pm["k"], 0.0, pm["seed"])
    stack = B.BlockStack(fsh, mh, B.lm_shape(d, vocab, lm_group, B.BF16), B.pred_shape(d, wl.pred_rank, G, B.BF16),
                         B.pred_shape(d, r_mha, H, B.BF16), plan_f, plan_a, blocks, Q_lm, S_lm)
    K_start = [hb(b["K"]) for b in blocks]
    V_start = [hb(b["V"]) for b in blocks]
    step0 = 3
    h0, h_out, logits, ta, tf = run(wl, stack, H, vocab, steps, pos0, step0)
    Kc, Vc = [k.copy() for k in K_start], [v.copy() for v in V_start]
    lost_a = lost_f = 0
    for s in range(steps):
        pos = pos0 + s
        h = h0[s].cpu().numpy().astype(np.float64).reshape(1, d)
        xa_all, xf_all = hb(ta["x"]), hb(tf["x"])
        for l in range(L):
            b, hw = blocks[l], host[l]
            heavy = hw is not None                         # the oracle's outputs are recomputed for this layer
            x_a, x_f = xa_all[s, l], xf_all[s, l]
            Kg, Vg = hb(b["K"][:, pos]), hb(b["V"][:, pos])
            if heavy:
                K32, V32 = R.to_f64(Kc[l]).astype(np.float32), R.to_f64(Vc[l]).astype(np.float32)
                R.mha_kv_append_i4(hw["Wk"], hw["Sk"], hw["Wv"], hw["Sv"], x_a[0], pos, K32, V32)
                kk = K32[:, pos].astype(np.float64)
                assert np.abs(R.to_f64(Kg) - kk).max() <= 2 ** -7 * np.abs(kk).max()
                assert np.abs(R.to_f64(Vg) - V32[:, pos]).max() <= 2 ** -7 * np.abs(kk).max()
            Kc[l][:, pos], Vc[l][:, pos] = Kg, Vg          # teacher forcing: go on from the GPU's own cache bytes
            sa = ta["scores"][s, l].cpu().numpy()
            if l > 0 and heavy:
                ref = R.predict(hw["W1_mha"], hw["W2_mha"], xa_all[s, l - 1])
                assert U.rel_err(sa, ref.astype(np.float64)) <= tol
            sel = R.select(sa, pm["loss_rate"], pm["share_weight"], R.SEL_TOPK, pm["k"], 0.0, pm["seed"], step0 + s, 2 * l,
                           force_all=(l == 0))
            nk = int(ta["n_keep"][s, l].item())
            assert nk == sel["n_keep"] and (ta["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            assert (ta["arrived"][s, l, :na].cpu().numpy() == sel["arrived"]).all()
            lost_a += int(nk < H)
            y = ta["y"][s, l, 0].cpu().numpy()
            if heavy:
                P = R.group_mha_i4(hw["W_mha"], hw["S_mha"], H, x_a[0], Kc[l], Vc[l], pos, sel["keep_list"][:nk],
                                   sel["dev_of_group"], na)
                assert U.rel_err(y, P.sum(0)) <= tol, ("mha", s, l)
            h, x_next = R.glue(h, y.astype(np.float64).reshape(1, d), B.BF16)
            assert np.abs(R.to_f64(x_next) - R.to_f64(x_f)).max() <= 2 ** -7 * np.abs(R.to_f64(x_next)).max()
            sf = tf["scores"][s, l].cpu().numpy()
            if l > 0 and heavy:
                ref = R.predict(hw["W1_ffn"], hw["W2_ffn"], xf_all[s, l - 1])
                assert U.rel_err(sf, ref.astype(np.float64)) <= tol
            sel = R.select(sf, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, step0 + s, 2 * l + 1,
                           force_all=(l == 0))
            nk = int(tf["n_keep"][s, l].item())
            assert nk == sel["n_keep"] and (tf["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            lost_f += int(nk < G)
            y = tf["y"][s, l].cpu().numpy()
            if heavy:
                y_ref = R.merge(R.group_ffn_i4(hw["W_ffn"], hw["S_ffn"], x_f, sel["keep_list"][:nk], sel["dev_of_group"], nf))
                assert U.rel_err(y, y_ref) <= tol, ("ffn", s, l)
            h, x_next = R.glue(h, y.astype(np.float64), B.BF16)
            if l + 1 < L:
                xr, xg = R.to_f64(x_next), R.to_f64(xa_all[s, l + 1])
                assert np.abs(xr - xg).max() <= 2 ** -7 * np.abs(xr).max()
        assert np.abs(h_out[s].cpu().numpy() - h[0]).max() <= 1e-4 * np.abs(h).max()
        _, x_o = R.glue(h_out[s].cpu().numpy().astype(np.float64).reshape(1, d), None, B.BF16)
        ref = R.group_lm_head_i4(Q_lm.cpu().numpy(), hb(S_lm), x_o, lm_group)
        got = logits[s].cpu().numpy()
        assert np.abs(got - ref[0]).max() <= tol * np.sqrt(np.mean(ref ** 2)) + 2 ** -6 * np.abs(ref).max()
    assert lost_a > 0 and lost_f > 0


def test_block_stack_full_size_7b_sampled_layers():
    """The configuration bench.py times: 32 layers at the 7B shape (32 heads of 128, 86 groups of 128), 1024 cached
    positions, LM head of 32000 rows.  Selections of EVERY block bit for bit from the recorded scores; keys / values,
    attention, FFN outputs and predictor scores of sampled layers against the oracle from the recorded inputs; the
    residual chain through all 64 blocks from the GPU's own block outputs; sampled logits."""
    wl = synth.small_variant(synth.workload("llama2-7b-decode"), 32, 2)
    H, dh, steps, pos0, vocab, lm_group, r_mha = 32, 128, 2, 1024, 32000, 256, 64
    sample = (0, 1, 17, 31)
    max_len = pos0 + steps + 3
    pm = dict(loss_rate=(0.0, 0.3, 0.6), share_weight=(2, 1, 1), k=H // 2, seed=11)
    stack, blocks, W_lm = build(wl, H, dh, max_len, r_mha, vocab, lm_group, pm)
    hb = synth.host_bits
    g = torch.Generator(device=DEV).manual_seed(5)
    for b in blocks:
        b["K"][:, :pos0] = torch.randn((H, pos0, dh), generator=g, device=DEV).to(torch.bfloat16)
        b["V"][:, :pos0] = torch.randn((H, pos0, dh), generator=g, device=DEV).to(torch.bfloat16)
    step0 = 7
    h0, h_out, logits, ta, tf = run(wl, stack, H, vocab, steps, pos0, step0)
    assert stack.status() == 0
    L, G, d, nf, na = wl.n_layers, wl.n_groups, wl.d_model, wl.n_dev, 3
    tol = U.TOL_BF16
    xa_all, xf_all = hb(ta["x"]), hb(tf["x"])
    lost_a = lost_f = 0
    for s in range(steps):
        pos = pos0 + s
        h = h0[s].cpu().numpy().astype(np.float64).reshape(1, d)
        for l in range(L):
            b = blocks[l]
            x_a, x_f = xa_all[s, l], xf_all[s, l]
            sa, sf = ta["scores"][s, l].cpu().numpy(), tf["scores"][s, l].cpu().numpy()
            sel_a = R.select(sa, pm["loss_rate"], pm["share_weight"], R.SEL_TOPK, pm["k"], 0.0, pm["seed"], step0 + s, 2 * l,
                             force_all=(l == 0))
            sel_f = R.select(sf, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, step0 + s, 2 * l + 1,
                             force_all=(l == 0))
            nka, nkf = int(ta["n_keep"][s, l].item()), int(tf["n_keep"][s, l].item())
            assert nka == sel_a["n_keep"] and (ta["keep_list"][s, l].cpu().numpy() == sel_a["keep_list"]).all()
            assert nkf == sel_f["n_keep"] and (tf["keep_list"][s, l].cpu().numpy() == sel_f["keep_list"]).all()
            assert (ta["dev_of_group"][s, l].cpu().numpy() == sel_a["dev_of_group"]).all()
            assert (tf["dev_of_group"][s, l].cpu().numpy() == sel_f["dev_of_group"]).all()
            lost_a += int(nka < H)
            lost_f += int(nkf < G)
            y_a = ta["y"][s, l, 0].cpu().numpy()
            y_f = tf["y"][s, l].cpu().numpy()
            if l in sample:
                Kc, Vc = hb(b["K"]), hb(b["V"])                   # the cache as the GPU left it (rows up to pos0+steps-1)
                Kr, Vr = Kc.copy(), Vc.copy()
                R.mha_kv_append(hb(b["Wk"]), hb(b["Wv"]), x_a[0], pos, Kr, Vr)
                kk = R.to_f64(Kr[:, pos])
                assert np.abs(R.to_f64(Kc[:, pos]) - kk).max() <= 2 ** -7 * np.abs(kk).max()
                assert np.abs(R.to_f64(Vc[:, pos]) - R.to_f64(Vr[:, pos])).max() <= 2 ** -7 * np.abs(kk).max()
                if l > 0:
                    ref = R.predict(hb(b["W1_mha"]), hb(b["W2_mha"]), xa_all[s, l - 1])
                    assert U.rel_err(sa, ref.astype(np.float64)) <= tol
                    ref = R.predict(hb(b["W1_ffn"]), hb(b["W2_ffn"]), xf_all[s, l - 1])
                    assert U.rel_err(sf, ref.astype(np.float64)) <= tol
                P = R.group_mha(hb(b["W_mha"]), x_a[0], Kc, Vc, pos, sel_a["keep_list"][:nka], sel_a["dev_of_group"], na)
                assert U.rel_err(y_a, P.sum(0)) <= tol, ("mha", s, l)
                y_ref = R.merge(R.group_ffn(hb(b["W_ffn"]), x_f, sel_f["keep_list"][:nkf], sel_f["dev_of_group"], nf))
                assert U.rel_err(y_f, y_ref) <= tol, ("ffn", s, l)
            # the chain, from the GPU's own block outputs
            h, x_next = R.glue(h, y_a.astype(np.float64).reshape(1, d), B.BF16)
            assert np.abs(R.to_f64(x_next) - R.to_f64(x_f)).max() <= 2 ** -7 * np.abs(R.to_f64(x_next)).max()
            h, x_next = R.glue(h, y_f.astype(np.float64), B.BF16)
            if l + 1 < L:
                assert np.abs(R.to_f64(x_next) - R.to_f64(xa_all[s, l + 1])).max() <= 2 ** -7 * np.abs(R.to_f64(x_next)).max()
        assert np.abs(h_out[s].cpu().numpy() - h[0]).max() <= 1e-4 * np.abs(h).max()
        _, x_o = R.glue(h_out[s].cpu().numpy().astype(np.float64).reshape(1, d), None, B.BF16)
        rows = [0, 255, 256, 12345, 31999]
        ref = R.group_lm_head(hb(W_lm), x_o, lm_group)[0]
        got = logits[s].cpu().numpy()
        assert np.abs(got - ref).max() <= tol * np.sqrt(np.mean(ref ** 2)) + 2 ** -6 * np.abs(ref).max(), rows
    assert lost_a > 0 and lost_f > 0
