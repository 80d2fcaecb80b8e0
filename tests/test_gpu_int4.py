"""GPU parity of the int4 group-quantised decode FFN: codes and scales bit for bit, outputs against the oracle's
FFN on the dequantised weights."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U
from tests import test_gpu_stack as TS

pytestmark = pytest.mark.gpu
DEV = U.DEV


def _quantize(wl, Wp):
    G, S, d = wl.n_groups, wl.group_size, wl.d_model
    sh = B.ffn_shape(d, wl.d_ffn, S, U.dtype_code(wl))
    Q = torch.empty((G, 3, S, d // 2), dtype=torch.uint8, device=DEV)
    Sc = torch.empty((G, 3, S, d // 128), dtype=torch.bfloat16, device=DEV)
    B.halo_quantize_weights_i4(sh, Wp, Q, Sc)
    torch.cuda.synchronize()
    return sh, Q, Sc


def _run(sh, Q, Sc, x, keep, dev, n_dev, G):
    n_tok, d = x.shape
    kl = torch.full((G,), -1, dtype=torch.int32, device=DEV)
    if len(keep):
        kl[: len(keep)] = torch.as_tensor(np.asarray(keep, dtype=np.int32), device=DEV)
    nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
    dg = None if dev is None else torch.as_tensor(np.asarray(dev, dtype=np.int32), device=DEV)
    P = torch.full((n_dev + 1, n_tok, d), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.halo_group_ffn_i4(sh, Q, Sc, x, n_tok, kl, nk, dg, n_dev, P, status)
    torch.cuda.synchronize()
    return P.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("dtype,d,G,S,n_tok", [("bf16", 256, 5, 16, 1), ("f32", 384, 4, 24, 2), ("bf16", 4096, 6, 128, 1),
                                               ("bf16", 8192, 3, 40, 1), ("bf16", 1024, 7, 256, 3),
                                               ("bf16", 2048, 9, 64, 2)])
def test_int4_codes_bit_exact_and_ffn_matches_the_oracle(dtype, d, G, S, n_tok):
    wl = synth.Workload("q", 1, d, G * S, S, 16, dtype, (0.0, 0.3, 0.6), (1, 1, 1), 500, 1)
    Wp = synth.packed_layer(wl, 0, DEV)
    sh, Q, Sc = _quantize(wl, Wp)
    hb = synth.host_bits
    Q_ref, Sc_ref = R.quantize_i4(hb(Wp))
    assert (Q.cpu().numpy() == Q_ref).all()                      # integer work: bit exact
    assert (hb(Sc) == Sc_ref).all()
    xw = synth.Workload("qx", 1, d, G * S, S, 16, "bf16", (0.0,), (1,), 500, 1)   # activations are bf16
    x = synth.activation(xw, 3, DEV, n_tok=n_tok)
    dev = (np.arange(G, dtype=np.int32) % 4) - 1
    for keep in (list(range(G)), [g for g in range(G) if g != 1], [G - 1], []):
        P, status = _run(sh, Q, Sc, x, keep, dev, 3, G)
        assert status == 0
        ref = R.group_ffn_i4(Q_ref, Sc_ref, hb(x), keep, dev, 3)
        if not keep:
            assert (P == 0).all()
            continue
        rms = np.sqrt(np.mean(R.merge(ref) ** 2))
        assert np.abs(P - ref).max() <= U.TOL_BF16 * rms, (keep, np.abs(P - ref).max() / rms)


def test_int4_flags_bad_indices_and_works_without_devices():
    wl = synth.Workload("q", 1, 512, 64 * 4, 64, 16, "bf16", (), (), 500, 1)
    Wp = synth.packed_layer(wl, 0, DEV)
    sh, Q, Sc = _quantize(wl, Wp)
    x = synth.activation(wl, 1, DEV)
    P, status = _run(sh, Q, Sc, x, [0, 9, 2], None, 0, 4)
    assert status & B.DEV_BAD_INDEX
    Qh, Sh = Q.cpu().numpy(), synth.host_bits(Sc)
    ref = R.group_ffn_i4(Qh, Sh, synth.host_bits(x), [0, 2])
    assert np.abs(P - ref).max() <= U.TOL_BF16 * np.sqrt(np.mean(ref ** 2))


def test_int4_full_size_7b_block_sampled_groups():
    """One 7B-shaped block (86 groups of 128, d 4096): codes of sampled groups bit exact, outputs of a kept set
    against the oracle."""
    wl = synth.workload("llama2-7b-decode")
    Wp = synth.packed_layer(wl, 2, DEV)
    sh, Q, Sc = _quantize(wl, Wp)
    hb = synth.host_bits
    sample = [0, 41, 85]
    Q_ref, Sc_ref = R.quantize_i4(hb(Wp[sample]))
    assert (Q[sample].cpu().numpy() == Q_ref).all() and (hb(Sc[sample]) == Sc_ref).all()
    x = synth.activation(wl, 5, DEV)
    G = wl.n_groups
    dev = np.full(G, -1, dtype=np.int32)
    dev[41], dev[85] = 0, 2
    # keep exactly the sampled groups: the oracle needs only their weights (re-indexed 0, 1, 2)
    P, status = _run(sh, Q, Sc, x, sample, dev, wl.n_dev, G)
    assert status == 0
    ref = R.group_ffn_i4(Q_ref, Sc_ref, hb(x), [0, 1, 2], np.array([-1, 0, 2], dtype=np.int32), wl.n_dev)
    rms = np.sqrt(np.mean(R.merge(ref) ** 2))
    assert np.abs(P - ref).max() <= U.TOL_BF16 * rms


@pytest.mark.parametrize("form", [-1, 1, 2, 3])
def test_int4_full_size_7b_block_all_groups_kept_every_element(form):
    """The case the benchmark times: one 7B-shaped block on int4 weights with all 86 groups kept (the shared-memory
    ring kernel with a full kept set; also the plain-load form and the tensor-core form).  Codes and scales of the
    whole block bit for bit, every output element of every holder slot against the oracle."""
    B.halo_set_option("i4_no_ring", form)
    try:
        _full_block_all_groups()
    finally:
        B.halo_set_option("i4_no_ring", -1)


def _full_block_all_groups():
    wl = synth.workload("llama2-7b-decode")
    Wp = synth.packed_layer(wl, 3, DEV)
    sh, Q, Sc = _quantize(wl, Wp)
    hb = synth.host_bits
    Q_ref, Sc_ref = R.quantize_i4(hb(Wp))
    assert (Q.cpu().numpy() == Q_ref).all() and (hb(Sc) == Sc_ref).all()
    x = synth.activation(wl, 6, DEV)
    G = wl.n_groups
    dev = (np.arange(G, dtype=np.int32) % (wl.n_dev + 1)) - 1
    keep = list(range(G))
    P, status = _run(sh, Q, Sc, x, keep, dev, wl.n_dev, G)
    assert status == 0
    ref = R.group_ffn_i4(Q_ref, Sc_ref, hb(x), keep, dev, wl.n_dev)
    rms = np.sqrt(np.mean(R.merge(ref) ** 2))
    assert np.abs(P - ref).max() <= U.TOL_BF16 * rms
    # and against the bf16 block it was quantised from: the quantisation error itself stays small
    P16 = R.group_ffn(hb(Wp), hb(x), keep, dev, wl.n_dev)
    diff = R.merge(ref) - R.merge(P16)
    assert np.sqrt(np.mean(diff ** 2)) <= 0.5 * np.sqrt(np.mean(R.merge(P16) ** 2))


@pytest.mark.parametrize("mode", [0, B.STACK_PER_STEP_LAUNCHES, B.STACK_LOAD_SERIAL, B.STACK_DETERMINISTIC])
@pytest.mark.parametrize("name,layers,steps", [("tinyllama-1.1b-decode", 4, 3), ("llama2-7b-decode", 3, 3)])
def test_int4_stack_teacher_forced(name, layers, steps, mode):
    """The FFN stack on int4 weights (halo_stack_create_i4): scores and selections as for the bf16 stack, every block's
    output against the oracle's FFN on the dequantised weights from the recorded input.  Mode 0 and LOAD_SERIAL run as
    one persistent launch, the others as one launch per step of the path."""
    wl = synth.small_variant(synth.workload(name), layers, steps)
    L, G, d, n = wl.n_layers, wl.n_groups, wl.d_model, wl.n_dev
    hb = synth.host_bits
    quant = []
    for l in range(L):
        Wp = synth.packed_layer(wl, l, DEV)
        _, Q, Sc = _quantize(wl, Wp)
        quant.append((Q, Sc))
    preds = [synth.predictor(wl, l, DEV) for l in range(L)]
    plan = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    stack = B.Stack(B.ffn_shape(d, wl.d_ffn, wl.group_size, B.BF16), B.pred_shape(d, wl.pred_rank, G, B.BF16), 1, plan,
                    [q[0] for q in quant], [p[0] for p in preds], [p[1] for p in preds], i4_scales=[q[1] for q in quant])
    h0 = torch.stack([synth.stream_input(wl, s, DEV) for s in range(steps)])
    h_out = torch.empty_like(h0)
    t = dict(x=torch.zeros((steps, L, 1, d), dtype=torch.bfloat16, device=DEV),
             scores=torch.zeros((steps, L, G), dtype=torch.float32, device=DEV),
             dev_of_group=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             arrived=torch.zeros((steps, L, n), dtype=torch.uint8, device=DEV),
             keep_list=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             n_keep=torch.zeros((steps, L), dtype=torch.int32, device=DEV),
             y=torch.zeros((steps, L, 1, d), dtype=torch.float32, device=DEV))
    taps = B.Taps(*[t[k].data_ptr() for k in ("x", "scores", "dev_of_group", "arrived", "keep_list", "n_keep", "y")])
    stack.set_mode(mode)
    stack.decode(h0, steps, 2, h_out, taps)
    torch.cuda.synchronize()
    assert stack.status() == 0
    if mode in (0, B.STACK_LOAD_SERIAL):
        assert stack.last_launches() == 1                  # the persistent kernel
    else:
        assert stack.last_launches() > steps * L
    x_all = hb(t["x"])
    lost = 0
    for s in range(steps):
        for l in range(L):
            scores = t["scores"][s, l].cpu().numpy()
            if l > 0:
                ref = R.predict(hb(preds[l][0]), hb(preds[l][1]), x_all[s, l - 1])
                assert U.rel_err(scores, ref.astype(np.float64)) <= U.TOL_BF16
            sel = R.select(scores, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, 2 + s, l,
                           force_all=(l == 0))
            nk = int(t["n_keep"][s, l].item())
            assert nk == sel["n_keep"] and (t["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            lost += int(nk < G)
            Q, Sc = quant[l]
            P = R.group_ffn_i4(Q.cpu().numpy(), hb(Sc), x_all[s, l], sel["keep_list"][:nk], sel["dev_of_group"], n)
            y_ref = R.merge(P)
            assert U.rel_err(t["y"][s, l].cpu().numpy(), y_ref) <= U.TOL_BF16, (s, l)
    assert lost > 0


def test_int4_stack_full_size_7b_sampled_blocks():
    """The configuration bench.py times: 32 blocks at the 7B shape on int4 weights in ONE persistent launch.  Scores
    and selections of every block (selection integers bit for bit from the recorded scores), the oracle's FFN on the
    dequantised weights for sampled blocks from the recorded inputs."""
    wl = synth.small_variant(synth.workload("llama2-7b-decode"), 32, 2)
    L, G, d, n, steps = wl.n_layers, wl.n_groups, wl.d_model, wl.n_dev, 2
    sample = {(0, 0), (0, 1), (1, 16), (1, 31)}
    hb = synth.host_bits
    quant = []
    for l in range(L):
        Wp = synth.packed_layer(wl, l, DEV)
        _, Q, Sc = _quantize(wl, Wp)
        quant.append((Q, Sc))
        del Wp
    preds = [synth.predictor(wl, l, DEV) for l in range(L)]
    plan = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    stack = B.Stack(B.ffn_shape(d, wl.d_ffn, wl.group_size, B.BF16), B.pred_shape(d, wl.pred_rank, G, B.BF16), 1, plan,
                    [q[0] for q in quant], [p[0] for p in preds], [p[1] for p in preds], i4_scales=[q[1] for q in quant])
    h0 = torch.stack([synth.stream_input(wl, s, DEV) for s in range(steps)])
    h_out = torch.empty_like(h0)
    t = dict(x=torch.zeros((steps, L, 1, d), dtype=torch.bfloat16, device=DEV),
             scores=torch.zeros((steps, L, G), dtype=torch.float32, device=DEV),
             dev_of_group=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             arrived=torch.zeros((steps, L, n), dtype=torch.uint8, device=DEV),
             keep_list=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             n_keep=torch.zeros((steps, L), dtype=torch.int32, device=DEV),
             y=torch.zeros((steps, L, 1, d), dtype=torch.float32, device=DEV))
    taps = B.Taps(*[t[k].data_ptr() for k in ("x", "scores", "dev_of_group", "arrived", "keep_list", "n_keep", "y")])
    stack.decode(h0, steps, 3, h_out, taps)
    torch.cuda.synchronize()
    assert stack.status() == 0 and stack.last_launches() == 1
    x_all = hb(t["x"])
    lost = 0
    for s in range(steps):
        for l in range(L):
            scores = t["scores"][s, l].cpu().numpy()
            sel = R.select(scores, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, 3 + s, l,
                           force_all=(l == 0))
            nk = int(t["n_keep"][s, l].item())
            assert nk == sel["n_keep"] and (t["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            assert (t["dev_of_group"][s, l].cpu().numpy() == sel["dev_of_group"]).all()
            assert (t["arrived"][s, l, :n].cpu().numpy() == sel["arrived"]).all()
            lost += int(nk < G)
            if (s, l) in sample:
                if l > 0:
                    ref = R.predict(hb(preds[l][0]), hb(preds[l][1]), x_all[s, l - 1])
                    assert U.rel_err(scores, ref.astype(np.float64)) <= U.TOL_BF16
                Q, Sc = quant[l]
                P = R.group_ffn_i4(Q.cpu().numpy(), hb(Sc), x_all[s, l], sel["keep_list"][:nk], sel["dev_of_group"], n)
                assert U.rel_err(t["y"][s, l].cpu().numpy(), R.merge(P)) <= U.TOL_BF16, (s, l)
    assert lost > 0


@pytest.mark.parametrize("d,G,S", [(256, 5, 16), (4096, 6, 128), (1024, 7, 256)])
def test_int4_dequantise_is_exact(d, G, S):
    """halo_dequantize_weights_i4: every element IS the oracle's (nibble - 8) * s (the format's scales have 5
    significant bits, so the value is a bf16 number and the cast below loses nothing); with a kept list only the named
    groups are written, a bad index is reported."""
    wl = synth.Workload("q", 1, d, G * S, S, 16, "bf16", (), (), 500, 1)
    Wp = synth.packed_layer(wl, 1, DEV)
    sh, Q, Sc = _quantize(wl, Wp)
    exact = R.dequantize_i4(Q.cpu().numpy(), synth.host_bits(Sc))                 # fp32, exact
    as_bf16 = torch.from_numpy(exact).to(torch.bfloat16)
    assert (as_bf16.to(torch.float32).numpy() == exact).all()
    want = synth.host_bits(as_bf16)
    out = torch.full((G, 3, S, d), 7.0, dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.halo_dequantize_weights_i4(sh, Q, Sc, None, None, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and (synth.host_bits(out) == want).all()
    keep = [G - 1, 0, 9, 2]                                                       # 9 is out of range
    kl = torch.full((G,), -1, dtype=torch.int32, device=DEV)
    kl[: len(keep)] = torch.tensor(keep, dtype=torch.int32)
    nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
    out.fill_(7.0)
    B.halo_dequantize_weights_i4(sh, Q, Sc, kl, nk, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) & B.DEV_BAD_INDEX
    got = synth.host_bits(out)
    seven = synth.host_bits(torch.tensor([7.0], dtype=torch.bfloat16))[0]
    for g in range(G):
        assert (got[g] == (want[g] if g in keep else seven)).all(), g


def _int4_prompt_stack(wl):
    L, G, d = wl.n_layers, wl.n_groups, wl.d_model
    quant, host = [], []
    for l in range(L):
        Wp = synth.packed_layer(wl, l, DEV)
        _, Q, Sc = _quantize(wl, Wp)
        quant.append((Q, Sc))
        host.append((Q.cpu().numpy(), synth.host_bits(Sc)))
        del Wp
    preds = [synth.predictor(wl, l, DEV) for l in range(L)]
    plan = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    stack = B.Stack(B.ffn_shape(d, wl.d_ffn, wl.group_size, B.BF16), B.pred_shape(d, wl.pred_rank, G, B.BF16), wl.n_tok,
                    plan, [q[0] for q in quant], [p[0] for p in preds], [p[1] for p in preds],
                    i4_scales=[q[1] for q in quant])

    def ffn_ref(l, x, keep, dev):
        return R.group_ffn_i4(host[l][0], host[l][1], x, keep, dev, wl.n_dev)
    return stack, preds, ffn_ref


@pytest.mark.parametrize("n_tok,d,loss", [(5, 512, (0.0, 0.3, 0.6)), (64, 512, (0.0, 0.3, 0.6)), (300, 256, (0.0, 0.3, 0.6)),
                                          (160, 512, (0.85, 0.9, 0.95))])
def test_int4_stack_prompts(n_tok, d, loss):
    """An int4 stack made for prompts: five tokens go through the decode form token by token, 64, 160 and 300 through
    the tensor-core path on the kept groups turned back into bf16 (exactly: the format's scales have 5 significant
    bits); the last case has devices that mostly fail, so blocks run with a quarter of their groups.  Teacher-forced
    against the oracle's FFN on the dequantised weights through the records; then the run without the y records (down
    projection adding into the residual stream) chained from the recorded inputs."""
    wl = synth.Workload("pq", 3, d, 64 * 12, 64, 64, "bf16", loss, (2, 1, 1), 250, 2, n_tok=n_tok)
    stack, preds, ffn_ref = _int4_prompt_stack(wl)
    h0, h_out, t = TS.run_with_taps(wl, stack, wl.steps)
    lost = TS.check_teacher_forced(wl, None, preds, h0, h_out, t, wl.steps, ffn_ref=ffn_ref)
    assert lost > 0
    plain, t2 = TS.run_without_y(wl, stack, h0, wl.steps)
    assert TS.check_chained_without_y(wl, None, preds, h0, plain, t2, wl.steps, 0, list(range(n_tok)), ffn_ref=ffn_ref) == lost
    upd = float((h_out - h0).double().pow(2).mean().sqrt().item())
    assert (plain - h_out).abs().max().item() <= U.TOL_BF16 * upd


def test_int4_prompt_stack_at_the_benchmarked_shape():
    """512 tokens, d 4096, groups of 128, lossy devices, int4 weights: teacher-forced on sampled token rows, then the
    timed form (no y records) chained from the recorded inputs."""
    wl = synth.workload("llama2-7b-prefill", n_layers=3, steps=1, loss_rate=(0.0, 0.3, 0.5, 0.7))
    stack, preds, ffn_ref = _int4_prompt_stack(wl)
    h0, h_out, t = TS.run_with_taps(wl, stack, wl.steps, step0=5)
    tokens = [0, 127, 128, 300, 511]
    lost = TS.check_teacher_forced(wl, None, preds, h0, h_out, t, wl.steps, step0=5, tokens=tokens, ffn_ref=ffn_ref)
    assert lost > 0
    plain, t2 = TS.run_without_y(wl, stack, h0, wl.steps, step0=5)
    assert TS.check_chained_without_y(wl, None, preds, h0, plain, t2, wl.steps, 5, tokens, ffn_ref=ffn_ref) == lost


def _run_prompt(sh, Q, Sc, x, keep, dev, n_dev, G):
    n_tok, d = x.shape
    kl = torch.full((G,), -1, dtype=torch.int32, device=DEV)
    if len(keep):
        kl[: len(keep)] = torch.as_tensor(np.asarray(keep, dtype=np.int32), device=DEV)
    nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
    dg = None if dev is None else torch.as_tensor(np.asarray(dev, dtype=np.int32), device=DEV)
    P = torch.full((n_dev + 1, n_tok, d), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    need = B.halo_group_ffn_i4_workspace_bytes(sh, n_tok)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device=DEV)
    B.halo_group_ffn_i4_prompt(sh, Q, Sc, x, n_tok, kl, nk, dg, n_dev, P, ws, status)
    torch.cuda.synchronize()
    return P.cpu().numpy(), int(status.item()), need


@pytest.mark.parametrize("d,G,S,n_tok", [(256, 12, 64, 40), (512, 9, 128, 300), (1024, 5, 256, 130), (512, 7, 64, 3),
                                         (384, 6, 24, 20)])
def test_int4_prompt_entry_point_matches_the_oracle(d, G, S, n_tok):
    """halo_group_ffn_i4_prompt: with a workspace the kept groups go through the tensor cores (their dequantised values
    are exact in bf16), without one (few tokens, a group size the tensor-core form does not take) through the decode
    form; per-holder slots against the oracle's FFN on the dequantised weights, every token."""
    wl = synth.Workload("q", 1, d, G * S, S, 16, "bf16", (0.0, 0.3, 0.6), (1, 1, 1), 500, 1)
    Wp = synth.packed_layer(wl, 0, DEV)
    sh, Q, Sc = _quantize(wl, Wp)
    hb = synth.host_bits
    Qh, Sh = Q.cpu().numpy(), hb(Sc)
    x = synth.activation(wl, 4, DEV, n_tok=n_tok)
    dev = (np.arange(G, dtype=np.int32) % 4) - 1
    needs = set()
    for keep in (list(range(G)), [g for g in range(G) if g % 3 != 1][::-1], [G - 1], []):
        P, status, need = _run_prompt(sh, Q, Sc, x, keep, dev, 3, G)
        needs.add(need > 0)
        assert status == 0
        if not keep:
            assert (P == 0).all()
            continue
        ref = R.group_ffn_i4(Qh, Sh, hb(x), keep, dev, 3)
        rms = np.sqrt(np.mean(R.merge(ref) ** 2))
        assert np.abs(P - ref).max() <= U.TOL_BF16 * rms, (keep, np.abs(P - ref).max() / rms)
    assert needs == {n_tok >= 16 and S in (64, 128, 256)}
    if n_tok >= 16 and S in (64, 128, 256):
        with pytest.raises(B.HaloError):                              # a workspace that is too small is refused
            kl = torch.zeros(G, dtype=torch.int32, device=DEV)
            nk = torch.ones(1, dtype=torch.int32, device=DEV)
            Pz = torch.empty((1, n_tok, d), dtype=torch.float32, device=DEV)
            B.halo_group_ffn_i4_prompt(sh, Q, Sc, x, n_tok, kl, nk, None, 0, Pz, torch.empty(1024, dtype=torch.uint8, device=DEV))


def test_int4_prompt_entry_point_full_size_7b_block_sampled_tokens():
    """One 7B-shaped block, 512 tokens, lossy holders, through the tensor cores: sampled token rows of every holder
    slot against the oracle."""
    wl = synth.workload("llama2-7b-decode")
    Wp = synth.packed_layer(wl, 1, DEV)
    sh, Q, Sc = _quantize(wl, Wp)
    del Wp
    hb = synth.host_bits
    Qh, Sh = Q.cpu().numpy(), hb(Sc)
    xw = synth.workload("llama2-7b-decode", n_tok=512)
    x = synth.activation(xw, 8, DEV, n_tok=512)
    G = wl.n_groups
    dev = (np.arange(G, dtype=np.int32) % (wl.n_dev + 1)) - 1
    keep = [g for g in range(G) if g % 7 != 3]
    P, status, need = _run_prompt(sh, Q, Sc, x, keep, dev, wl.n_dev, G)
    assert status == 0 and need > 0
    tokens = [0, 127, 128, 255, 256, 400, 511]
    ref = R.group_ffn_i4(Qh, Sh, hb(x)[tokens], keep, dev, wl.n_dev)
    rms = np.sqrt(np.mean(R.merge(ref) ** 2))
    assert np.abs(P[:, tokens] - ref).max() <= U.TOL_BF16 * rms


def test_int4_quantiser_extreme_magnitudes_bit_exact():
    """Blocks of very small (fp32 subnormal), very large and mixed magnitudes, all-zero blocks and a lone non-zero
    element: codes and scales of the GPU quantiser equal the oracle's bit for bit (both decide in IEEE fp32 without
    flushing subnormals); the dequantised values stay finite."""
    d, rows = 512, 24
    g = torch.Generator().manual_seed(3)
    W = torch.randn((rows, d), generator=g)
    mags = torch.tensor([1e-42, 3e-39, 1e-30, 1e-8, 1.0, 1e8, 1e30, 3e37])
    W = W * mags.repeat_interleave(3)[:, None]
    W[5, 128:256] = 0.0                                      # an all-zero block
    W[6, :128] = 0.0
    W[6, 77] = -2.5e-41                                      # a lone subnormal
    W = W.to(DEV)
    Q = torch.empty((rows, d // 2), dtype=torch.uint8, device=DEV)
    Sc = torch.empty((rows, d // 128), dtype=torch.bfloat16, device=DEV)
    B.halo_quantize_rows_i4(d, rows, B.F32, W, Q, Sc)
    torch.cuda.synchronize()
    Q_ref, Sc_ref = R.quantize_i4(W.cpu().numpy())
    assert (synth.host_bits(Sc) == Sc_ref).all()
    assert (Q.cpu().numpy() == Q_ref).all()
    assert np.isfinite(R.dequantize_i4(Q_ref, Sc_ref)).all()
