"""GPU parity of the FFN stack runner: teacher-forced per block against the oracle, via the recorded taps."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = U.DEV


def build_stack(wl, mode=B.SEL_TOPK, threshold=0.0, act=B.ACT_RELU):
    code = U.dtype_code(wl)
    Wp = [synth.packed_layer(wl, l, DEV) for l in range(wl.n_layers)]
    preds = [synth.predictor(wl, l, DEV) for l in range(wl.n_layers)]
    plan = B.Plan(wl.n_groups, wl.loss_rate, wl.share_weight, mode, B.k_of(wl), threshold, wl.seed)
    stack = B.Stack(B.ffn_shape(wl.d_model, wl.d_ffn, wl.group_size, code),
                    B.pred_shape(wl.d_model, wl.pred_rank, wl.n_groups, code, act), wl.n_tok, plan, Wp,
                    [p[0] for p in preds], [p[1] for p in preds])
    return stack, Wp, preds


def run_with_taps(wl, stack, steps, step0=0):
    L, G, d, T, n = wl.n_layers, wl.n_groups, wl.d_model, wl.n_tok, wl.n_dev
    h0 = torch.stack([synth.stream_input(wl, step0 + s, DEV) for s in range(steps)])
    h_out = torch.empty_like(h0)
    t = dict(x=torch.zeros((steps, L, T, d), dtype=wl.torch_dtype, device=DEV),
             scores=torch.zeros((steps, L, G), dtype=torch.float32, device=DEV),
             dev_of_group=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             arrived=torch.zeros((steps, L, max(n, 1)), dtype=torch.uint8, device=DEV),
             keep_list=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             n_keep=torch.zeros((steps, L), dtype=torch.int32, device=DEV),
             y=torch.zeros((steps, L, T, d), dtype=torch.float32, device=DEV))
    taps = B.Taps(*[t[k].data_ptr() for k in ("x", "scores", "dev_of_group", "arrived", "keep_list", "n_keep", "y")])
    stack.decode(h0, steps, step0, h_out, taps)
    torch.cuda.synchronize()
    assert stack.status() == 0
    return h0, h_out, t


def run_without_y(wl, stack, h0, steps, step0=0):
    """The same run recording everything except the blocks' outputs."""
    L, G, d, T, n = wl.n_layers, wl.n_groups, wl.d_model, wl.n_tok, wl.n_dev
    h_out = torch.empty_like(h0)
    t = dict(x=torch.zeros((steps, L, T, d), dtype=wl.torch_dtype, device=DEV),
             scores=torch.zeros((steps, L, G), dtype=torch.float32, device=DEV),
             dev_of_group=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             arrived=torch.zeros((steps, L, max(n, 1)), dtype=torch.uint8, device=DEV),
             keep_list=torch.zeros((steps, L, G), dtype=torch.int32, device=DEV),
             n_keep=torch.zeros((steps, L), dtype=torch.int32, device=DEV))
    taps = B.Taps(*[t[k].data_ptr() for k in ("x", "scores", "dev_of_group", "arrived", "keep_list", "n_keep")], None)
    stack.decode(h0, steps, step0, h_out, taps)
    torch.cuda.synchronize()
    assert stack.status() == 0
    return h_out, t


def check_teacher_forced(wl, Wp, preds, h0, h_out, t, steps, step0=0, mode=R.SEL_TOPK, threshold=0.0,
                         act=R.ACT_RELU, tokens=None, ffn_ref=None):
    """`tokens`: token rows whose FFN output the oracle recomputes (all when None); scores, selection integers and
    the glue chain are always checked in full.  `ffn_ref(l, x, keep_list, dev_of_group)`: the oracle's holder slots
    of block l when the weights are not a packed bf16/fp32 tensor (int4 stacks)."""
    hb = synth.host_bits
    tol = U.tol_for(wl)
    L, n = wl.n_layers, wl.n_dev
    x_all = hb(t["x"])
    lost_layers = 0
    for s in range(steps):
        h = h0[s].cpu().numpy().astype(np.float64)
        # first input: normalised stream
        _, x0 = R.glue(h, None, U.dtype_code(wl))
        assert np.abs(R.to_f64(x0) - R.to_f64(x_all[s, 0])).max() <= 2 ** -7 * np.abs(R.to_f64(x0)).max()
        for l in range(L):
            x_l = x_all[s, l]
            scores = t["scores"][s, l].cpu().numpy()
            if l == 0:
                assert (scores == 0).all()
            else:
                s_ref = R.predict(hb(preds[l][0]), hb(preds[l][1]), x_all[s, l - 1], act=act, mean_pool=wl.n_tok > 1)
                assert U.rel_err(scores, s_ref.astype(np.float64)) <= tol
            sel = R.select(scores, wl.loss_rate, wl.share_weight, mode, R.k_of(wl), threshold, wl.seed,
                           step0 + s, l, force_all=(l == 0))
            nk = int(t["n_keep"][s, l].item())
            assert nk == sel["n_keep"]
            assert (t["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            assert (t["dev_of_group"][s, l].cpu().numpy() == sel["dev_of_group"]).all()
            if n:
                assert (t["arrived"][s, l, :n].cpu().numpy() == sel["arrived"]).all()
            lost_layers += int(nk < wl.n_groups)
            y = t["y"][s, l].cpu().numpy()
            x_ffn = x_l if tokens is None else x_l[tokens]
            if ffn_ref is not None:
                P = ffn_ref(l, x_ffn, sel["keep_list"][:nk], sel["dev_of_group"])
            else:
                P = R.group_ffn(hb(Wp[l]), x_ffn, sel["keep_list"][:nk], sel["dev_of_group"], n)
            y_ref = R.merge(P)
            assert U.rel_err(y if tokens is None else y[tokens], y_ref) <= tol, (s, l)
            # glue, from the GPU's own y: next input and residual stream
            h, x_next = R.glue(h, y.astype(np.float64), U.dtype_code(wl))
            if l + 1 < L:
                xr, xg = R.to_f64(x_next), R.to_f64(x_all[s, l + 1])
                assert np.abs(xr - xg).max() <= 2 ** -7 * np.abs(xr).max()
        assert np.abs(h_out[s].cpu().numpy() - h).max() <= 1e-4 * np.abs(h).max()
    return lost_layers


@pytest.mark.parametrize("mode", [0, 1])  # 0: persistent single kernel where supported; 1: one launch per step
@pytest.mark.parametrize("name,layers,steps", [("tinyllama-1.1b-decode", 4, 3), ("llama2-7b-decode", 3, 2),
                                               ("llama2-13b-decode", 3, 2)])
def test_stack_decode_teacher_forced(name, layers, steps, mode):
    wl = synth.small_variant(synth.workload(name), layers, steps)
    stack, Wp, preds = build_stack(wl)
    stack.set_mode(mode)
    h0, h_out, t = run_with_taps(wl, stack, steps, step0=3)
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, steps, step0=3)
    assert stack.last_launches() == 1 if mode == 0 else stack.last_launches() > 1


def test_stack_persistent_many_steps_with_losses_and_single_layer():
    """Longer run of the single-kernel path: lossy devices so kept sets change every block; and a 1-block stack."""
    wl = synth.Workload("m", 5, 2048, 64 * 12, 64, 128, "bf16", (0.0, 0.3, 0.6), (2, 1, 1), 250, 10)
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps)
    assert stack.last_launches() == 1
    lost = check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps)
    assert lost > 0
    one = synth.Workload("o", 1, 4096, 128 * 5, 128, 64, "bf16", (0.5,), (1,), 400, 3)
    stack, Wp, preds = build_stack(one)
    h0, h_out, t = run_with_taps(one, stack, one.steps)
    check_teacher_forced(one, Wp, preds, h0, h_out, t, one.steps)


def test_stack_persistent_everything_lost_gives_identity_blocks():
    """k = 0 and every device always lost: from the second block on nothing is kept and the stream passes through."""
    wl = synth.Workload("z", 3, 4096, 128 * 4, 128, 64, "bf16", (1.0, 1.0), (1, 1), 0, 2)
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps)
    assert (t["n_keep"][:, 1:] == 0).all().item() and (t["n_keep"][:, 0] == wl.n_groups).all().item()
    assert (t["y"][:, 1:] == 0).all().item()
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps)


def test_stack_small_f32_many_steps_sees_losses():
    wl = synth.Workload("s", 3, 256, 688, 16, 32, "f32", (0.0, 0.3, 0.5), (2, 1, 1), 300, 12)
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps)
    lost = check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps)
    assert lost > 0


def test_stack_host_entry_matches_device_entry():
    wl = synth.small_variant(synth.workload("tinyllama-1.1b-decode"), 3, 5)
    stack, _, _ = build_stack(wl)
    h0 = torch.stack([synth.stream_input(wl, s, DEV) for s in range(5)])
    out_dev = torch.empty_like(h0)
    stack.decode(h0, 5, 0, out_dev)
    torch.cuda.synchronize()
    h0_host = h0.cpu().pin_memory()
    out_host = torch.empty_like(h0_host).pin_memory()
    stack.decode_host(h0_host, 5, 0, out_host)
    assert np.abs(out_host.numpy() - out_dev.cpu().numpy()).max() <= 1e-3 * np.abs(out_host.numpy()).max()


def test_stack_multi_token_prompt():
    wl = synth.Workload("p", 3, 512, 768, 64, 64, "bf16", (0.0, 0.3, 0.6), (1, 1, 1), 500, 1, n_tok=5)
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, 1)
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, 1)


@pytest.mark.parametrize("n_tok,d", [(64, 512), (160, 512), (300, 256)])
def test_stack_prompt_on_the_tensor_core_path(n_tok, d):
    """Prompts long enough for the tensor-core kernels (one 128-token tile, and more than one): teacher-forced
    against the oracle through the taps; then the same run without taps, where the down projection adds straight
    into the residual stream, must give the same stream."""
    wl = synth.Workload("pt", 3, d, 64 * 12, 64, 64, "bf16", (0.0, 0.3, 0.6), (2, 1, 1), 250, 2, n_tok=n_tok)
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps)
    lost = check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps)
    assert lost > 0
    upd = float((h_out - h0).double().pow(2).mean().sqrt().item())
    for mode in (0, B.STACK_PROMPT_ONE_LAUNCH):
        stack.set_mode(mode)
        plain, t2 = run_without_y(wl, stack, h0, wl.steps)
        assert check_chained_without_y(wl, Wp, preds, h0, plain, t2, wl.steps, 0, list(range(n_tok))) == lost
        assert (plain - h_out).abs().max().item() <= U.TOL_BF16 * upd


def check_chained_without_y(wl, Wp, preds, h0, h_out, t, steps, step0, tokens, act=R.ACT_RELU, ffn_ref=None):
    """Check of a run that recorded every block's input x, scores and selection but NOT its output y (the form in
    which the prompt path adds the down projection straight into the residual stream).  Scores and selection
    integers are checked as usual.  For the sampled token rows the oracle computes y_l from the recorded x_l and
    chains the stream h_{l+1} = h_l + y_l from the given h_0; the GPU's x_{l+1} must equal the normalised chain and
    the final stream must equal its end, each within the sum of the per-block output bounds collected so far (the
    GPU's error in y_l given the same x_l is what the bound covers; nothing else enters)."""
    hb = synth.host_bits
    tol = U.tol_for(wl)
    L, n, code = wl.n_layers, wl.n_dev, U.dtype_code(wl)
    x_all = hb(t["x"])
    lost = 0
    for s in range(steps):
        h = h0[s].cpu().numpy().astype(np.float64)[tokens]
        _, x0 = R.glue(h, None, code)
        assert np.abs(R.to_f64(x0) - R.to_f64(x_all[s, 0][tokens])).max() <= 2 ** -7 * np.abs(R.to_f64(x0)).max()
        bound = 0.0
        for l in range(L):
            scores = t["scores"][s, l].cpu().numpy()
            if l == 0:
                assert (scores == 0).all()
            else:
                s_ref = R.predict(hb(preds[l][0]), hb(preds[l][1]), x_all[s, l - 1], act=act, mean_pool=wl.n_tok > 1)
                assert U.rel_err(scores, s_ref.astype(np.float64)) <= tol
            sel = R.select(scores, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, step0 + s, l,
                           force_all=(l == 0))
            nk = int(t["n_keep"][s, l].item())
            assert nk == sel["n_keep"]
            assert (t["keep_list"][s, l].cpu().numpy() == sel["keep_list"]).all()
            assert (t["dev_of_group"][s, l].cpu().numpy() == sel["dev_of_group"]).all()
            if n:
                assert (t["arrived"][s, l, :n].cpu().numpy() == sel["arrived"]).all()
            lost += int(nk < wl.n_groups)
            if ffn_ref is not None:
                y_ref = R.merge(ffn_ref(l, x_all[s, l][tokens], sel["keep_list"][:nk], sel["dev_of_group"]))
            else:
                y_ref = R.merge(R.group_ffn(hb(Wp[l]), x_all[s, l][tokens], sel["keep_list"][:nk], sel["dev_of_group"], n))
            bound += tol * float(np.sqrt(np.mean(y_ref ** 2)))
            h, x_next = R.glue(h, y_ref, code)
            if l + 1 < L:
                xr, xg = R.to_f64(x_next), R.to_f64(x_all[s, l + 1][tokens])
                scale = np.sqrt(np.mean(h ** 2, axis=-1, keepdims=True) + 1e-5)       # x = h / scale
                assert (np.abs(xr - xg) <= bound / scale + 2 ** -7 * np.abs(xr) + 1e-6).all(), (s, l)
        assert np.abs(h_out[s].cpu().numpy()[tokens] - h).max() <= bound + 1e-5 * np.abs(h).max(), s
    return lost


@pytest.mark.parametrize("variant", ["wide_rank512", "group256", "three_token_tiles", "everything_lost", "no_devices",
                                     "linear_predictor", "full_tile_of_tokens"])
def test_prompt_stack_single_launch_variants(variant):
    """The one-launch prompt kernel under the other settings: a 5120-wide block with a 512-unit predictor (two unit
    tiles), the paper's 256-neuron groups (two hidden tiles per group), three token tiles with a ragged last one,
    k = 0 with every device always lost (blocks from the second on keep nothing), no devices at all, a predictor
    without the ReLU, exactly 256 tokens.  Checked by chaining the oracle's outputs from the recorded inputs."""
    kw = dict(act=B.ACT_RELU)
    if variant == "wide_rank512":
        wl = synth.Workload("v", 3, 5120, 128 * 6, 128, 512, "bf16", (0.0, 0.4, 0.8), (1, 2, 1), 300, 1, n_tok=300)
    elif variant == "group256":
        wl = synth.Workload("v", 3, 512, 256 * 5, 256, 64, "bf16", (0.1, 0.6), (1, 1), 400, 2, n_tok=257)
    elif variant == "three_token_tiles":
        wl = synth.Workload("v", 4, 256, 64 * 12, 64, 64, "bf16", (0.0, 0.3, 0.6), (2, 1, 1), 250, 1, n_tok=700)
    elif variant == "everything_lost":
        wl = synth.Workload("v", 3, 512, 128 * 4, 128, 64, "bf16", (1.0, 1.0), (1, 1), 0, 2, n_tok=200)
    elif variant == "no_devices":
        wl = synth.Workload("v", 3, 512, 64 * 9, 64, 128, "bf16", (), (), 400, 1, n_tok=129)
    elif variant == "linear_predictor":
        wl = synth.Workload("v", 3, 1024, 128 * 5, 128, 200, "bf16", (0.2, 0.7), (1, 1), 334, 2, n_tok=160)
        kw.update(act=B.ACT_NONE)
    else:
        wl = synth.Workload("v", 2, 768, 64 * 7, 64, 96, "bf16", (0.0, 0.5), (3, 1), 430, 1, n_tok=256)
    stack, Wp, preds = build_stack(wl, **kw)
    stack.set_mode(B.STACK_PROMPT_ONE_LAUNCH)
    h0 = torch.stack([synth.stream_input(wl, s, DEV) for s in range(wl.steps)])
    plain, t = run_without_y(wl, stack, h0, wl.steps, step0=2)
    assert stack.last_launches() == wl.steps                      # one launch per prompt
    check_chained_without_y(wl, Wp, preds, h0, plain, t, wl.steps, 2, list(range(0, wl.n_tok, 7)) + [wl.n_tok - 1],
                            act=kw["act"])
    if variant == "everything_lost":
        assert (t["n_keep"][:, 1:] == 0).all().item()
        # nothing kept from the second block on: the stream stays what the first block left
    # and the same stack through the one-launch-per-step path gives the same selections
    stack.set_mode(0)
    plain1, t1 = run_without_y(wl, stack, h0, wl.steps, step0=2)
    assert stack.last_launches() > wl.steps
    assert (t1["n_keep"] == t["n_keep"]).all().item()
    upd = (plain1 - h0).double().pow(2).mean().sqrt().item()
    assert (plain - plain1).abs().max().item() <= U.TOL_BF16 * max(upd, 1e-3) * 4


def test_prompt_stack_at_the_benchmarked_shape():
    """The prompt path as bench.py times it: 512 tokens, d 4096, groups of 128, lossy devices.  First with every
    record, teacher-forced block by block against the oracle on a sample of token rows; then the form that is
    timed, in which the down projection adds straight into the residual stream and the predictor runs beside the
    FFN, recording inputs, scores and selections only, checked by chaining the oracle's outputs.  The two runs'
    final streams agree within the path's bound (not more tightly: one bf16 rounding of x that falls the other way
    is amplified by the following blocks)."""
    wl = synth.workload("llama2-7b-prefill", n_layers=3, steps=2, loss_rate=(0.0, 0.3, 0.5, 0.7))
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps, step0=5)
    tokens = [0, 127, 128, 255, 256, 300, 511]
    lost = check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps, step0=5, tokens=tokens)
    assert lost > 0                                   # some block really ran with groups dropped
    upd = float((h_out - h0).double().pow(2).mean().sqrt().item())
    for mode in (0, B.STACK_PROMPT_ONE_LAUNCH):      # the default (timed) form, and the one-launch-per-prompt kernel
        stack.set_mode(mode)
        plain, t2 = run_without_y(wl, stack, h0, wl.steps, step0=5)
        assert (stack.last_launches() == wl.steps) == (mode != 0)
        lost2 = check_chained_without_y(wl, Wp, preds, h0, plain, t2, wl.steps, 5, tokens)
        assert lost2 == lost
        assert (plain - h_out).abs().max().item() <= U.TOL_BF16 * upd


@pytest.mark.parametrize("name,steps,sample,permille", [
    ("llama2-7b-decode", 3, [(0, 0), (0, 1), (1, 16), (2, 30), (2, 31)], 500),
    ("llama2-7b-decode", 2, [(0, 1), (1, 17), (1, 31)], 300),
    ("llama2-7b-decode", 2, [(0, 1), (1, 9)], 700),
    ("llama2-7b-decode", 2, [(0, 2), (1, 31)], 1000),
    ("llama2-13b-decode", 2, [(0, 1), (1, 20), (1, 39)], 500),
    ("tinyllama-1.1b-decode", 4, [(0, 0), (1, 1), (2, 11), (3, 21)], 500),
])
def test_full_size_stack_in_bench_configuration_sampled_blocks(name, steps, sample, permille):
    """The whole stack at its stated size, run the way bench.py times it (one persistent launch), at every keep
    ratio of the 7B sweep; the oracle recomputes a sample of (step, block) records from the recorded inputs.
    Selection integers are checked for every record (they are cheap), FFN outputs for the sample."""
    wl = synth.workload(name, keep_permille=permille)
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, steps, step0=7)
    assert stack.last_launches() == 1
    hb = synth.host_bits
    x_all = hb(t["x"])
    n = wl.n_dev
    scores_all = t["scores"].cpu().numpy()
    kl_all, dg_all, nk_all = t["keep_list"].cpu().numpy(), t["dev_of_group"].cpu().numpy(), t["n_keep"].cpu().numpy()
    arr_all = t["arrived"].cpu().numpy()
    for s in range(steps):
        for l in range(wl.n_layers):
            sel = R.select(scores_all[s, l], wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed,
                           7 + s, l, force_all=(l == 0))
            assert int(nk_all[s, l]) == sel["n_keep"], (s, l)
            assert (kl_all[s, l] == sel["keep_list"]).all() and (dg_all[s, l] == sel["dev_of_group"]).all()
            assert (arr_all[s, l, :n] == sel["arrived"]).all()
    for s, l in sample:
        if l > 0:
            s_ref = R.predict(hb(preds[l][0]), hb(preds[l][1]), x_all[s, l - 1])
            assert U.rel_err(scores_all[s, l], s_ref.astype(np.float64)) <= U.TOL_BF16
        nk = int(nk_all[s, l])
        P = R.group_ffn(hb(Wp[l]), x_all[s, l], kl_all[s, l][:nk], dg_all[s, l], n)
        y_ref = R.merge(P)
        assert U.rel_err(t["y"][s, l].cpu().numpy(), y_ref) <= U.TOL_BF16, (s, l)
    # the residual stream that comes out is the input plus every block's recorded output
    for s in range(steps):
        want = h0[s].double() + t["y"][s].double().sum(dim=0)
        assert (h_out[s].double() - want).abs().max().item() <= 1e-3 * want.abs().max().item()


def test_stack_with_the_papers_group_size_of_256():
    """Sec. II-A fixes the group size to 256: 43 groups at the 7B FFN width, persistent kernel, two blocks."""
    wl = synth.Workload("g256", 2, 4096, 11008, 256, 256, "bf16", (0.0, 0.1, 0.5), (2, 1, 1), 500, 3)
    assert wl.n_groups == 43
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps)
    assert stack.last_launches() == 1
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps)


@pytest.mark.parametrize("variant", ["threshold", "act_none", "no_devices", "d8192", "single_device_lossless"])
def test_stack_persistent_variants(variant):
    """Persistent path under the other settings of the method: threshold choice of the critical groups, a linear
    predictor, no virtual devices at all, the widest supported d_model, one lossless device."""
    kw = dict(mode=B.SEL_TOPK, threshold=0.0, act=B.ACT_RELU)
    if variant == "threshold":
        wl = synth.Workload("v", 4, 2048, 64 * 20, 64, 128, "bf16", (0.0, 0.5, 1.0), (1, 2, 1), 0, 6)
        kw.update(mode=B.SEL_THRESHOLD, threshold=0.5)
    elif variant == "act_none":
        wl = synth.Workload("v", 3, 4096, 128 * 6, 128, 64, "bf16", (0.2, 0.7), (1, 1), 334, 4)
        kw.update(act=B.ACT_NONE)
    elif variant == "no_devices":
        wl = synth.Workload("v", 3, 4096, 128 * 5, 128, 64, "bf16", (), (), 400, 3)
    elif variant == "d8192":
        wl = synth.Workload("v", 3, 8192, 32 * 9, 32, 64, "bf16", (0.0, 0.6), (1, 3), 300, 4)
    else:
        wl = synth.Workload("v", 3, 5120, 128 * 4, 128, 512, "bf16", (0.0,), (7,), 250, 3)
    stack, Wp, preds = build_stack(wl, **kw)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps)
    assert stack.last_launches() == 1      # really the persistent kernel
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps, mode=kw["mode"], threshold=kw["threshold"], act=kw["act"])
    if variant == "threshold":
        nk = t["n_keep"][:, 1:].cpu().numpy()
        assert nk.min() < wl.n_groups and len(np.unique(nk)) > 1   # the critical count really varies with the scores


def test_long_runs_are_split_into_several_persistent_launches():
    """The persistent kernel's counters are 32 bit, so very long runs are cut into several launches; forced here
    with a tiny limit: the arrival draws and records must continue seamlessly across the cut."""
    wl = synth.Workload("c", 3, 2048, 64 * 10, 64, 128, "bf16", (0.0, 0.4, 0.8), (1, 1, 1), 300, 5)
    B.halo_set_option("max_steps_per_launch", 2)
    try:
        stack, Wp, preds = build_stack(wl)
    finally:
        B.halo_set_option("max_steps_per_launch", -1)
    h0, h_out, t = run_with_taps(wl, stack, wl.steps, step0=11)
    assert stack.last_launches() == 3
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, wl.steps, step0=11)
    ref_stack, _, _ = build_stack(wl)
    _, h_ref, t_ref = run_with_taps(wl, ref_stack, wl.steps, step0=11)
    assert ref_stack.last_launches() == 1
    assert (t["keep_list"] == t_ref["keep_list"]).all().item() and (t["n_keep"] == t_ref["n_keep"]).all().item()
    assert (h_out - h_ref).abs().max().item() <= 1e-3 * h_ref.abs().max().item()


@pytest.mark.parametrize("mode", [0, B.STACK_PRED_SERIAL, B.STACK_DETERMINISTIC])
@pytest.mark.parametrize("name,layers,steps", [("tinyllama-1.1b-decode", 5, 4), ("llama2-7b-decode", 4, 3)])
def test_stack_with_the_ring_extended_into_tensor_memory(name, layers, steps, mode):
    """Option "tmem_ring": landed stages are moved on into tensor memory (tcgen05.cp) and the consumers read them from
    there (tcgen05.ld).  Same path, same records: teacher-forced against the oracle, same selections as the default."""
    wl = synth.small_variant(synth.workload(name), layers, steps)
    B.halo_set_option("tmem_ring", 1)
    try:
        stack, Wp, preds = build_stack(wl)
    finally:
        B.halo_set_option("tmem_ring", -1)
    stack.set_mode(mode)
    h0, h_out, t = run_with_taps(wl, stack, steps, step0=5)
    assert stack.last_launches() == 1 and stack.status() == 0
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, steps, step0=5)
    ref_stack, _, _ = build_stack(wl)
    _, h_ref, t_ref = run_with_taps(wl, ref_stack, steps, step0=5)
    assert (t["n_keep"] == t_ref["n_keep"]).all().item() and (t["keep_list"] == t_ref["keep_list"]).all().item()


@pytest.mark.parametrize("mode", [B.STACK_PRED_SERIAL, B.STACK_LOAD_SERIAL, B.STACK_PRED_SERIAL | B.STACK_LOAD_SERIAL])
@pytest.mark.parametrize("name,layers,steps", [("tinyllama-1.1b-decode", 4, 3), ("llama2-7b-decode", 3, 2),
                                               ("llama2-13b-decode", 3, 2)])
def test_stack_ablation_arms_teacher_forced(name, layers, steps, mode):
    """The arms of the overlap ablation (predictor not beside the previous block's stream, no weights fetched across
    the block boundary, both) compute the same path: teacher-forced against the oracle like the default mode."""
    wl = synth.small_variant(synth.workload(name), layers, steps)
    stack, Wp, preds = build_stack(wl)
    stack.set_mode(mode)
    h0, h_out, t = run_with_taps(wl, stack, steps, step0=9)
    assert stack.last_launches() == 1                       # still the persistent kernel
    check_teacher_forced(wl, Wp, preds, h0, h_out, t, steps, step0=9)
    stack.set_mode(0)
    _, h_ref, t_ref = run_with_taps(wl, stack, steps, step0=9)
    assert (t["n_keep"] == t_ref["n_keep"]).all().item() and (t["keep_list"] == t_ref["keep_list"]).all().item()


@pytest.mark.parametrize("name,layers,steps", [("tinyllama-1.1b-decode", 6, 4), ("llama2-7b-decode", 4, 3),
                                               ("llama2-13b-decode", 3, 2)])
def test_stack_deterministic_mode_is_bitwise_repeatable(name, layers, steps):
    """Fixed batch assignment and fixed-order sums: two runs give the same bits in every recorded output and in the
    final stream; the results are the default mode's within the tolerance (and teacher-forced against the oracle).
    With the memory checker closed this is what exposes a race: a racy kernel does not repeat."""
    wl = synth.small_variant(synth.workload(name), layers, steps)
    stack, Wp, preds = build_stack(wl)
    stack.set_mode(B.STACK_DETERMINISTIC)
    h0, h_a, t_a = run_with_taps(wl, stack, steps, step0=4)
    assert stack.last_launches() == 1
    runs = [run_with_taps(wl, stack, steps, step0=4) for _ in range(3)]
    for _, h_b, t_b in runs:
        assert torch.equal(h_a, h_b) and torch.equal(t_a["y"], t_b["y"]) and torch.equal(t_a["x"].view(torch.int16), t_b["x"].view(torch.int16))
        assert torch.equal(t_a["scores"], t_b["scores"]) and torch.equal(t_a["keep_list"], t_b["keep_list"])
    check_teacher_forced(wl, Wp, preds, h0, h_a, t_a, steps, step0=4)
    stack.set_mode(0)
    _, h_d, t_d = run_with_taps(wl, stack, steps, step0=4)
    upd = (h_d - h0).double().pow(2).mean().sqrt().item()
    assert (h_d - h_a).abs().max().item() <= U.TOL_BF16 * upd


def test_score_margins_and_free_running_drift_7b(capsys):
    """Report for the 7B-shaped stack over 3 steps (printed; run pytest with -s to read it):
      - for every (step, block): the oracle's scores from the recorded input against the GPU's scores, the smallest
        gap between two scores that straddle a boundary of the priority partition (critical cut or a chunk cut), and
        whether the selection made from the oracle's scores differs from the GPU's;
      - the drift of the free-running GPU stream against a chain computed by the oracle alone from the same h_0.
    Gated: a selection may differ only where a straddling gap is smaller than the score tolerance (two groups whose
    scores the two sides cannot order the same way); inside a chunk the order does not matter."""
    wl = synth.workload("llama2-7b-decode")
    steps, step0 = 3, 21
    stack, Wp, preds = build_stack(wl)
    h0, h_out, t = run_with_taps(wl, stack, steps, step0=step0)
    hb = synth.host_bits
    L, G, n, k = wl.n_layers, wl.n_groups, wl.n_dev, R.k_of(wl)
    x_all = hb(t["x"])
    scores_gpu = t["scores"].cpu().numpy()
    kl_gpu, nk_gpu = t["keep_list"].cpu().numpy(), t["n_keep"].cpu().numpy()
    _, _, bnd = R.plan(wl.loss_rate, wl.share_weight, G - k)
    cuts = sorted(set([k] + [k + int(b) for b in bnd[1:-1]]))        # rank positions where the holder changes
    W1 = [None] + [hb(preds[l][0]) for l in range(1, L)]
    W2 = [None] + [hb(preds[l][1]) for l in range(1, L)]
    differing, min_gap_all, worst_score_err = 0, np.inf, 0.0
    for s in range(steps):
        for l in range(1, L):
            s_ref = R.predict(W1[l], W2[l], x_all[s, l - 1]).astype(np.float64)
            bound = U.TOL_BF16 * float(np.sqrt(np.mean(s_ref ** 2)))
            err = float(np.abs(scores_gpu[s, l] - s_ref).max())
            worst_score_err = max(worst_score_err, err / bound)
            assert err <= bound
            srt = np.sort(s_ref)[::-1]
            gap = min(float(srt[c - 1] - srt[c]) for c in cuts if 0 < c < G)
            min_gap_all = min(min_gap_all, gap)
            sel_ref = R.select(s_ref.astype(np.float32), wl.loss_rate, wl.share_weight, R.SEL_TOPK, k, 0.0, wl.seed,
                               step0 + s, l)
            same = sel_ref["n_keep"] == int(nk_gpu[s, l]) and (sel_ref["keep_list"] == kl_gpu[s, l]).all()
            if not same:
                differing += 1
                assert gap <= 2 * bound, (s, l, gap, bound)      # explainable: a straddling pair within the tolerance
    # free-running chain by the oracle alone
    code = U.dtype_code(wl)
    drift = []
    for s in range(steps):
        h = h0[s].cpu().numpy().astype(np.float64)
        x_prev = None
        for l in range(L):
            _, x = R.glue(h, None, code)
            if l == 0:
                scores = np.zeros(G, dtype=np.float32)
            else:
                scores = R.predict(W1[l], W2[l], x_prev)
            sel = R.select(scores, wl.loss_rate, wl.share_weight, R.SEL_TOPK, k, 0.0, wl.seed, step0 + s, l,
                           force_all=(l == 0))
            y = R.merge(R.group_ffn(hb(Wp[l]), x, sel["keep_list"][: sel["n_keep"]], sel["dev_of_group"], n))
            h = h + y
            x_prev = x
        upd = np.sqrt(np.mean((h - h0[s].cpu().numpy()) ** 2))
        drift.append(float(np.abs(h_out[s].cpu().numpy() - h).max() / upd))
    with capsys.disabled():
        print(f"\n[7B stack, {steps} steps x {L - 1} scored blocks] worst score error {worst_score_err:.3f} of the bound; "
              f"smallest straddling gap {min_gap_all:.3e}; selections differing from the oracle-score selection: "
              f"{differing} of {steps * (L - 1)}; free-running drift max|h - h_oracle| / rms(update) per step: "
              + ", ".join(f"{v:.2e}" for v in drift))
    assert all(np.isfinite(drift))
