"""GPU parity: every entry point of libhalo against the CPU fp64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = U.DEV


def _wl(dtype="bf16", d=512, F=768, S=64, r=64, loss=(0.0, 0.2, 0.6), shares=(3, 2, 1), **kw):
    return synth.Workload("t", kw.pop("n_layers", 2), d, F, S, r, dtype, tuple(loss), tuple(shares),
                          kw.pop("keep_permille", 500), kw.pop("steps", 2), **kw)


# ---- a2..a5 ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("G,n_dev", [(1, 1), (43, 2), (86, 4), (108, 8), (257, 3), (1024, 32), (88, 0)])
@pytest.mark.parametrize("mode", [B.SEL_TOPK, B.SEL_THRESHOLD])
def test_select_bit_exact(G, n_dev, mode):
    rng = np.random.default_rng(G * 31 + n_dev)
    rho = rng.uniform(0, 0.6, n_dev).round(2)
    w = rng.integers(1, 5, n_dev)
    k = int(rng.integers(0, G + 1))
    theta = 0.1
    plan = B.Plan(G, rho, w, mode, k, theta, seed=1234567890123)
    for trial in range(6):
        s = rng.normal(size=G).astype(np.float32)
        if trial == 1:
            s = np.round(s)  # many ties
        if trial == 2 and G > 4:
            s[1] = np.nan; s[2] = -0.0; s[3] = 0.0; s[4] = np.inf
        if trial == 3:
            s[:] = 0.5
        force = trial == 4
        gpu, _ = U.gpu_select(plan, torch.from_numpy(s).to(DEV), step=trial * 7, layer=trial + 1, force_all=force)
        ref = R.select(s, rho, w, mode, k, theta, 1234567890123, trial * 7, trial + 1, force)
        U.assert_select_equal(gpu, ref)


def test_select_arrival_stream_matches_oracle_over_many_steps():
    wl = synth.workload("tiny")
    plan = B.Plan(wl.n_groups, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    s = torch.randn(wl.n_groups, generator=torch.Generator().manual_seed(1))
    sd = s.to(DEV)
    lost = 0
    for step in range(0, 1000, 7):
        gpu, _ = U.gpu_select(plan, sd, step=step, layer=3)
        ref = R.select(s.numpy(), wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, step, 3)
        U.assert_select_equal(gpu, ref)
        lost += int(gpu["n_keep"] < wl.n_groups)
    assert 0 < lost < 143  # both outcomes occur


# ---- a1 ----------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,d,r,G,n_tok", [("f32", 256, 32, 43, 1), ("bf16", 2048, 128, 88, 1),
                                                ("bf16", 4096, 256, 86, 3), ("bf16", 5120, 512, 108, 1),
                                                ("f32", 264, 40, 5, 2)])
@pytest.mark.parametrize("act", [B.ACT_RELU, B.ACT_NONE])
def test_predict_scores(dtype, d, r, G, n_tok, act):
    wl = _wl(dtype, d=d, F=G * 8, S=8, r=r)
    W1, W2 = synth.predictor(wl, 1, DEV)
    feat = synth.activation(wl, 3, DEV, n_tok=n_tok)
    tol = U.tol_for(wl)
    for pool in ([False, True] if n_tok > 1 else [False]):
        s, status = U.gpu_predict(U.dtype_code(wl), W1, W2, feat, mean_pool=pool, act=act)
        ref = R.predict(synth.host_bits(W1), synth.host_bits(W2), synth.host_bits(feat), act=act, mean_pool=pool)
        assert status == 0
        assert s.shape == ref.shape
        assert U.rel_err(s.cpu().numpy(), ref.astype(np.float64)) <= tol


# ---- layout ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_pack_weights_bit_exact(dtype):
    wl = _wl(dtype, d=264, F=6 * 24, S=24)
    wg, wu, wd = synth.ffn_matrices(wl, 0, DEV)
    out = torch.empty((wl.n_groups, 3, wl.group_size, wl.d_model), dtype=wl.torch_dtype, device=DEV)
    B.halo_pack_weights(B.ffn_shape(wl.d_model, wl.d_ffn, wl.group_size, U.dtype_code(wl)), wg, wu, wd, out)
    torch.cuda.synchronize()
    ref = R.pack_weights(synth.host_bits(wg), synth.host_bits(wu), synth.host_bits(wd), wl.group_size)
    assert (synth.host_bits(out) == ref).all()


# ---- a6..a9 ------------------------------------------------------------------------------------------------

def _ffn_case(wl, layer, keep, dev_of_group=None, n_tok=1):
    Wp = synth.packed_layer(wl, layer, DEV)
    x = synth.activation(wl, 11 + layer, DEV, n_tok=n_tok)
    n_dev = wl.n_dev if dev_of_group is not None else 0
    P, status = U.gpu_group_ffn(wl, Wp, x, keep, dev_of_group, n_dev)
    ref = R.group_ffn(synth.host_bits(Wp), synth.host_bits(x), keep, dev_of_group, n_dev)
    return P, ref, status


def test_tiny_config_all_kept_single_group_and_empty():
    wl = synth.workload("tiny")
    G = wl.n_groups
    P, ref, status = _ffn_case(wl, 0, list(range(G)))
    assert status == 0 and U.rel_err(P.cpu().numpy(), ref) <= U.TOL_F32
    # dense SwiGLU on the same bytes through a library matmul (fp64) as a second witness
    Wp = synth.host_bits(synth.packed_layer(wl, 0, DEV)).astype(np.float64)
    x = synth.host_bits(synth.activation(wl, 11, DEV)).astype(np.float64)
    a = Wp[:, 0].reshape(-1, wl.d_model) @ x[0]
    b = Wp[:, 1].reshape(-1, wl.d_model) @ x[0]
    dense = (a / (1 + np.exp(-a)) * b) @ Wp[:, 2].reshape(-1, wl.d_model)
    assert U.rel_err(P[0, 0].cpu().numpy(), dense) <= U.TOL_F32
    for g in (0, G - 1):
        P, ref, _ = _ffn_case(wl, 0, [g])
        assert U.rel_err(P.cpu().numpy(), ref) <= U.TOL_F32
    P, ref, status = _ffn_case(wl, 0, [])
    assert status == 0 and (P == 0).all().item() and (ref == 0).all()


@pytest.mark.parametrize("name", ["tiny", "tinyllama-1.1b-decode", "llama2-7b-decode", "llama2-13b-decode"])
def test_group_ffn_full_layer_shapes_with_slots(name):
    """One full-size layer of every decode workload, kept set and holders from the oracle's selection."""
    wl = synth.workload(name)
    G = wl.n_groups
    scores = np.random.default_rng(3).normal(size=G).astype(np.float32)
    for step in (0, 5):
        sel = R.select(scores, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, step, 2)
        keep = sel["keep_list"][: sel["n_keep"]]
        P, ref, status = _ffn_case(wl, 1, keep, sel["dev_of_group"])
        assert status == 0
        tol = U.tol_for(wl)
        y = U.gpu_merge(P).cpu().numpy()
        y_ref = R.merge(ref)
        assert U.rel_err(y, y_ref) <= tol
        # every holder's slot, measured against the merged output's scale
        rms = np.sqrt(np.mean(y_ref ** 2))
        assert np.abs(P.cpu().numpy() - ref).max() <= tol * rms
        # slots of devices that did not arrive hold nothing
        for i, a in enumerate(sel["arrived"]):
            if not a:
                assert (P[i + 1] == 0).all().item()


@pytest.mark.parametrize("dtype,d,S", [("bf16", 520, 24), ("f32", 264, 10), ("bf16", 5120, 16), ("bf16", 8192, 8)])
def test_group_ffn_ragged_shapes_multi_token(dtype, d, S):
    wl = _wl(dtype, d=d, F=S * 7, S=S)
    dev = np.array([-1, 0, 1, 2, 2, 0, -1], dtype=np.int32)
    keep = [0, 1, 3, 4, 6]
    P, ref, status = _ffn_case(wl, 0, keep, dev, n_tok=3)
    assert status == 0
    rms = np.sqrt(np.mean(R.merge(ref) ** 2))
    assert np.abs(P.cpu().numpy() - ref).max() <= U.tol_for(wl) * rms


def test_group_ffn_flags_bad_indices_and_skips_them():
    wl = _wl("f32", d=256, F=64, S=16)
    Wp = synth.packed_layer(wl, 0, DEV)
    x = synth.activation(wl, 1, DEV)
    P, status = U.gpu_group_ffn(wl, Wp, x, [0, 99, 2])
    assert status & B.DEV_BAD_INDEX
    ref = R.group_ffn(synth.host_bits(Wp), synth.host_bits(x), [0, 2])
    assert U.rel_err(P.cpu().numpy(), ref) <= U.TOL_F32


def test_merge_and_glue():
    rng = torch.Generator(device=DEV).manual_seed(5)
    P = torch.randn((5, 3, 520), generator=rng, device=DEV)
    arr = [1, 0, 1, 1]
    y = U.gpu_merge(P, arr).cpu().numpy()
    ref = R.merge(P.cpu().numpy().astype(np.float64), arr)
    assert np.abs(y - ref).max() <= 1e-6
    assert np.abs(U.gpu_merge(P).cpu().numpy() - P.cpu().numpy().astype(np.float64).sum(0)).max() <= 1e-5
    h = torch.randn((3, 520), generator=rng, device=DEV)
    yt = torch.from_numpy(y.astype(np.float32)).to(DEV)
    for code, tdt in ((B.F32, torch.float32), (B.BF16, torch.bfloat16)):
        h_out = torch.empty_like(h)
        x_out = torch.empty((3, 520), dtype=tdt, device=DEV)
        B.halo_glue(520, 3, code, h, yt, h_out, x_out)
        torch.cuda.synchronize()
        h_ref, x_ref = R.glue(h.cpu().numpy(), yt.cpu().numpy(), code)
        assert np.abs(h_out.cpu().numpy() - h_ref).max() <= 1e-6
        xr = R.to_f64(x_ref)
        xg = R.to_f64(synth.host_bits(x_out))
        assert np.abs(xg - xr).max() <= (1e-6 if code == B.F32 else 2 ** -7) * np.abs(xr).max()


# ---- whole layer, tiny config (fp32): selection must coincide with the oracle's own ----------------------------

def test_tiny_layer_end_to_end_masks_over_steps():
    wl = synth.workload("tiny")
    Wp, W1, W2 = U.layer_tensors(wl, 0)
    x = synth.activation(wl, 0, DEV)
    plan = B.Plan(wl.n_groups, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    scores, status = U.gpu_predict(B.F32, W1, W2, x)
    hb = synth.host_bits
    s_ref = R.predict(hb(W1), hb(W2), hb(x))
    assert U.rel_err(scores.cpu().numpy(), s_ref.astype(np.float64)) <= U.TOL_F32
    outcomes = set()
    for step in range(0, 40):
        gpu, dev_bufs = U.gpu_select(plan, scores, step, 1)
        # gate 1: same fp32 scores -> identical integers
        ref_same = R.select(scores.cpu().numpy(), wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0,
                            wl.seed, step, 1)
        U.assert_select_equal(gpu, ref_same)
        # gate 3: the oracle's own scores give the same selection in fp32
        full = R.layer(hb(Wp), hb(W1), hb(W2), hb(x), hb(x), wl.loss_rate, wl.share_weight, R.SEL_TOPK,
                       R.k_of(wl), 0.0, wl.seed, step, 1)
        assert (full["keep_list"] == gpu["keep_list"]).all()
        keep = gpu["keep_list"][: gpu["n_keep"]]
        P, st = U.gpu_group_ffn(wl, Wp, x, keep, gpu["dev_of_group"], wl.n_dev)
        y = U.gpu_merge(P, gpu["arrived"]).cpu().numpy()
        assert st == 0 and U.rel_err(y, full["y"]) <= U.TOL_F32
        outcomes.add(gpu["n_keep"])
    # the lossy device both arrives and is lost; when lost, exactly its chunk of the less-critical groups goes
    order, _, bnd = R.plan(wl.loss_rate, wl.share_weight, wl.n_groups - R.k_of(wl))
    j = list(order).index(1)
    assert outcomes == {wl.n_groups - int(bnd[j + 1] - bnd[j]), wl.n_groups}


# ---- failure detection: a wait that runs out becomes a status bit, not a hang ----------------------------------

def test_bounded_waits_time_out_cleanly_and_context_stays_usable():
    flag = torch.zeros(1, dtype=torch.int32, device=DEV)       # nothing ever sets it
    report = torch.zeros(2, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.halo_selftest_bounded_wait(flag, 2_000_000, report, status)   # about a millisecond per wait
    t1.record()
    torch.cuda.synchronize()
    assert report.tolist() == [128, 1]
    assert int(status.item()) & B.DEV_TIMEOUT
    assert "timed out" in B.status_message(int(status.item()))
    assert t0.elapsed_time(t1) < 200.0                               # bounded: milliseconds, not forever
    # the context is intact: an ordinary call still works and is clean
    wl = synth.workload("tiny")
    P, st = U.gpu_group_ffn(wl, synth.packed_layer(wl, 0, DEV), synth.activation(wl, 1, DEV), [0, 1, 2])
    assert st == 0 and torch.isfinite(P).all().item()
    with pytest.raises(B.HaloError):
        B.halo_selftest_bounded_wait(flag, 0, report, status)


# ---- true importance of the groups (what the predictors regress) -------------------------------------------------

@pytest.mark.parametrize("name", ["tiny", "tinyllama-1.1b-decode", "llama2-7b-decode"])
def test_group_importance_matches_isolated_group_partials(name):
    wl = synth.workload(name)
    Wp = synth.packed_layer(wl, 1, DEV)
    x = synth.activation(wl, 21, DEV)
    norms = torch.full((wl.n_groups,), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.halo_group_importance(B.ffn_shape(wl.d_model, wl.d_ffn, wl.group_size, U.dtype_code(wl)), Wp, x, norms,
                            dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    _, gp = R.group_ffn(synth.host_bits(Wp), synth.host_bits(x), list(range(wl.n_groups)), want_group_partials=True)
    ref = np.sqrt((gp[:, 0, :] ** 2).sum(axis=1))
    got = norms.cpu().numpy()
    assert np.abs(got - ref).max() <= U.tol_for(wl) * ref.mean()


def test_fitted_predictor_beats_random_dropping_on_structured_groups():
    """Calibration tool end to end (small): a predictor fitted to the true importance must expose better groups
    to loss than a random choice, and can be no better than the true ranking."""
    from paper_2601_11676_b200 import calibrate
    res = calibrate.run("tinyllama-1.1b-decode", n_train=1024, n_test=16, drop_fractions=(0.25,), train_steps=200,
                        verbose=False)
    e = res["drop"][0][1]
    assert e["true-least"] <= e["predicted-least"] + 1e-6
    assert e["predicted-least"] < e["random"] < e["true-most"]
    assert res["bottom_quarter_overlap"] > 0.35


# ---- one block in one call ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name,n_tok", [("tiny", 1), ("llama2-7b-decode", 1), ("tinyllama-1.1b-decode", 40)])
def test_layer_fused_matches_oracle_layer(name, n_tok):
    wl = synth.workload(name)
    code = U.dtype_code(wl)
    Wp, W1, W2 = U.layer_tensors(wl, 2)
    feat = synth.activation(wl, 30, DEV, n_tok=n_tok)
    x = synth.activation(wl, 31, DEV, n_tok=n_tok)
    G, n, d = wl.n_groups, wl.n_dev, wl.d_model
    plan = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    ffn = B.ffn_shape(d, wl.d_ffn, wl.group_size, code)
    pred = B.pred_shape(d, wl.pred_rank, G, code)
    scores = torch.zeros(G, dtype=torch.float32, device=DEV)
    dg = torch.zeros(G, dtype=torch.int32, device=DEV)
    arr = torch.zeros(max(n, 1), dtype=torch.uint8, device=DEV)
    keep = torch.zeros(G, dtype=torch.uint8, device=DEV)
    y = torch.zeros((n_tok, d), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = None
    hb = synth.host_bits
    sample = list(range(n_tok)) if n_tok <= 4 else [0, 17, n_tok - 1]
    for step in (0, 3):
        ws = B.halo_layer_fused(ffn, pred, plan, Wp, W1, W2, feat, x, n_tok, step, 5, False, scores, dg, arr, keep, y,
                                ws, status)
        torch.cuda.synchronize()
        assert B.halo_read_status(int(status.item())) == "clean"
        s_ref = R.predict(hb(W1), hb(W2), hb(feat), mean_pool=n_tok > 1)
        assert U.rel_err(scores.cpu().numpy(), s_ref.astype(np.float64)) <= U.tol_for(wl)
        sel = R.select(scores.cpu().numpy(), wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed,
                       step, 5)
        assert (dg.cpu().numpy() == sel["dev_of_group"]).all() and (keep.cpu().numpy() == sel["keep"]).all()
        assert (arr.cpu().numpy()[:n] == sel["arrived"]).all()
        P = R.group_ffn(hb(Wp), hb(x)[sample], sel["keep_list"][: sel["n_keep"]], sel["dev_of_group"], n)
        assert U.rel_err(y[sample].cpu().numpy(), R.merge(P)) <= U.tol_for(wl)
