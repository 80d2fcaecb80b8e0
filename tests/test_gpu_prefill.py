"""GPU parity of the tensor-core (many-token) form of halo_group_ffn against the oracle."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = U.DEV


def _wl(d, G, S, n_dev=3):
    return synth.Workload("pf", 1, d, G * S, S, 64, "bf16", (0.0, 0.2, 0.6)[:n_dev], (3, 2, 1)[:n_dev], 500, 1)


@pytest.mark.parametrize("d,G,S,n_tok", [(256, 3, 128, 32), (512, 5, 64, 130), (1024, 4, 128, 257), (256, 6, 64, 16),
                                         (512, 3, 256, 200), (256, 2, 256, 64), (384, 3, 256, 130)])
def test_prefill_ffn_small_shapes_all_tokens(d, G, S, n_tok):
    wl = _wl(d, G, S)
    sh = B.ffn_shape(d, G * S, S, B.BF16)
    assert B.halo_group_ffn_workspace_bytes(sh, n_tok, wl.n_dev) >= n_tok * G * S * 2
    Wp = synth.packed_layer(wl, 0, DEV)
    x = synth.activation(wl, 1, DEV, n_tok=n_tok)
    dev = np.array([-1, 0, 1, 2, 0, -1], dtype=np.int32)[:G]
    for keep in ([g for g in range(G) if g != 1], list(range(G)), [G - 1], []):
        P, status = U.gpu_group_ffn(wl, Wp, x, keep, dev, wl.n_dev)
        ref = R.group_ffn(synth.host_bits(Wp), synth.host_bits(x), keep, dev, wl.n_dev)
        assert status == 0
        y_ref = R.merge(ref)
        rms = np.sqrt(np.mean(y_ref ** 2)) if len(keep) else 1.0
        err = np.abs(P.cpu().numpy() - ref).max() / rms
        assert err <= U.TOL_BF16, (keep, err)
        if not keep:
            assert (P == 0).all().item()


@pytest.mark.parametrize("d,G,S,n_tok", [(256, 160, 64, 100), (256, 80, 128, 300), (128, 150, 128, 129),
                                         (256, 42, 256, 300)])
def test_prefill_more_tiles_than_sms_splits_the_last_wave(d, G, S, n_tok):
    """With more hidden-layer tiles than SMs the groups of the last wave are computed as two half-width tiles
    each; every token of every kept group is checked, with all groups kept and with a ragged kept list."""
    wl = _wl(d, G, S)
    Wp = synth.packed_layer(wl, 0, DEV)
    x = synth.activation(wl, 1, DEV, n_tok=n_tok)
    dev = (np.arange(G, dtype=np.int32) % 4) - 1
    for keep in (list(range(G)), [g for g in range(G) if g % 17 != 3]):
        P, status = U.gpu_group_ffn(wl, Wp, x, keep, dev, wl.n_dev)
        ref = R.group_ffn(synth.host_bits(Wp), synth.host_bits(x), keep, dev, wl.n_dev)
        assert status == 0
        rms = np.sqrt(np.mean(R.merge(ref) ** 2))
        assert np.abs(P.cpu().numpy() - ref).max() <= U.TOL_BF16 * rms, len(keep)


@pytest.mark.parametrize("d,G,S,n_tok", [(256, 9, 128, 700), (512, 14, 64, 385)])
def test_prefill_single_launch_edge_cases(d, G, S, n_tok):
    """The one-launch form (more than 128 tokens, d % 256 == 0) on three token tiles with a ragged last one: no
    devices at all, every group on one device, a kept list with bad indices (flagged, skipped), a workspace reused
    across calls with different kept sets (its control words must come back zeroed)."""
    wl = _wl(d, G, S)
    Wp = synth.packed_layer(wl, 0, DEV)
    x = synth.activation(wl, 1, DEV, n_tok=n_tok)
    hb = synth.host_bits
    # no devices: one slot
    P, status = U.gpu_group_ffn(wl, Wp, x, [0, 2, G - 1], None, 0)
    ref = R.group_ffn(hb(Wp), hb(x), [0, 2, G - 1])
    rms = np.sqrt(np.mean(ref ** 2))
    assert status == 0 and np.abs(P.cpu().numpy() - ref).max() <= U.TOL_BF16 * rms
    # everything on the last device, slots in between stay zero
    dev = np.full(G, 2, dtype=np.int32)
    P, status = U.gpu_group_ffn(wl, Wp, x, list(range(G)), dev, 3)
    ref = R.group_ffn(hb(Wp), hb(x), list(range(G)), dev, 3)
    rms = np.sqrt(np.mean(R.merge(ref) ** 2))
    assert status == 0 and np.abs(P.cpu().numpy() - ref).max() <= U.TOL_BF16 * rms
    assert (P[:3] == 0).all().item()
    # bad indices are flagged and skipped
    dev = (np.arange(G, dtype=np.int32) % 3) - 1
    P, status = U.gpu_group_ffn(wl, Wp, x, [1, G + 5, 3, -2, 4], dev, 2)
    ref = R.group_ffn(hb(Wp), hb(x), [1, 3, 4], dev, 2)
    rms = np.sqrt(np.mean(R.merge(ref) ** 2))
    assert status & B.DEV_BAD_INDEX
    assert np.abs(P.cpu().numpy() - ref).max() <= U.TOL_BF16 * rms
    # one workspace, several calls with different kept sets
    sh = B.ffn_shape(d, G * S, S, B.BF16)
    ws = torch.empty(B.halo_group_ffn_workspace_bytes(sh, n_tok, 2), dtype=torch.uint8, device=DEV)
    dg = torch.as_tensor(dev, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    for keep in ([0, 1, 2, 3], [G - 1], list(range(G))[::-1], []):
        kl = torch.full((G,), -1, dtype=torch.int32, device=DEV)
        if keep:
            kl[: len(keep)] = torch.as_tensor(keep, dtype=torch.int32)
        nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
        P = torch.full((3, n_tok, d), float("nan"), dtype=torch.float32, device=DEV)
        B.halo_group_ffn(sh, Wp, x, n_tok, kl, nk, dg, 2, P, ws, st)
        torch.cuda.synchronize()
        ref = R.group_ffn(hb(Wp), hb(x), keep, dev, 2)
        scale = np.sqrt(np.mean(R.merge(ref) ** 2)) if keep else 1.0
        assert int(st.item()) == 0 and np.abs(P.cpu().numpy() - ref).max() <= U.TOL_BF16 * scale, keep


def test_prefill_matches_decode_path_token_by_token():
    wl = _wl(512, 4, 128)
    Wp = synth.packed_layer(wl, 0, DEV)
    x = synth.activation(wl, 2, DEV, n_tok=64)
    keep, dev = [0, 2, 3], np.array([-1, 1, 0, 1], dtype=np.int32)
    P_many, _ = U.gpu_group_ffn(wl, Wp, x, keep, dev, wl.n_dev)
    for t in (0, 31, 63):
        P_one, _ = U.gpu_group_ffn(wl, Wp, x[t:t + 1].contiguous(), keep, dev, wl.n_dev)
        ref = P_one[:, 0].cpu().numpy().astype(np.float64)
        rms = np.sqrt(np.mean(ref.sum(0) ** 2))
        assert np.abs(P_many[:, t].cpu().numpy() - ref).max() <= U.TOL_BF16 * rms


@pytest.mark.parametrize("name,n_tok", [("llama2-7b-prefill", 512), ("llama2-13b-decode", 512),
                                        ("tinyllama-1.1b-decode", 512), ("llama2-7b-prefill", 1900)])
def test_prefill_full_size_block_sampled_tokens(name, n_tok):
    """A prompt through one block of each stated shape (512 tokens; 1900 = eight token tiles, the last one ragged,
    more output tiles than SMs); the oracle checks a sample of the tokens."""
    wl = synth.workload(name, n_tok=n_tok)
    G = wl.n_groups
    Wp = synth.packed_layer(wl, 1, DEV)
    x = synth.activation(wl, 3, DEV, n_tok=wl.n_tok)
    scores = np.random.default_rng(5).normal(size=G).astype(np.float32)
    sel = R.select(scores, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, 0, 1)
    keep = sel["keep_list"][: sel["n_keep"]]
    P, status = U.gpu_group_ffn(wl, Wp, x, keep, sel["dev_of_group"], wl.n_dev)
    assert status == 0
    sample = [0, 127, 128, 300, 511] + ([1023, 1024, 1792, 1899] if n_tok > 512 else [])
    xs = synth.host_bits(x)[sample]
    ref = R.group_ffn(synth.host_bits(Wp), xs, keep, sel["dev_of_group"], wl.n_dev)
    y_ref = R.merge(ref)
    rms = np.sqrt(np.mean(y_ref ** 2))
    got = P[:, sample].cpu().numpy()
    assert np.abs(got - ref).max() <= U.TOL_BF16 * rms
    y = U.gpu_merge(P, sel["arrived"])[sample].cpu().numpy()
    assert U.rel_err(y, y_ref) <= U.TOL_BF16


@pytest.mark.parametrize("d,r,G,n_tok,pool", [(256, 64, 6, 32, True), (512, 200, 43, 130, False), (4096, 256, 86, 512, True),
                                              (5120, 512, 108, 64, True)])
@pytest.mark.parametrize("act", [B.ACT_RELU, B.ACT_NONE])
def test_predictor_many_tokens_tensor_core_hidden_layer(d, r, G, n_tok, pool, act):
    wl = synth.Workload("pp", 1, d, G * 8, 8, r, "bf16", (0.0,), (1,), 500, 1)
    W1, W2 = synth.predictor(wl, 1, DEV)
    feat = synth.activation(wl, 9, DEV, n_tok=n_tok)
    s, status = U.gpu_predict(B.BF16, W1, W2, feat, mean_pool=pool, act=act)
    assert status == 0
    sample = slice(None) if n_tok <= 130 else [0, 1, 127, 128, 255, 256, 511]
    hb = synth.host_bits
    if pool:
        ref = R.predict(hb(W1), hb(W2), hb(feat), act=act, mean_pool=True)
        assert U.rel_err(s.cpu().numpy(), ref.astype(np.float64)) <= U.TOL_BF16
    else:
        ref = R.predict(hb(W1), hb(W2), hb(feat)[sample], act=act)
        assert U.rel_err(s[sample].cpu().numpy(), ref.astype(np.float64)) <= U.TOL_BF16
