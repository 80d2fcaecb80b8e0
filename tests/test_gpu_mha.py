"""GPU parity of the MHA neuron-group entry points against the oracle."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = U.DEV


def _wl(dtype, d, seed=0):
    return synth.Workload("a", 1, d, 64, 16, 32, dtype, (0.0, 0.2, 0.6), (2, 1, 1), 500, 1, seed=seed)


def _caches(wl, H, L, dh, fill):
    g = torch.Generator(device=DEV).manual_seed(1234)
    K = torch.zeros((H, L, dh), dtype=wl.torch_dtype, device=DEV)
    V = torch.zeros((H, L, dh), dtype=wl.torch_dtype, device=DEV)
    K[:, :fill] = torch.randn((H, fill, dh), generator=g, device=DEV).to(wl.torch_dtype)
    V[:, :fill] = torch.randn((H, fill, dh), generator=g, device=DEV).to(wl.torch_dtype)
    return K, V


@pytest.mark.parametrize("dtype,d,H,dh,L,positions", [("f32", 64, 4, 16, 40, (0, 7, 39)), ("bf16", 512, 8, 64, 300, (0, 127, 128, 299)),
                                                      ("bf16", 4096, 32, 128, 1024, (5, 700, 1023)),
                                                      ("bf16", 256, 8, 32, 5000, (255, 2047, 2048, 4999)),
                                                      ("f32", 512, 2, 256, 70, (0, 69))])
def test_group_mha_and_kv_append_match_oracle(dtype, d, H, dh, L, positions):
    wl = _wl(dtype, d)
    code = U.dtype_code(wl)
    sh = B.mha_shape(d, H, dh, L, code)
    Wq, Wk, Wv, Wo = synth.mha_matrices(wl, 0, H, DEV)
    Wp = torch.empty((H, 2, dh, d), dtype=wl.torch_dtype, device=DEV)
    B.halo_pack_mha_weights(sh, Wq, Wo, Wp)
    torch.cuda.synchronize()
    hb = synth.host_bits
    Wp_ref = R.pack_mha(hb(Wq), hb(Wo), H)
    assert (hb(Wp) == Wp_ref).all()                               # layout: bit exact
    K, V = _caches(wl, H, L, dh, L)
    ws = torch.empty(B.halo_group_mha_workspace_bytes(sh), dtype=torch.uint8, device=DEV)
    tol = U.tol_for(wl)
    dev = np.array([(-1, 0, 1, 2)[h % 4] for h in range(H)], dtype=np.int32)
    dg = torch.as_tensor(dev, device=DEV)
    for pos in positions:
        x = synth.activation(wl, 50 + pos, DEV)
        # keys / values of this token: within one rounding step of the oracle's
        K_before, V_before = K.clone(), V.clone()
        B.halo_mha_kv_append(sh, Wk, Wv, x, pos, K, V)
        torch.cuda.synchronize()
        Kh, Vh = hb(K), hb(V)
        Kr, Vr = Kh.copy(), Vh.copy()
        R.mha_kv_append(hb(Wk), hb(Wv), hb(x)[0], pos, Kr, Vr)
        kk = R.to_f64(Kr[:, pos])
        assert np.abs(R.to_f64(Kh[:, pos]) - kk).max() <= (1e-5 if dtype == "f32" else 2 ** -7) * np.abs(kk).max()
        assert np.abs(R.to_f64(Vh[:, pos]) - R.to_f64(Vr[:, pos])).max() <= (1e-5 if dtype == "f32" else 2 ** -7) * np.abs(kk).max()
        # and the rest of the cache is untouched
        other = [p for p in (0, L // 2, L - 1) if p != pos]
        assert (Kh[:, other] == hb(K_before)[:, other]).all() and (Vh[:, other] == hb(V_before)[:, other]).all()
        # attention of the kept heads, from the GPU's own cache bytes
        for keep in (list(range(H)), [h for h in range(H) if h % 3 != 1], [H - 1], []):
            kl = torch.full((H,), -1, dtype=torch.int32, device=DEV)
            if keep:
                kl[: len(keep)] = torch.as_tensor(keep, dtype=torch.int32, device=DEV)
            nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
            P = torch.full((4, d), float("nan"), dtype=torch.float32, device=DEV)
            status = torch.zeros(1, dtype=torch.int32, device=DEV)
            B.halo_group_mha(sh, Wp, x, K, V, pos, kl, nk, dg, 3, P, ws, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            ref = R.group_mha(Wp_ref, hb(x)[0], Kh, Vh, pos, keep, dev, 3)
            if not keep:
                assert (P == 0).all().item()
                continue
            rms = np.sqrt(np.mean(ref.sum(0) ** 2))
            assert np.abs(P.cpu().numpy() - ref).max() <= tol * rms, (pos, len(keep))
            y = U.gpu_merge(P[:, None, :].contiguous()).cpu().numpy()[0]
            assert U.rel_err(y, ref.sum(0)) <= tol


def test_mha_heads_under_the_selection_machinery():
    """Heads as groups: scores -> selection (Algorithm-3 chunks, arrival draw) -> kept heads -> merge."""
    wl = synth.Workload("a", 1, 512, 64, 16, 32, "bf16", (0.0, 0.4, 0.9), (1, 1, 2), 375, 1)
    H, dh, L, d = 8, 64, 64, 512
    sh = B.mha_shape(d, H, dh, L, B.BF16)
    Wq, Wk, Wv, Wo = synth.mha_matrices(wl, 0, H, DEV)
    Wp = torch.empty((H, 2, dh, d), dtype=torch.bfloat16, device=DEV)
    B.halo_pack_mha_weights(sh, Wq, Wo, Wp)
    K, V = _caches(wl, H, L, dh, L)
    plan = B.Plan(H, wl.loss_rate, wl.share_weight, B.SEL_TOPK, 3, 0.0, 77)
    scores = torch.randn(H, generator=torch.Generator().manual_seed(3)).to(DEV)
    ws = torch.empty(B.halo_group_mha_workspace_bytes(sh), dtype=torch.uint8, device=DEV)
    hb = synth.host_bits
    seen = set()
    for step in range(12):
        gpu, bufs = U.gpu_select(plan, scores, step, 2)
        ref_sel = R.select(scores.cpu().numpy(), wl.loss_rate, wl.share_weight, R.SEL_TOPK, 3, 0.0, 77, step, 2)
        U.assert_select_equal(gpu, ref_sel)
        x = synth.activation(wl, step, DEV)
        P = torch.empty((4, d), dtype=torch.float32, device=DEV)
        B.halo_group_mha(sh, Wp, x, K, V, 40, bufs["keep_list"], bufs["n_keep"], bufs["dev_of_group"], 3, P, ws)
        y = U.gpu_merge(P[:, None, :].contiguous(), gpu["arrived"]).cpu().numpy()[0]
        ref = R.group_mha(hb(Wp), hb(x)[0], hb(K), hb(V), 40, ref_sel["keep_list"][: ref_sel["n_keep"]],
                          ref_sel["dev_of_group"], 3)
        assert U.rel_err(y, R.merge(ref[:, None, :], ref_sel["arrived"])[0]) <= U.TOL_BF16
        seen.add(gpu["n_keep"])
    assert len(seen) > 1


def test_mha_argument_checks():
    sh = B.mha_shape(512, 8, 60, 64, B.BF16)       # head_dim not a multiple of 16
    assert B.halo_group_mha_workspace_bytes(sh) == 0
    t = torch.zeros(16, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(B.HaloError):
        B.halo_mha_kv_append(sh, t, t, t, 0, t, t)
    ok = B.mha_shape(512, 8, 64, 64, B.BF16)
    with pytest.raises(B.HaloError):
        B.halo_mha_kv_append(ok, t, t, t, 64, t, t)   # position beyond the cache


@pytest.mark.parametrize("dtype,d,H,dh,L,positions", [("f32", 64, 4, 16, 40, (0, 7, 39)), ("bf16", 512, 8, 64, 300, (0, 128, 299)),
                                                      ("bf16", 4096, 32, 128, 1100, (3, 1023, 1099)),
                                                      ("bf16", 2048, 32, 64, 600, (511,))])
def test_mha_block_one_launch_matches_oracle_and_the_two_calls(dtype, d, H, dh, L, positions):
    """halo_mha_block: keys / values of every head appended and the kept heads attended in one launch.  The cache rows
    it writes are the bits halo_mha_kv_append writes (and within a rounding step of the oracle's); the partials are
    the oracle's from those cache bytes, also when the token's own position is the only one (pos 0) and for heads
    that are not kept (their keys and values must still land)."""
    wl = _wl(dtype, d)
    code = U.dtype_code(wl)
    sh = B.mha_shape(d, H, dh, L, code)
    Wq, Wk, Wv, Wo = synth.mha_matrices(wl, 1, H, DEV)
    Wp = torch.empty((H, 2, dh, d), dtype=wl.torch_dtype, device=DEV)
    B.halo_pack_mha_weights(sh, Wq, Wo, Wp)
    hb = synth.host_bits
    Wp_ref = hb(Wp)
    K, V = _caches(wl, H, L, dh, L)
    tol = U.tol_for(wl)
    dev = np.array([(-1, 0, 1, 2)[h % 4] for h in range(H)], dtype=np.int32)
    dg = torch.as_tensor(dev, device=DEV)
    ws = torch.empty(B.halo_group_mha_workspace_bytes(sh), dtype=torch.uint8, device=DEV)
    for pos in positions:
        for keep in (list(range(H)), [h for h in range(H) if h % 3 != 1], [H - 1], []):
            x = synth.activation(wl, 90 + pos + len(keep), DEV)
            K2, V2 = K.clone(), V.clone()
            kl = torch.full((H,), -1, dtype=torch.int32, device=DEV)
            if keep:
                kl[: len(keep)] = torch.as_tensor(keep, dtype=torch.int32, device=DEV)
            nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
            P = torch.full((4, d), float("nan"), dtype=torch.float32, device=DEV)
            status = torch.zeros(1, dtype=torch.int32, device=DEV)
            B.halo_mha_block(sh, Wp, Wk, Wv, x, K, V, pos, kl, nk, dg, 3, P, status)
            # the two calls, on copies of the caches
            B.halo_mha_kv_append(sh, Wk, Wv, x, pos, K2, V2)
            P2 = torch.empty_like(P)
            B.halo_group_mha(sh, Wp, x, K2, V2, pos, kl, nk, dg, 3, P2, ws, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert torch.equal(K.view(torch.uint8), K2.view(torch.uint8)) and torch.equal(V.view(torch.uint8), V2.view(torch.uint8))
            Kh, Vh = hb(K), hb(V)
            Kr, Vr = Kh.copy(), Vh.copy()
            R.mha_kv_append(hb(Wk), hb(Wv), hb(x)[0], pos, Kr, Vr)
            kk = R.to_f64(Kr[:, pos])
            rt = 1e-5 if dtype == "f32" else 2 ** -7
            assert np.abs(R.to_f64(Kh[:, pos]) - kk).max() <= rt * np.abs(kk).max()
            assert np.abs(R.to_f64(Vh[:, pos]) - R.to_f64(Vr[:, pos])).max() <= rt * np.abs(kk).max()
            if not keep:
                assert (P == 0).all().item()
                continue
            ref = R.group_mha(Wp_ref, hb(x)[0], Kh, Vh, pos, keep, dev, 3)
            rms = np.sqrt(np.mean(ref.sum(0) ** 2))
            assert np.abs(P.cpu().numpy() - ref).max() <= tol * rms, (pos, len(keep))
            assert np.abs(P2.cpu().numpy() - ref).max() <= tol * rms


def _quant_rows(W):
    rows, d = W.shape
    Q = torch.empty((rows, d // 2), dtype=torch.uint8, device=DEV)
    S = torch.empty((rows, d // 128), dtype=torch.bfloat16, device=DEV)
    B.halo_quantize_rows_i4(d, rows, B.BF16, W, Q, S)
    torch.cuda.synchronize()
    return Q, S


@pytest.mark.parametrize("d,H,dh,L,positions", [(512, 8, 64, 300, (0, 128, 299)), (4096, 32, 128, 1100, (3, 1023, 1099)),
                                                (2048, 32, 64, 600, (511,)), (8192, 4, 128, 64, (40,)), (128, 3, 16, 20, (0, 19))])
def test_mha_block_on_int4_weights_matches_the_oracle(d, H, dh, L, positions):
    """halo_mha_block_i4: the appended cache rows against the oracle's keys and values from the dequantised Wk / Wv
    (one bf16 rounding apart), the partials against the oracle's attention on the dequantised packed weights from the
    GPU's cache bytes; heads that are not kept must still append, an empty kept set leaves zeros."""
    wl = _wl("bf16", d)
    sh = B.mha_shape(d, H, dh, L, B.BF16)
    Wq, Wk, Wv, Wo = synth.mha_matrices(wl, 2, H, DEV)
    Wp = torch.empty((H, 2, dh, d), dtype=torch.bfloat16, device=DEV)
    B.halo_pack_mha_weights(sh, Wq, Wo, Wp)
    Qp, Sp = _quant_rows(Wp.view(H * 2 * dh, d))
    Qk, Sk = _quant_rows(Wk)
    Qv, Sv = _quant_rows(Wv)
    hb = synth.host_bits
    Qp_h, Sp_h, Qk_h, Sk_h, Qv_h, Sv_h = Qp.cpu().numpy(), hb(Sp), Qk.cpu().numpy(), hb(Sk), Qv.cpu().numpy(), hb(Sv)
    ref_q = R.quantize_i4(hb(Wk))
    assert (Qk_h == ref_q[0]).all() and (Sk_h == ref_q[1]).all()
    K, V = _caches(wl, H, L, dh, L)
    dev = np.array([(-1, 0, 1, 2)[h % 4] for h in range(H)], dtype=np.int32)
    dg = torch.as_tensor(dev, device=DEV)
    for pos in positions:
        for keep in (list(range(H)), [h for h in range(H) if h % 3 != 1], [H - 1], []):
            x = synth.activation(wl, 190 + pos + len(keep), DEV)
            kl = torch.full((H,), -1, dtype=torch.int32, device=DEV)
            if keep:
                kl[: len(keep)] = torch.as_tensor(keep, dtype=torch.int32, device=DEV)
            nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
            P = torch.full((4, d), float("nan"), dtype=torch.float32, device=DEV)
            status = torch.zeros(1, dtype=torch.int32, device=DEV)
            B.halo_mha_block_i4(sh, Qp, Sp, Qk, Sk, Qv, Sv, x, K, V, pos, kl, nk, dg, 3, P, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            Kh, Vh = hb(K), hb(V)
            K32, V32 = R.to_f64(Kh).astype(np.float32), R.to_f64(Vh).astype(np.float32)
            R.mha_kv_append_i4(Qk_h, Sk_h, Qv_h, Sv_h, hb(x)[0], pos, K32, V32)      # overwrites row `pos`, unrounded
            kk = K32[:, pos].astype(np.float64)
            assert np.abs(R.to_f64(Kh[:, pos]) - kk).max() <= 2 ** -7 * np.abs(kk).max()
            assert np.abs(R.to_f64(Vh[:, pos]) - V32[:, pos]).max() <= 2 ** -7 * np.abs(V32[:, pos]).max()
            if not keep:
                assert (P == 0).all().item()
                continue
            ref = R.group_mha_i4(Qp_h, Sp_h, H, hb(x)[0], Kh, Vh, pos, keep, dev, 3)
            rms = np.sqrt(np.mean(ref.sum(0) ** 2))
            assert np.abs(P.cpu().numpy() - ref).max() <= U.TOL_BF16 * rms, (pos, len(keep))
