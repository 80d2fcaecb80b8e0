"""GPU parity of halo_group_lm_head (groups of vocabulary rows, concatenated outputs) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = U.DEV


def _run(W, x, S, keep, dtype_code, fill=-123.0):
    vocab, d = W.shape
    n_tok = x.shape[0]
    sh = B.lm_shape(d, vocab, S, dtype_code)
    logits = torch.full((n_tok, vocab), fill, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    if keep is None:
        B.halo_group_lm_head(sh, W, x, n_tok, None, None, logits, status)
    else:
        n_groups = (vocab + S - 1) // S
        kl = torch.zeros(max(n_groups, len(keep), 1), dtype=torch.int32, device=DEV)
        kl[: len(keep)] = torch.as_tensor(keep, dtype=torch.int32)
        nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
        B.halo_group_lm_head(sh, W, x, n_tok, kl, nk, logits, status)
    torch.cuda.synchronize()
    return logits.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("dtype,code,tol", [(torch.bfloat16, B.BF16, U.TOL_BF16), (torch.float32, B.F32, U.TOL_F32)])
@pytest.mark.parametrize("vocab,d,S,n_tok", [(1000, 512, 256, 1), (777, 1024, 100, 3), (50, 64, 256, 2), (4099, 2048, 256, 1),
                                             (1003, 4096, 96, 1), (5, 4096, 256, 1), (300, 2048, 20, 1)])
def test_lm_head_groups_match_the_oracle(dtype, code, tol, vocab, d, S, n_tok):
    g = torch.Generator().manual_seed(vocab + d)
    W = (torch.randn((vocab, d), generator=g) / np.sqrt(d)).to(dtype).to(DEV)
    x = torch.randn((n_tok, d), generator=g).to(dtype).to(DEV)
    n_groups = (vocab + S - 1) // S
    for keep in (None, [gi for gi in range(n_groups) if gi % 3 != 1][::-1], [n_groups - 1], []):
        got, status = _run(W, x, S, keep, code)
        assert status == 0
        ref = R.group_lm_head(synth.host_bits(W), synth.host_bits(x), S, keep, fill=-123.0)
        rms = np.sqrt(np.mean(R.group_lm_head(synth.host_bits(W), synth.host_bits(x), S) ** 2))
        assert np.abs(got - ref).max() <= tol * rms, keep          # untouched entries compare -123 with -123


def test_lm_head_flags_a_bad_group_index_and_computes_the_rest():
    W = torch.randn((300, 256), dtype=torch.float32, device=DEV)
    x = torch.randn((1, 256), dtype=torch.float32, device=DEV)
    got, status = _run(W, x, 64, [0, 9, 2], B.F32)
    assert status & 1 or status != 0
    ref = R.group_lm_head(W.cpu().numpy(), x.cpu().numpy(), 64, [0, 2], fill=-123.0)
    assert np.abs(got - ref).max() <= U.TOL_F32 * np.abs(ref[ref != -123.0]).max()


def test_lm_head_streaming_form_flags_a_bad_group_index_and_computes_the_rest():
    """One token, bf16, d 4096: the shared-memory ring form; a bad index in the list costs a status bit, not the call."""
    g = torch.Generator().manual_seed(3)
    W = (torch.randn((700, 4096), generator=g) / 64.0).to(torch.bfloat16).to(DEV)
    x = torch.randn((1, 4096), generator=g).to(torch.bfloat16).to(DEV)
    got, status = _run(W, x, 64, [0, 99, 10, -1, 2], B.BF16)
    assert status != 0
    ref = R.group_lm_head(synth.host_bits(W), synth.host_bits(x), 64, [0, 10, 2], fill=-123.0)
    rms = np.sqrt(np.mean(R.group_lm_head(synth.host_bits(W), synth.host_bits(x), 64) ** 2))
    assert np.abs(got - ref).max() <= U.TOL_BF16 * rms


def test_lm_head_full_vocabulary_at_7b_width():
    """32000 x 4096 bf16 (262 MB streamed once); a sample of rows against the oracle, all rows against a library product."""
    vocab, d, S = 32000, 4096, 256
    g = torch.Generator().manual_seed(7)
    W = (torch.randn((vocab, d), generator=g) / np.sqrt(d)).to(torch.bfloat16).to(DEV)
    x = torch.randn((1, d), generator=g).to(torch.bfloat16).to(DEV)
    got, status = _run(W, x, S, None, B.BF16)
    assert status == 0
    groups = [0, 57, 124]
    ref = R.group_lm_head(synth.host_bits(W), synth.host_bits(x), S, groups)
    rows = np.concatenate([np.arange(gi * S, (gi + 1) * S) for gi in groups])
    rms = np.sqrt(np.mean(ref[:, rows] ** 2))
    assert np.abs(got[:, rows] - ref[:, rows]).max() <= U.TOL_BF16 * rms
    lib = (x.double() @ W.double().T).cpu().numpy()
    assert np.abs(got - lib).max() <= U.TOL_BF16 * rms


def _quantize_rows(W, src_code):
    vocab, d = W.shape
    Q = torch.empty((vocab, d // 2), dtype=torch.uint8, device=DEV)
    Sc = torch.empty((vocab, d // 128), dtype=torch.bfloat16, device=DEV)
    B.halo_quantize_rows_i4(d, vocab, src_code, W, Q, Sc)
    torch.cuda.synchronize()
    return Q, Sc


def _run_i4(Q, Sc, x, vocab, S, keep, fill=-123.0):
    n_tok, d = x.shape
    sh = B.lm_shape(d, vocab, S, B.BF16)
    logits = torch.full((n_tok, vocab), fill, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    if keep is None:
        B.halo_group_lm_head_i4(sh, Q, Sc, x, n_tok, None, None, logits, status)
    else:
        n_groups = (vocab + S - 1) // S
        kl = torch.zeros(max(n_groups, len(keep), 1), dtype=torch.int32, device=DEV)
        kl[: len(keep)] = torch.as_tensor(keep, dtype=torch.int32)
        nk = torch.tensor([len(keep)], dtype=torch.int32, device=DEV)
        B.halo_group_lm_head_i4(sh, Q, Sc, x, n_tok, kl, nk, logits, status)
    torch.cuda.synchronize()
    return logits.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("src,code", [(torch.bfloat16, B.BF16), (torch.float32, B.F32)])
@pytest.mark.parametrize("vocab,d,S,n_tok", [(1000, 512, 256, 1), (777, 1024, 100, 3), (50, 128, 256, 2), (4099, 2048, 256, 1),
                                             (1003, 4096, 96, 1), (5, 4096, 256, 1), (300, 8192, 20, 1)])
def test_lm_head_int4_rows_match_the_oracle(src, code, vocab, d, S, n_tok):
    """Codes and scales of the row quantiser bit for bit; logits of the listed groups against the oracle's LM head on
    the dequantised rows, unlisted entries untouched."""
    g = torch.Generator().manual_seed(vocab + d + 1)
    W = (torch.randn((vocab, d), generator=g) / np.sqrt(d)).to(src).to(DEV)
    x = torch.randn((n_tok, d), generator=g).to(torch.bfloat16).to(DEV)
    Q, Sc = _quantize_rows(W, code)
    hb = synth.host_bits
    Q_ref, Sc_ref = R.quantize_i4(hb(W))
    assert (Q.cpu().numpy() == Q_ref).all() and (hb(Sc) == Sc_ref).all()
    n_groups = (vocab + S - 1) // S
    rms = np.sqrt(np.mean(R.group_lm_head_i4(Q_ref, Sc_ref, hb(x), S) ** 2))
    for keep in (None, [gi for gi in range(n_groups) if gi % 3 != 1][::-1], [n_groups - 1], []):
        got, status = _run_i4(Q, Sc, x, vocab, S, keep)
        assert status == 0
        ref = R.group_lm_head_i4(Q_ref, Sc_ref, hb(x), S, keep, fill=-123.0)
        assert np.abs(got - ref).max() <= U.TOL_BF16 * rms, keep


def test_lm_head_int4_flags_a_bad_group_index_and_computes_the_rest():
    g = torch.Generator().manual_seed(4)
    W = (torch.randn((700, 1024), generator=g) / 32.0).to(torch.bfloat16).to(DEV)
    x = torch.randn((1, 1024), generator=g).to(torch.bfloat16).to(DEV)
    Q, Sc = _quantize_rows(W, B.BF16)
    got, status = _run_i4(Q, Sc, x, 700, 64, [0, 99, 10, -1, 2])
    assert status & B.DEV_BAD_INDEX
    hb = synth.host_bits
    ref = R.group_lm_head_i4(Q.cpu().numpy(), hb(Sc), hb(x), 64, [0, 10, 2], fill=-123.0)
    rms = np.sqrt(np.mean(R.group_lm_head_i4(Q.cpu().numpy(), hb(Sc), hb(x), 64) ** 2))
    assert np.abs(got - ref).max() <= U.TOL_BF16 * rms


def test_lm_head_int4_full_vocabulary_at_7b_width():
    """The case the benchmark times: 32000 x 4096 in groups of 256, one token, every logit."""
    g = torch.Generator().manual_seed(11)
    W = (torch.randn((32000, 4096), generator=g) / 64.0).to(torch.bfloat16).to(DEV)
    x = torch.randn((1, 4096), generator=g).to(torch.bfloat16).to(DEV)
    Q, Sc = _quantize_rows(W, B.BF16)
    del W
    got, status = _run_i4(Q, Sc, x, 32000, 256, None)
    assert status == 0
    hb = synth.host_bits
    ref = R.group_lm_head_i4(Q.cpu().numpy(), hb(Sc), hb(x), 256)
    assert np.abs(got - ref).max() <= U.TOL_BF16 * np.sqrt(np.mean(ref ** 2))


def test_lm_head_int4_streaming_form_flags_a_bad_group_index_and_ragged_groups():
    """One token, d 4096: the shared-memory ring form of the int4 head; groups of 40 rows (a full batch of 32 and a
    ragged one of 8), a short last group, a bad index in the list."""
    g = torch.Generator().manual_seed(6)
    vocab, d, S = 1013, 4096, 40
    W = (torch.randn((vocab, d), generator=g) / 64.0).to(torch.bfloat16).to(DEV)
    x = torch.randn((1, d), generator=g).to(torch.bfloat16).to(DEV)
    Q, Sc = _quantize_rows(W, B.BF16)
    n_groups = (vocab + S - 1) // S
    keep = [0, 99, n_groups - 1, -1, 7, 3]
    got, status = _run_i4(Q, Sc, x, vocab, S, keep)
    assert status & B.DEV_BAD_INDEX
    hb = synth.host_bits
    ref = R.group_lm_head_i4(Q.cpu().numpy(), hb(Sc), hb(x), S, [0, n_groups - 1, 7, 3], fill=-123.0)
    rms = np.sqrt(np.mean(R.group_lm_head_i4(Q.cpu().numpy(), hb(Sc), hb(x), S) ** 2))
    assert np.abs(got - ref).max() <= U.TOL_BF16 * rms
