"""Pins for the oracle's int4 group quantisation (symmetric, blocks of 128 stored elements, bf16 scale)."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R


def _bf16_bits(a):
    return torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_values_on_the_grid_come_back_exactly_and_the_nibble_order_is_low_half_first():
    # one block whose values are k * 0.5 for k = -7 .. 7: amax = 3.5, s = 0.5 exactly, q = k
    ks = np.array(([-7, 7, 0, 1, -1, 3, -4, 6] * 16), dtype=np.int32)
    W = (ks * 0.5).astype(np.float32).reshape(1, 128)
    Q, Sc = R.quantize_i4(W)
    assert Q.shape == (1, 64) and Sc.shape == (1, 1)
    assert Sc[0, 0] == _bf16_bits([0.5])[0]
    assert (Q[0] & 15).tolist() == (ks[0::2] + 8).tolist()        # element 2i: low half of byte i
    assert (Q[0] >> 4).tolist() == (ks[1::2] + 8).tolist()        # element 2i+1: high half
    assert (R.dequantize_i4(Q, Sc) == W).all()


def test_zero_block_halfway_cases_and_scale_rounding():
    W = np.zeros((1, 256), dtype=np.float32)
    # second block: amax 7 -> s = 1; 2.5 and 3.5 are ties -> 2 and 4 (half to even); -0.5 -> -0, 0.5 -> 0
    W[0, 128:136] = [7.0, 2.5, 3.5, -2.5, -0.5, 0.5, -7.0, 6.49]
    Q, Sc = R.quantize_i4(W)
    assert Sc[0, 0] == 0 and (Q[0, :64] == 0x88).all()           # all-zero block: scale 0, every code 0 (nibble 8)
    assert Sc[0, 1] == _bf16_bits([1.0])[0]
    deq = R.dequantize_i4(Q, Sc)[0, 128:136]
    assert deq.tolist() == [7.0, 2.0, 4.0, -2.0, 0.0, 0.0, -7.0, 6.0]
    # a scale that is not on the grid: amax = 1 -> 1/7 = 0.142857.. -> bf16 0.142578125 = 1.140625 * 2^-3 -> up to
    # 5 significant bits (steps of 1/16 in the significand): 1.1875 * 2^-3 = 0.1484375
    W2 = np.zeros((1, 128), dtype=np.float32)
    W2[0, 0] = 1.0
    Q2, Sc2 = R.quantize_i4(W2)
    s = float(R.to_f64(Sc2)[0, 0])
    assert s == 0.1484375
    assert (Q2[0, 0] & 15) == 7 + 8                               # 1 / s = 6.74 -> 7, and never above 7
    # a scale that already has 5 bits stays; the carry of the rounding may reach the exponent:
    # amax = 7 * 1.96875 -> s = bf16(1.96875) = 1.96875 = 1.1111110b -> up: 2.0
    for amax, want in ((7 * 1.5, 1.5), (7 * 1.96875, 2.0), (7 * 0.0625, 0.0625)):
        W3 = np.zeros((1, 128), dtype=np.float32)
        W3[0, 5] = -amax
        _, Sc3 = R.quantize_i4(W3)
        assert float(R.to_f64(Sc3)[0, 0]) == want


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_error_bound_and_brute_force_python(dtype):
    g = torch.Generator().manual_seed(5)
    Wt = (torch.randn((6, 3, 5, 256), generator=g) * torch.rand((6, 3, 5, 1), generator=g) * 3).to(dtype)
    Wb = Wt.view(torch.int16).numpy().view(np.uint16) if dtype == torch.bfloat16 else Wt.numpy()
    Q, Sc = R.quantize_i4(Wb)
    assert Q.shape == (6, 3, 5, 128) and Sc.shape == (6, 3, 5, 2)
    w = R.to_f64(Wb).reshape(-1, 2, 128)
    s = R.to_f64(Sc).reshape(-1, 2, 1)
    deq = R.dequantize_i4(Q, Sc).astype(np.float64).reshape(-1, 2, 128)
    # every value within half a step (the scale is never below amax / 7 by more than the bf16 rounding, so only
    # that rounding can push the block maximum past 7.5 steps)
    assert (np.abs(w - deq) <= 0.5 * s * (1 + 2.0 ** -6)).all()
    # the scale: bf16(amax / 7) rounded UP to 5 significant bits, so within (-2^-8, +2^-4] of amax / 7 relatively,
    # with the three low bits of its bf16 significand clear
    amax = np.abs(w).max(axis=2, keepdims=True)
    assert (s >= amax / 7 * (1 - 2.0 ** -8)).all() and (s <= amax / 7 * (1 + 2.0 ** -8) * (1 + 2.0 ** -4)).all()
    assert ((Sc.reshape(-1) & 7) == 0).all()
    # hence every dequantised value is itself a bf16 number (what a bf16 tensor-core operand can carry exactly)
    deq32 = R.dequantize_i4(Q, Sc)
    assert (torch.from_numpy(deq32).to(torch.bfloat16).to(torch.float32).numpy() == deq32).all()
    # brute force in numpy float32 arithmetic, same decisions
    w32 = w.astype(np.float32)
    s32 = s.astype(np.float32)
    q = np.clip(np.rint(w32 / s32), -8, 7).astype(np.int32).reshape(-1, 128)
    nib = np.empty_like(q)
    Qf = Q.reshape(-1, 64)
    nib[:, 0::2] = Qf & 15
    nib[:, 1::2] = Qf >> 4
    assert (nib - 8 == q).all()


def test_ffn_on_int4_weights_is_the_ffn_on_the_dequantised_values():
    from paper_2601_11676_b200 import synth
    wl = synth.Workload("q", 1, 256, 64 * 3, 64, 16, "bf16", (0.0, 0.5), (1, 1), 500, 1)
    Wp = synth.host_bits(synth.packed_layer(wl, 0))
    x = synth.host_bits(synth.activation(wl, 1))
    Q, Sc = R.quantize_i4(Wp)
    dev = np.array([-1, 0, 1], dtype=np.int32)
    P4 = R.group_ffn_i4(Q, Sc, x, [0, 2], dev, 2)
    P16 = R.group_ffn(Wp, x, [0, 2], dev, 2)
    # same structure: the skipped group's slot is empty, and 4-bit weights stay close to the bf16 result
    assert (P4[1] == 0).all() and (P16[1] == 0).all()
    rel = np.abs(P4 - P16).max() / np.abs(P16).max()
    assert 1e-4 < rel < 0.25


def test_lm_head_on_int4_rows_is_a_plain_matrix_product_of_the_code_grid():
    """Rows built ON the int4 grid (integer codes times a power-of-two scale) with integer activations: the logits
    are integers that a numpy int64 product gives exactly; unlisted groups keep the fill value; a short last group."""
    rng = np.random.default_rng(5)
    vocab, d, S = 37, 256, 8
    codes = rng.integers(-7, 8, size=(vocab, d))
    codes[:, 0] = 7                                              # amax = 7 * scale in every block ...
    codes[:, 128] = -7                                           # ... so the scale comes back exactly
    scale = np.where(np.arange(vocab)[:, None] % 2 == 0, 0.5, 2.0)
    W = torch.tensor(codes * scale, dtype=torch.float32).numpy()
    Q, Sc = R.quantize_i4(W)
    assert (R.dequantize_i4(Q, Sc) == W).all()
    x_int = rng.integers(-3, 4, size=(2, d))
    x = torch.tensor(x_int, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    want = (x_int.astype(np.int64) @ (codes * 2).astype(np.int64).T) * np.where(np.arange(vocab) % 2 == 0, 0.25, 1.0)
    full = R.group_lm_head_i4(Q, Sc, x, S)
    assert full.shape == (2, vocab) and (full == want).all()
    part = R.group_lm_head_i4(Q, Sc, x, S, group_list=[4, 0], fill=-1.0)      # group 4 = rows 32..36 (short)
    listed = np.zeros(vocab, dtype=bool)
    listed[0:8] = True
    listed[32:37] = True
    assert (part[:, listed] == want[:, listed]).all() and (part[:, ~listed] == -1.0).all()


def test_mha_on_int4_weights_is_the_mha_on_the_dequantised_values():
    """Weights built ON the int4 grid: the int4 wrappers must give exactly what the float32 functions give on the same
    weights (catches a mixed-up code / scale array, a wrong reshape of the packed rows, a cache that is not widened)."""
    rng = np.random.default_rng(9)
    d, H, dh, L = 128, 2, 16, 6

    def on_grid(rows):
        c = rng.integers(-7, 8, size=(rows, d)).astype(np.float32)
        c[:, 0] = 7
        return c * np.where(np.arange(rows)[:, None] % 2 == 0, 2.0 ** -4, 2.0 ** -5).astype(np.float32)
    Wq, Wk, Wv = on_grid(H * dh), on_grid(H * dh), on_grid(H * dh)
    Wo_rows = on_grid(H * dh)                                  # row h*dh + j = column h*dh + j of Wo
    Wp = np.stack([np.stack([Wq[h * dh:(h + 1) * dh], Wo_rows[h * dh:(h + 1) * dh]]) for h in range(H)])   # [H][2][dh][d]
    assert (R.pack_mha(Wq, np.ascontiguousarray(Wo_rows.T), H) == Wp).all()
    x = (rng.integers(-4, 5, size=d) / 4.0).astype(np.float32)
    xb = _bf16_bits(x)
    Qp, Sp = R.quantize_i4(Wp.reshape(H * 2 * dh, d))
    Qk, Sk = R.quantize_i4(Wk)
    Qv, Sv = R.quantize_i4(Wv)
    K32 = rng.standard_normal((H, L, dh)).astype(np.float32)
    V32 = rng.standard_normal((H, L, dh)).astype(np.float32)
    Ka, Va, Kb, Vb = K32.copy(), V32.copy(), K32.copy(), V32.copy()
    R.mha_kv_append_i4(Qk, Sk, Qv, Sv, xb, 3, Ka, Va)
    R.mha_kv_append(Wk, Wv, x, 3, Kb, Vb)
    assert (Ka == Kb).all() and (Va == Vb).all() and not (Ka[:, 3] == K32[:, 3]).all()
    dev = np.array([0, -1], dtype=np.int32)
    got = R.group_mha_i4(Qp, Sp, H, xb, Ka, Va, 3, [1, 0], dev, 1)
    want = R.group_mha(Wp, x, Kb, Vb, 3, [1, 0], dev, 1)
    assert (got == want).all() and np.abs(want).max() > 0
    # bf16 caches are widened, not reinterpreted
    Kbits, Vbits = _bf16_bits(Ka), _bf16_bits(Va)
    got16 = R.group_mha_i4(Qp, Sp, H, xb, Kbits, Vbits, 3, [0], dev, 1)
    want16 = R.group_mha(Wp, x, R.to_f64(Kbits).astype(np.float32), R.to_f64(Vbits).astype(np.float32), 3, [0], dev, 1)
    assert (got16 == want16).all()
