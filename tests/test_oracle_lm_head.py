"""Pins for the oracle's LM-head neuron groups (Sec. II-A: an up-projection only, a collection of groups of
vocabulary rows; Sec. III-B.3: delivered reliably, so nothing is dropped and the outputs are concatenated)."""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R


def _bits(t):
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()


def test_hand_computed_integers():
    # 5 vocabulary rows of width 3, groups of 2 rows (the last group has one row), two tokens
    W = np.array([[1, 2, 3], [0, -1, 4], [2, 2, 2], [-3, 0, 1], [5, -5, 0]], dtype=np.float32)
    x = np.array([[1, 0, -1], [2, 3, 4]], dtype=np.float32)
    want = np.array([[-2, -4, 0, -4, 5], [20, 13, 18, -2, -5]], dtype=np.float64)
    assert (R.group_lm_head(W, x, 2) == want).all()
    # groups 0 and 2 only: rows 0, 1 and 4; rows 2, 3 keep the fill value
    got = R.group_lm_head(W, x, 2, [2, 0], fill=-7.0)
    assert (got[:, [0, 1, 4]] == want[:, [0, 1, 4]]).all() and (got[:, [2, 3]] == -7.0).all()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("vocab,S", [(96, 32), (100, 32), (7, 16)])
def test_equals_the_dense_product_and_concatenates_disjoint_groups(dtype, vocab, S):
    g = torch.Generator().manual_seed(vocab * 131 + S)
    W = torch.randn((vocab, 48), generator=g).to(dtype)
    x = torch.randn((3, 48), generator=g).to(dtype)
    Wb, xb = _bits(W), _bits(x)
    dense = R.to_f64(xb) @ R.to_f64(Wb).T            # the library routine on the widened operands
    full = R.group_lm_head(Wb, xb, S)
    assert np.abs(full - dense).max() <= 1e-12 * np.abs(dense).max()
    n_groups = (vocab + S - 1) // S
    even, odd = list(range(0, n_groups, 2)), list(range(1, n_groups, 2))
    a = R.group_lm_head(Wb, xb, S, even, fill=0.0)
    b = R.group_lm_head(Wb, xb, S, odd, fill=0.0)
    assert (a + b == full).all()                     # every row belongs to exactly one group
    rows_even = [v for v in range(vocab) if (v // S) % 2 == 0]
    assert (b[:, rows_even] == 0.0).all() and (a[:, rows_even] == full[:, rows_even]).all()


def test_rejects_a_group_index_outside_the_vocabulary():
    W = np.zeros((10, 4), dtype=np.float32)
    x = np.zeros((1, 4), dtype=np.float32)
    with pytest.raises(Exception):
        R.group_lm_head(W, x, 4, [3])
    assert np.isfinite(R.group_lm_head(W, x, 4, [2])[:, 8:]).all()
