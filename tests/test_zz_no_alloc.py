"""The workspace-free predictor entry point (halo_predict_groups_static) against halo_predict_groups and the oracle.

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything else.
It is written for callers that cannot allocate device memory; here it must give the same scores as the entry
point that takes a workspace, on two calls in a row (the second call finds the first call's leftovers in the
library's fixed scratch array and must not care), agree with the CPU oracle, leave the amount of free device
memory untouched, and refuse sizes beyond the fixed array.
"""
import numpy as np
import pytest
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = U.DEV


def _static_scores(code, W1, W2, feat, mean_pool):
    r, d_in = W1.shape
    G = W2.shape[0]
    n_tok = feat.shape[0]
    sh = B.pred_shape(d_in, r, G, code)
    scores = torch.full((G,) if (mean_pool or n_tok == 1) else (n_tok, G), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.halo_predict_groups_static(sh, W1, W2, feat, n_tok, mean_pool, scores, status)
    torch.cuda.synchronize()
    return scores, int(status.item())


@pytest.mark.parametrize("name,n_tok,pool", [("tiny", 1, False), ("llama2-7b-decode", 1, False),
                                             ("llama2-13b-decode", 4, True), ("tinyllama-1.1b-decode", 3, False),
                                             ("llama2-7b-decode", 48, True), ("llama2-13b-decode", 200, False)])
def test_static_predictor_matches_workspace_predictor_twice_in_a_row(name, n_tok, pool):
    """From 16 tokens on the hidden layer runs on the tensor cores, with the fixed array as its output: the last
    two cases cover that branch with non-zero features.  Every call is also compared with the oracle."""
    wl = synth.workload(name)
    code = U.dtype_code(wl)
    tol = U.tol_for(wl)
    hb = synth.host_bits
    for call, layer in enumerate((1, 2)):           # two calls in a row, different weights and inputs
        W1, W2 = synth.predictor(wl, layer, DEV)
        feat = synth.activation(wl, 40 + layer, DEV, n_tok=n_tok)
        ref, st_ref = U.gpu_predict(code, W1, W2, feat, mean_pool=pool)
        got, st = _static_scores(code, W1, W2, feat, pool)
        assert st == 0 and st_ref == 0
        assert got.shape == ref.shape
        assert torch.isfinite(got).all().item()
        assert U.rel_err(got.cpu().numpy(), ref.cpu().numpy().astype(np.float64)) <= tol, (name, call)
        oracle = R.predict(hb(W1), hb(W2), hb(feat), mean_pool=pool)
        assert oracle.shape == tuple(got.shape)
        assert U.rel_err(got.cpu().numpy(), oracle.astype(np.float64)) <= tol, (name, call, "oracle")


def test_static_predictor_leaves_device_memory_alone():
    """What the entry point is for: after a first call (which looks up the address of the library's array), further
    calls must not change the free device memory as the driver reports it, nor what torch's allocator holds."""
    wl = synth.workload("llama2-7b-decode")
    W1, W2 = synth.predictor(wl, 1, DEV)
    sh = B.pred_shape(wl.d_model, wl.pred_rank, wl.n_groups, B.BF16)
    feats = [synth.activation(wl, 70 + i, DEV, n_tok=n) for i, n in enumerate((1, 5, 32))]
    outs = [torch.empty((wl.n_groups,), dtype=torch.float32, device=DEV) for _ in feats]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.halo_predict_groups_static(sh, W1, W2, feats[0], 1, True, outs[0], status)      # set-up call
    B.halo_predict_groups_static(sh, W1, W2, feats[2], 32, True, outs[2], status)     # and the tensor-core branch
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    held_before, reserved_before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(5):
        for f, o in zip(feats, outs):
            B.halo_predict_groups_static(sh, W1, W2, f, f.shape[0], True, o, status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert torch.cuda.memory_allocated() == held_before and torch.cuda.memory_reserved() == reserved_before
    assert int(status.item()) == 0


def test_static_predictor_rejects_sizes_beyond_its_fixed_array():
    wl = synth.workload("llama2-13b-decode")
    W1, W2 = synth.predictor(wl, 1, DEV)
    per_tok = wl.pred_rank + wl.n_groups
    too_many = B.STATIC_SCRATCH_FLOATS // per_tok + 1
    feat = torch.zeros((too_many, wl.d_model), dtype=torch.bfloat16, device=DEV)
    scores = torch.zeros((wl.n_groups,), dtype=torch.float32, device=DEV)
    sh = B.pred_shape(wl.d_model, wl.pred_rank, wl.n_groups, B.BF16)
    with pytest.raises(B.HaloError) as err:
        B.halo_predict_groups_static(sh, W1, W2, feat, too_many, True, scores)
    assert err.value.code == -8
    # the largest size that fits is accepted
    fits = B.STATIC_SCRATCH_FLOATS // per_tok
    B.halo_predict_groups_static(sh, W1, W2, feat[:fits], fits, True, scores)
    torch.cuda.synchronize()
    assert (scores == 0).all().item()  # zero features -> zero scores
