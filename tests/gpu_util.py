"""Helpers shared by the GPU parity tests: run steps of the path through the C-ABI and fetch results to numpy."""
from __future__ import annotations

import numpy as np
import torch

from oracle import halo_ref as R
from paper_2601_11676_b200 import binding as B
from paper_2601_11676_b200 import synth

DEV = "cuda:0"

# max |y - y_ref| <= TOL * rms(y_ref): bf16 inputs with fp32 accumulation / fp32 inputs
TOL_BF16 = 2e-2
TOL_F32 = 1e-4


def tol_for(wl) -> float:
    return TOL_F32 if wl.dtype == "f32" else TOL_BF16


def dtype_code(wl) -> int:
    return B.F32 if wl.dtype == "f32" else B.BF16


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    rms = float(np.sqrt(np.mean(np.square(ref))))
    if rms == 0.0:
        return float(np.abs(got).max())
    return float(np.abs(got.astype(np.float64) - ref).max() / rms)


def gpu_select(plan: B.Plan, scores: torch.Tensor, step: int, layer: int, force_all: bool = False):
    G, n = plan.n_groups, plan.n_dev
    i32 = lambda k: torch.full((k,), -7, dtype=torch.int32, device=DEV)
    out = dict(order=i32(G), dev_of_group=i32(G), arrived=torch.full((max(n, 1),), 9, dtype=torch.uint8, device=DEV),
               keep=torch.full((G,), 9, dtype=torch.uint8, device=DEV), keep_list=i32(G), n_keep=i32(1),
               status=torch.zeros(1, dtype=torch.int32, device=DEV))
    B.halo_select_groups(plan, scores, step, layer, force_all, out["order"], out["dev_of_group"], out["arrived"],
                         out["keep"], out["keep_list"], out["n_keep"], out["status"])
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    res["arrived"] = res["arrived"][:n]
    res["n_keep"] = int(res["n_keep"][0])
    res["status"] = int(res["status"][0])
    return res, out


def assert_select_equal(gpu: dict, ref: dict):
    assert gpu["n_keep"] == ref["n_keep"]
    for k in ("order", "dev_of_group", "arrived", "keep", "keep_list"):
        assert (gpu[k] == ref[k]).all(), k
    assert (gpu["status"] & B.DEV_NONFINITE_SCORE != 0) == (ref["status"] & R.STATUS_NONFINITE != 0)


def gpu_predict(wl_dtype: int, W1, W2, feat, mean_pool=False, act=B.ACT_RELU):
    r, d_in = W1.shape
    G = W2.shape[0]
    n_tok = feat.shape[0]
    sh = B.pred_shape(d_in, r, G, wl_dtype, act)
    ws = torch.empty(B.halo_predict_workspace_bytes(sh, n_tok) // 4 + 4, dtype=torch.float32, device=DEV)
    scores = torch.empty((G,) if (mean_pool or n_tok == 1) else (n_tok, G), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.halo_predict_groups(sh, W1, W2, feat, n_tok, mean_pool, scores, ws, status)
    torch.cuda.synchronize()
    return scores, int(status.item())


def gpu_group_ffn(wl, Wp: torch.Tensor, x: torch.Tensor, keep_list, dev_of_group=None, n_dev=0):
    G = wl.n_groups
    sh = B.ffn_shape(wl.d_model, wl.d_ffn, wl.group_size, dtype_code(wl))
    n_tok = x.shape[0]
    kl = torch.full((G,), -1, dtype=torch.int32, device=DEV)
    if len(keep_list):
        kl[: len(keep_list)] = torch.as_tensor(np.asarray(keep_list, dtype=np.int32), device=DEV)
    nk = torch.tensor([len(keep_list)], dtype=torch.int32, device=DEV)
    dg = None if dev_of_group is None else torch.as_tensor(np.asarray(dev_of_group, dtype=np.int32), device=DEV)
    P = torch.full((n_dev + 1, n_tok, wl.d_model), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws_bytes = B.halo_group_ffn_workspace_bytes(sh, n_tok, n_dev)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=DEV) if ws_bytes else None
    B.halo_group_ffn(sh, Wp, x, n_tok, kl, nk, dg, n_dev, P, ws, status)
    torch.cuda.synchronize()
    return P, int(status.item())


def gpu_merge(P: torch.Tensor, arrived=None):
    n_slots, n_tok, d = P.shape
    y = torch.empty((n_tok, d), dtype=torch.float32, device=DEV)
    arr = None if arrived is None else torch.as_tensor(np.asarray(arrived, dtype=np.uint8), device=DEV)
    B.halo_merge_partials(P, arr, n_slots - 1, n_tok, d, y)
    torch.cuda.synchronize()
    return y


def layer_tensors(wl, layer: int):
    Wp = synth.packed_layer(wl, layer, DEV)
    W1, W2 = synth.predictor(wl, layer, DEV)
    return Wp, W1, W2
