"""Fit a predictor to the true group importance, and measure what importance-aware dropping buys.

    python -m paper_2601_11676_b200.calibrate [--workload tinyllama-1.1b-decode] [--train 2048] [--test 64]

The paper trains its semantic-aware predictors on activation norms gathered from a calibration set (Sec.
III-B.2).  No checkpoint or dataset is available here, so this tool works on a synthetic block whose groups
differ in importance and on inputs that carry "topic" content those groups respond to (synth.structured_layer,
synth.semantic_inputs).  Steps:
  1. targets: halo_group_importance (GPU) gives ||p_g|| for every calibration input;
  2. fit: the two-layer predictor s = W2 relu(W1 x) is trained on (x, norm) pairs by full-batch Adam with a mean
     squared error on the norms, the output layer initialised by ridge regression (offline training code in
     plain PyTorch; not part of the inference path);
  3. evaluation on held-out inputs through the library: halo_predict_groups scores vs true norms (relative
     validation loss, rank agreement), and the relative output error of the masked FFN when a fraction of the
     groups is dropped (a) lowest predicted score first = what HALO exposes to the lossy devices, (b) at random,
     (c) lowest true norm first (the best any predictor could do), (d) highest true norm first (the worst case).
Prints a table; returns the numbers as a dict.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2601_11676_b200 import binding as B  # noqa: E402
from paper_2601_11676_b200 import synth  # noqa: E402


def true_importance(ffn, Wp, X):
    G = ffn.d_ffn // ffn.group_size
    out = torch.empty((X.shape[0], G), dtype=torch.float32, device=X.device)
    ws = None
    for i in range(X.shape[0]):
        ws = B.halo_group_importance(ffn, Wp, X[i:i + 1].contiguous(), out[i], ws)
    torch.cuda.synchronize()
    return out


def masked_output(ffn, Wp, x, keep_ids, P, kl, nk):
    G = ffn.d_ffn // ffn.group_size
    kl.fill_(-1)
    ids = torch.sort(keep_ids).values.to(torch.int32)
    kl[: ids.numel()] = ids
    nk.fill_(ids.numel())
    B.halo_group_ffn(ffn, Wp, x, 1, kl, nk, None, 0, P, None, None)
    return P[0, 0].clone()


def run(workload="tinyllama-1.1b-decode", n_train=2048, n_test=64, drop_fractions=(0.125, 0.25, 0.5), ridge=1e-2,
        train_steps=400, lr=2e-3, seed=0, dev="cuda:0", verbose=True):
    wl = synth.workload(workload, seed=seed)
    assert wl.dtype == "bf16"
    G, d, r = wl.n_groups, wl.d_model, wl.pred_rank
    ffn = B.ffn_shape(d, wl.d_ffn, wl.group_size, B.BF16)
    Wp, topics = synth.structured_layer(wl, 1, dev)
    X = synth.semantic_inputs(wl, 777, topics, n_train + n_test)
    N = true_importance(ffn, Wp, X)
    Xtr, Ntr, Xte, Nte = X[:n_train].float(), N[:n_train], X[n_train:], N[n_train:]
    # fit (offline): start from a random hidden layer with a ridge-regressed output layer, then train both
    gen = torch.Generator(device=dev).manual_seed(seed * 1000003 + 4242)
    W1f = torch.empty((r, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    Z = torch.relu(Xtr @ W1f.T)
    A = Z.T @ Z + ridge * n_train * torch.eye(r, device=dev)
    W2f = torch.linalg.solve(A, Z.T @ Ntr).T.contiguous()                          # [G][r]
    W1f.requires_grad_(True)
    W2f.requires_grad_(True)
    opt = torch.optim.Adam([W1f, W2f], lr=lr)
    scale = float(Ntr.var().item())
    for _ in range(train_steps):
        opt.zero_grad(set_to_none=True)
        loss = ((torch.relu(Xtr @ W1f.T) @ W2f.T - Ntr) ** 2).mean() / scale
        loss.backward()
        opt.step()
    W1 = W1f.detach().to(torch.bfloat16).contiguous()
    W2 = W2f.detach().to(torch.bfloat16).contiguous()
    # evaluation through the library
    pred = B.pred_shape(d, r, G, B.BF16)
    ws = torch.empty(B.halo_predict_workspace_bytes(pred, n_test), dtype=torch.uint8, device=dev)
    S = torch.empty((n_test, G), dtype=torch.float32, device=dev)
    B.halo_predict_groups(pred, W1, W2, Xte.contiguous(), n_test, False, S, ws)
    torch.cuda.synchronize()
    val_loss = float(((S - Nte).abs().mean() / Nte.mean()).item())
    r2 = float((1.0 - ((S - Nte) ** 2).sum() / ((Nte - Nte.mean()) ** 2).sum()).item())
    # rank agreement: how much of the true bottom quarter is in the predicted bottom quarter
    q = max(1, G // 4)
    overlap = np.mean([len(set(torch.argsort(S[i])[:q].tolist()) & set(torch.argsort(Nte[i])[:q].tolist())) / q
                       for i in range(n_test)])
    P = torch.empty((1, 1, d), dtype=torch.float32, device=dev)
    kl = torch.empty((G,), dtype=torch.int32, device=dev)
    nk = torch.zeros((1,), dtype=torch.int32, device=dev)
    rng = torch.Generator(device="cpu").manual_seed(seed + 99)
    rows = []
    for f in drop_fractions:
        m = max(1, int(round(f * G)))
        errs = {"predicted-least": [], "random": [], "true-least": [], "true-most": []}
        for i in range(n_test):
            x = Xte[i:i + 1].contiguous()
            full = masked_output(ffn, Wp, x, torch.arange(G, device=dev), P, kl, nk)
            orders = {"predicted-least": torch.argsort(S[i]), "true-least": torch.argsort(Nte[i]),
                      "true-most": torch.argsort(Nte[i], descending=True),
                      "random": torch.randperm(G, generator=rng).to(dev)}
            for name, order in orders.items():
                y = masked_output(ffn, Wp, x, order[m:], P, kl, nk)
                errs[name].append(float(((y - full).norm() / full.norm()).item()))
        rows.append((f, {k: float(np.mean(v)) for k, v in errs.items()}))
    res = {"workload": workload, "groups": G, "train": n_train, "test": n_test, "val_loss": val_loss, "r2": r2,
           "bottom_quarter_overlap": float(overlap), "drop": rows}
    if verbose:
        print(f"{workload}: {G} groups, predictor rank {r}; relative L1 validation loss {val_loss:.3f}, R^2 {r2:.3f}; "
              f"bottom-quarter overlap {overlap:.2f} (chance {q / G:.2f})")
        print("| groups dropped | predicted-least (HALO) | random | true-least (best) | true-most (worst) |")
        print("|---|---|---|---|---|")
        for f, e in rows:
            print(f"| {f:.3f} | {e['predicted-least']:.3f} | {e['random']:.3f} | {e['true-least']:.3f} | {e['true-most']:.3f} |")
    return res


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="tinyllama-1.1b-decode")
    ap.add_argument("--train", type=int, default=2048)
    ap.add_argument("--test", type=int, default=64)
    a = ap.parse_args()
    B.lib()
    run(a.workload, a.train, a.test)
