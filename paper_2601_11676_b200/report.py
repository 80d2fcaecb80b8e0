"""Sweeps of the decode stack over workloads, keep ratios and execution modes; prints a markdown table.

    python -m paper_2601_11676_b200.report [--steps 64] [--quick]
    python -m paper_2601_11676_b200.report --prefill-vs-library


Rows: every decode workload at its stated keep ratio; the 7B keep-ratio sweep {0.3, 0.5, 0.7, 1.0}; the same
sweep with every virtual device always lost (kept fraction = keep ratio exactly: pure top-k sparsity); and the
overlap ablation: mode 0 (one persistent kernel, predictor + selection of block l+1 overlapped with the weight
stream of block l) against mode 1 (one launch per step of the path, nothing overlapped).

--prefill-vs-library: the FFN of one 7B-shaped block on a 512-token prompt (all 86 groups kept), through
halo_group_ffn and, beside it, the same two contractions as plain dense library GEMMs (torch.matmul; gate and up
as one GEMM, SiLU*mul by torch, then the down GEMM) on the same rotating weight sets, both timed over a run long
enough for the power cap to set the clocks.  The library arm does no masking, slots or reductions: it is the
dense ceiling for this shape, printed for context.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2601_11676_b200 import binding as B  # noqa: E402
from paper_2601_11676_b200 import synth  # noqa: E402


def measure(wl, weights, preds, steps, warm, mode, dev="cuda:0"):
    code = B.BF16
    plan = B.Plan(wl.n_groups, wl.loss_rate, wl.share_weight, B.SEL_TOPK, wl.k_critical, 0.0, wl.seed)
    ffn = B.ffn_shape(wl.d_model, wl.d_ffn, wl.group_size, code)
    pred = B.pred_shape(wl.d_model, wl.pred_rank, wl.n_groups, code)
    stack = B.Stack(ffn, pred, 1, plan, weights, [p[0] for p in preds], [p[1] for p in preds])
    stack.set_mode(mode)
    L, G = wl.n_layers, wl.n_groups
    total = warm + steps
    h0 = torch.stack([synth.stream_input(wl, s, dev) for s in range(total)])
    out = torch.empty_like(h0)
    nk = torch.zeros((total, L), dtype=torch.int32, device=dev)
    stack.decode(h0, total, 0, out, B.Taps(None, None, None, None, None, nk.data_ptr(), None))
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    stack.decode(h0[warm:], steps, warm, out[warm:])
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b)
    kept = int(nk[warm:].sum().item())
    byts = kept * wl.group_bytes + steps * (L - 1) * wl.pred_bytes
    res = dict(tokens_per_s=steps / (ms * 1e-3), us_per_block=ms * 1e3 / (steps * L), gbs=byts / (ms * 1e-3) / 1e9,
               kept_fraction=kept / float(steps * L * G), launches=stack.last_launches(), status=stack.status())
    stack.close()
    return res


def prefill_vs_library(dev="cuda:0", n_sets=8, reps=40):
    wl = synth.workload("llama2-7b-prefill")
    T, d, F, S, G = wl.n_tok, wl.d_model, wl.d_ffn, wl.group_size, wl.n_groups
    sh = B.ffn_shape(d, F, S, B.BF16)
    Wp = [synth.packed_layer(wl, l, dev) for l in range(n_sets)]                     # [G][3][S][d]
    Wgu = [w.view(G, 3, S, d)[:, :2].permute(1, 0, 2, 3).reshape(2 * F, d).contiguous() for w in Wp]   # [2F][d]
    Wdn = [w.view(G, 3, S, d)[:, 2].reshape(F, d).contiguous() for w in Wp]          # [F][d] (down columns as rows)
    x = synth.activation(wl, 3, dev, n_tok=T)
    ws = torch.empty(B.halo_group_ffn_workspace_bytes(sh, T, 0), dtype=torch.uint8, device=dev)
    P = torch.empty((1, T, d), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    kl = torch.arange(G, dtype=torch.int32, device=dev)
    nk = torch.tensor([G], dtype=torch.int32, device=dev)

    def ours(i):
        B.halo_group_ffn(sh, Wp[i % n_sets], x, T, kl, nk, None, 0, P, ws, status)

    def library(i):
        gu = torch.matmul(x, Wgu[i % n_sets].t())
        h = torch.nn.functional.silu(gu[:, :F].float()).mul_(gu[:, F:].float()).to(torch.bfloat16)
        return torch.matmul(h, Wdn[i % n_sets])

    def library_gemms_only(i):
        gu = torch.matmul(x, Wgu[i % n_sets].t())
        return torch.matmul(gu[:, :F], Wdn[i % n_sets])

    flops = 6.0 * T * F * d
    rows = []
    for name, fn in (("halo_group_ffn (one launch, 86 of 86 groups)", ours), ("library GEMMs + torch SiLU*mul", library),
                     ("library GEMMs only (no activation)", library_gemms_only)):
        for i in range(2 * n_sets):
            fn(i)
        torch.cuda.synchronize()
        times = []
        for _ in range(3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(reps * n_sets):
                fn(i)
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b) * 1e3 / (reps * n_sets))
        us = sorted(times)[1]
        rows.append((name, us, flops / us / 1e6))
    assert int(status.item()) == 0
    ref = library(0).float()
    ours(0)
    torch.cuda.synchronize()
    err = (P[0] - ref).abs().max().item() / ref.abs().max().item()
    print("| FFN of one 7B-shaped block, 512 tokens, bf16 | µs per block (median of 3 runs of %d calls) | TFLOP/s |" % (reps * n_sets))
    print("|---|---|---|")
    for name, us, tf in rows:
        print(f"| {name} | {us:.1f} | {tf:.0f} |")
    print(f"\nlargest difference between the two results: {err:.2e} of the largest output")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--prefill-vs-library", action="store_true",
                    help="time halo_group_ffn on a 512-token prompt beside plain dense library GEMMs")
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--quick", action="store_true", help="7B only")
    args = ap.parse_args()
    B.lib()
    dev = "cuda:0"
    if args.prefill_vs_library:
        prefill_vs_library(dev)
        return
    peak = 6544.0
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        peak = float(json.load(open(pk)).get("hbm_gbs", peak))
    rows = []
    names = ["llama2-7b-decode"] if args.quick else ["llama2-7b-decode", "llama2-13b-decode", "tinyllama-1.1b-decode"]
    for name in names:
        base = synth.workload(name)
        weights = [synth.packed_layer(base, l, dev) for l in range(base.n_layers)]
        preds = [synth.predictor(base, l, dev) for l in range(base.n_layers)]
        variants = [("as stated", base, 0), ("as stated, no overlap (mode 1)", base, 1)]
        if name == "llama2-7b-decode":
            for pm in (300, 700, 1000):
                variants.append((f"keep {pm / 1000:.1f}", dataclasses.replace(base, keep_permille=pm), 0))
            for pm in (300, 500, 700):
                lost = dataclasses.replace(base, keep_permille=pm, loss_rate=tuple(1.0 for _ in base.loss_rate))
                variants.append((f"keep {pm / 1000:.1f}, every device lost (supplementary)", lost, 0))
        for label, wl, mode in variants:
            r = measure(wl, weights, preds, args.steps, args.warmup, mode, dev)
            rows.append((name, label, r))
        del weights, preds
        torch.cuda.empty_cache()
    print("| workload | variant | kept | tokens/s | µs/block | algorithmic GB/s | of 8 TB/s | of measured %.0f | launches |" % peak)
    print("|---|---|---|---|---|---|---|---|---|")
    for name, label, r in rows:
        print(f"| {name} | {label} | {r['kept_fraction']:.3f} | {r['tokens_per_s']:.1f} | {r['us_per_block']:.2f} | "
              f"{r['gbs']:.0f} | {r['gbs'] / 8000:.3f} | {r['gbs'] / peak:.3f} | {r['launches']} |")
        assert r["status"] == 0, r


if __name__ == "__main__":
    main()
