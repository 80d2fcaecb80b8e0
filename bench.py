#!/usr/bin/env python
"""Benchmark of the group-sparse FFN hot path (predict -> select -> group FFN -> merge, chained as a stack).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl halo|reference]

One step = one token through every block of the workload's FFN stack.  Prints ONE JSON line (rank 0).
With N > 1 every rank runs an independent replica on its own GPU (the path has no exchange between GPUs).
`--impl reference` times the CPU fp64 oracle on the host cores instead (a deliberately plain program).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_11676_b200 import synth  # noqa: E402

METRIC = "group-sparse FFN decode tokens/s on 1 B200; achieved HBM GB/s vs ~8 TB/s"
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read+write per launch / algorithmic bytes per launch of stack_decode_kernel, from an ncu capture of a
# 4-block 7B-shaped case (profiles/stack_decode_kernel_llama2-7b_4blocks.md); traffic is proportional to the kept
# groups processed, so the ratio carries over to the full-size launch.  The figure belongs to the kernel sources with
# the hash below: when they change the line reports no traffic until the counters have been taken again.
STACK_KERNEL_TRAFFIC_RATIO = 1.0007
STACK_KERNEL_SOURCES = ("stack_persistent.cu", "stack_persistent.cuh", "ffn_math.cuh", "i4_math.cuh", "tma.cuh", "umma.cuh",
                        "select_device.cuh")
STACK_KERNEL_SOURCES_SHA1 = "7ae621467ca99f174feac17d4c5484231b8f22ea"
FALLBACK_HBM_GBS = 6650.0


def stack_kernel_sources_sha1():
    import hashlib
    h = hashlib.sha1()
    for name in STACK_KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2601_11676_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d.get("hbm_gbs", FALLBACK_HBM_GBS)), "measured"
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons, mx, pw = [], set(), None, []
        try:
            for ln in open(self.path):
                f = [v.strip() for v in ln.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx = float(f[2])
                except ValueError:
                    continue
                try:
                    pw.append(float(f[3]))
                except ValueError:
                    pass
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            busy = [v for v in sm if v >= 0.5 * max(sm)] or sm
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
            if pw:
                out.update(power_w_max=max(pw))
        return out


# ----------------------------------------------------------------------------------------------------------------
# replicas: every rank runs the same workload on its own GPU; the job's time is the slowest rank's
# ----------------------------------------------------------------------------------------------------------------

def max_over_ranks(values, world, device):
    """Element-wise maximum of a list of floats over all ranks (identity for a single process)."""
    if world <= 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_tokens_per_s(tokens_per_rank, ms_this_rank, world, device):
    """Whole-job tokens/s of `world` independent replicas: all ranks' tokens over the slowest rank's time."""
    (ms,) = max_over_ranks([ms_this_rank], world, device)
    return tokens_per_rank * world / (ms * 1e-3), ms


# ----------------------------------------------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------------------------------------------

def tokens_of(K, world):
    return K * world


def workload_config(wl, world):
    """The same keys in both arms: what the workload is, not how a particular run went."""
    return {"workload": wl.name, "n_layers": wl.n_layers, "d_model": wl.d_model, "d_ffn": wl.d_ffn,
            "group_size": wl.group_size, "n_groups": wl.n_groups, "pred_rank": wl.pred_rank,
            "keep_permille": wl.keep_permille, "k_critical": (wl.keep_permille * wl.n_groups + 999) // 1000,
            "virtual_devices": wl.n_dev, "loss_rate": list(wl.loss_rate),
            "l2": "inputs larger than L2 (weights of the stack: %.2f GB)" % (wl.n_layers * wl.layer_bytes / 1e9),
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def build_stack(wl, dev):
    from paper_2601_11676_b200 import binding as B
    code = B.F32 if wl.dtype == "f32" else B.BF16
    Wp = [synth.packed_layer(wl, l, dev) for l in range(wl.n_layers)]
    preds = [synth.predictor(wl, l, dev) for l in range(wl.n_layers)]
    plan = B.Plan(wl.n_groups, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    ffn = B.ffn_shape(wl.d_model, wl.d_ffn, wl.group_size, code)
    pred = B.pred_shape(wl.d_model, wl.pred_rank, wl.n_groups, code)
    stack = B.Stack(ffn, pred, wl.n_tok, plan, Wp, [p[0] for p in preds], [p[1] for p in preds])
    return stack, Wp, preds, plan, ffn


def run_halo(args, rank, world, local_rank):
    from paper_2601_11676_b200 import binding as B
    B.lib()  # fail loudly if the CUDA library is missing
    for item in args.option:
        name, _, value = item.partition("=")
        B.halo_set_option(name, int(value))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    wl = synth.workload(args.workload, keep_permille=args.keep_permille)
    if args.layers:
        wl = synth.small_variant(wl, args.layers, wl.steps)
    K, W = args.steps, args.warmup
    stack, Wp, preds, plan, ffn = build_stack(wl, dev)
    L, G, d = wl.n_layers, wl.n_groups, wl.d_model
    total_steps = W + K
    h0 = torch.stack([synth.stream_input(wl, s, dev) for s in range(total_steps)])
    h_out = torch.empty_like(h0)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    # ---- record the kept sets of the timed steps once (taps), for the byte accounting ------------------------
    nk_rec = torch.zeros((total_steps, L), dtype=torch.int32, device=dev)
    kl_rec = torch.zeros((total_steps, L, G), dtype=torch.int32, device=dev)
    dg_rec = torch.zeros((total_steps, L, G), dtype=torch.int32, device=dev)
    taps = B.Taps(None, None, dg_rec.data_ptr(), None, kl_rec.data_ptr(), nk_rec.data_ptr(), None)
    stack.decode(h0, total_steps, 0, h_out, taps)
    torch.cuda.synchronize()
    if stack.status() != 0:
        raise RuntimeError("device status: " + B.status_message(stack.status()))
    nk_timed = nk_rec[W:].cpu().numpy().astype(np.int64)
    kept_groups = int(nk_timed.sum())
    kept_fraction = kept_groups / float(K * L * G)
    weight_bytes = kept_groups * wl.group_bytes
    pred_bytes = K * (L - 1) * wl.pred_bytes
    algo_bytes_total = weight_bytes + pred_bytes

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps, REPS times back to back inside one
    #      sampled region; the median run is the reported one, all runs are listed ----------------------------------
    REPS = 5
    stack.decode(h0[:W], W, 0, h_out[:W])
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(REPS)]
    barrier()
    for ev0, ev1 in evs:
        ev0.record()
        stack.decode(h0[W:], K, W, h_out[W:])
        ev1.record()
    barrier()
    runs_ms = [ev0.elapsed_time(ev1) for ev0, ev1 in evs]
    ms = sorted(runs_ms)[REPS // 2]
    launches = stack.last_launches()
    clocks = sampler.stop() if rank == 0 else None
    if stack.status() != 0:
        raise RuntimeError("device status after the timed run: " + B.status_message(stack.status()))

    # ---- end to end through the host entry point: pinned host buffers, copies inside the timed region ----------
    h0_host = h0[W:].cpu().pin_memory()
    out_host = torch.empty_like(h0_host).pin_memory()
    stack.decode_host(h0_host[: max(W, 1)], max(W, 1), 0, out_host[: max(W, 1)])
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    stack.decode_host(h0_host, K, W, out_host)
    e1.record()
    torch.cuda.synchronize()
    ms_e2e = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)

    # ---- dominant kernel alone: the group FFN of every block, one sweep over the stack per timing ---------------
    x = synth.activation(wl, 1, dev)
    partials = torch.empty((wl.n_dev + 1, 1, d), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    sweep_steps = list(range(W, W + min(K, 8)))
    for l in range(L):  # warm-up sweep
        B.halo_group_ffn(ffn, Wp[l], x, 1, kl_rec[W, l], nk_rec[W, l:l + 1], dg_rec[W, l], wl.n_dev, partials, None, status)
    torch.cuda.synchronize()
    k_ms, k_bytes, k_launches = 0.0, 0, 0
    for s in sweep_steps:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for l in range(L):
            B.halo_group_ffn(ffn, Wp[l], x, 1, kl_rec[s, l], nk_rec[s, l:l + 1], dg_rec[s, l], wl.n_dev, partials, None,
                             status)
        b.record()
        torch.cuda.synchronize()
        k_ms += a.elapsed_time(b)
        k_launches += L
        k_bytes += int(nk_rec[s].sum().item()) * wl.group_bytes
    kernel_avg_us = k_ms * 1e3 / k_launches
    kernel_gbs = k_bytes / (k_ms * 1e-3) / 1e9

    # ---- max over ranks -------------------------------------------------------------------------------------------
    ms, ms_e2e = max_over_ranks([ms, ms_e2e], world, dev)
    runs_ms = max_over_ranks(runs_ms, world, dev)
    if rank != 0:
        return None

    peak, peak_kind = measured_peaks()
    tokens = K * world
    value = tokens / (ms * 1e-3)   # == aggregate_tokens_per_s(K, ms_local, world, dev)[0]: ms is already the max
    step_gbs = algo_bytes_total / (ms * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.dtype, "data": "synthetic",
        "config": dict(workload_config(wl, world), kept_fraction=kept_fraction),
        "runs": {"ms_per_step": [r / K for r in runs_ms], "tokens_per_s": [tokens_of(K, world) / (r * 1e-3) for r in runs_ms],
                 "reported": "median of %d back-to-back runs of the K timed steps" % len(runs_ms)},
        "clocks": clocks,
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": 4 * d * wl.n_tok,
                "d2h_bytes_per_step": 4 * d * wl.n_tok},
        "gpu_launches": int(launches),
        "hbm": {"algorithmic_gb_per_token": algo_bytes_total / K / 1e9, "achieved_gbs": step_gbs,
                "frac_of_nominal_8tbs": step_gbs / NOMINAL_HBM_GBS, "frac_of_peak": step_gbs / peak,
                "peak_gbs": peak, "peak_kind": peak_kind},
    }
    persistent = launches == 1
    if args.option:
        result["options"] = list(args.option)     # a tuning sweep, not the default configuration
    traffic_valid = STACK_KERNEL_TRAFFIC_RATIO is not None and stack_kernel_sources_sha1() == STACK_KERNEL_SOURCES_SHA1
    if persistent:
        # the timed region is ONE launch of the persistent stack kernel: its duration is the event time itself
        result["roofline"] = {
            "bound": "hbm", "kernel": "stack_decode_kernel (persistent: all steps x blocks, a1..a9 + glue)",
            "achieved": step_gbs, "peak": peak, "unit": "GB/s", "frac": step_gbs / peak, "peak_kind": peak_kind,
            "traffic": (algo_bytes_total * STACK_KERNEL_TRAFFIC_RATIO) if traffic_valid else None,
            "traffic_note": ("scaled: ncu DRAM bytes of a 4-block capture x kept groups processed "
                             "(kernel sources %s)" % STACK_KERNEL_SOURCES_SHA1[:12]) if traffic_valid else
                            "none: the kernel sources changed since the counters were taken",
            "peak_note": "the peak is a read+write copy; a read-only stream can pass it" if step_gbs > peak else None,
            "avg_launch_us": ms * 1e3, "launches_timed": len(runs_ms),
            "algorithmic_bytes_per_launch": algo_bytes_total, "frac_of_nominal_8tbs": step_gbs / NOMINAL_HBM_GBS}
    else:
        result["roofline"] = {
            "bound": "hbm", "kernel": "group_ffn kernel (one launch per block)", "achieved": kernel_gbs, "peak": peak,
            "unit": "GB/s", "frac": kernel_gbs / peak, "peak_kind": peak_kind, "traffic": None,
            "avg_launch_us": kernel_avg_us, "launches_timed": k_launches,
            "frac_of_nominal_8tbs": kernel_gbs / NOMINAL_HBM_GBS}
    # the unfused halo_group_ffn entry point timed alone (memset + kernel per call), for comparison
    result["group_ffn_entry"] = {"achieved_gbs": kernel_gbs, "avg_call_us": kernel_avg_us, "calls_timed": k_launches,
                                 "frac_of_peak": kernel_gbs / peak}
    if world == 1 and not args.no_prefill and wl.dtype == "bf16" and wl.n_tok == 1:
        result["prefill"] = prefill_report(wl, Wp, preds, plan, ffn, dev)
    if world == 1 and not args.no_extra and not args.layers:
        # the other decode workloads, briefly (same measurement, fewer steps); the headline stays `value`
        del stack, Wp, preds
        torch.cuda.empty_cache()
        result["other_workloads"] = [decode_brief(n, dev, peak) for n in
                                     ("llama2-13b-decode", "tinyllama-1.1b-decode", "llama2-7b-decode")
                                     if n != wl.name]
        result["other_blocks"] = other_blocks_report(dev, peak)
        result["int4_stack"] = int4_stack_report(dev, peak)
        result["block_stack"] = block_stack_report(dev, peak)
        result["block_stack_int4"] = block_stack_report(dev, peak, int4=True)
        result["keep_sweep"] = keep_sweep(dev, peak)
        result["overlap_ablation"] = overlap_ablation(dev)
    if world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(wl, budget_s=args.cpu_budget)
    return result


def other_blocks_report(dev, peak, reps=12):
    """The paper's two other block types at the 7B shape, one token: LM-head groups (32000 x 4096, all groups) and
    MHA groups (32 heads of 128, 1024 cached positions, K/V append + attention + output projection); microseconds
    per call and algorithmic GB/s.  Weight sets rotate so that every call streams from HBM."""
    from paper_2601_11676_b200 import binding as B
    d, vocab, S, H, dh, Lmax, pos = 4096, 32000, 256, 32, 128, 1024, 1023
    wl = synth.Workload("blocks", 1, d, 64, 16, 32, "bf16", (0.0, 0.2, 0.6), (2, 1, 1), 500, 1)
    x = synth.activation(wl, 1, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def timed(fn):
        for _ in range(4):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):          # 32 calls back to back per window: the first launch's latency is not what is measured
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(32):
                fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3 / 32)
        return float(sorted(ts)[len(ts) // 2])

    g = torch.Generator(device="cpu").manual_seed(11)
    lm = B.lm_shape(d, vocab, S, B.BF16)
    Wl = [(torch.randn((vocab, d), generator=g) / 64).to(torch.bfloat16).to(dev) for _ in range(3)]
    logits = torch.empty((1, vocab), dtype=torch.float32, device=dev)
    i = [0]

    def lm_call():
        B.halo_group_lm_head(lm, Wl[i[0] % 3], x, 1, None, None, logits, status)
        i[0] += 1

    lm_us = timed(lm_call)
    lm_bytes = vocab * d * 2
    # the same head on int4 rows (three quantised copies rotate)
    lmq = []
    for W in Wl:
        q = torch.empty((vocab, d // 2), dtype=torch.uint8, device=dev)
        sc = torch.empty((vocab, d // 128), dtype=torch.bfloat16, device=dev)
        B.halo_quantize_rows_i4(d, vocab, B.BF16, W, q, sc)
        lmq.append((q, sc))
    torch.cuda.synchronize()
    del Wl

    def lm_i4_call():
        q, sc = lmq[i[0] % 3]
        B.halo_group_lm_head_i4(lm, q, sc, x, 1, None, None, logits, status)
        i[0] += 1

    lm_i4_us = timed(lm_i4_call)
    lm_i4_bytes = vocab * (d // 2 + (d // 128) * 2)
    del lmq
    mh = B.mha_shape(d, H, dh, Lmax, B.BF16)
    sets = []
    for l in range(6):
        Wq, Wk, Wv, Wo = synth.mha_matrices(wl, l, H, dev)
        Wp = torch.empty((H, 2, dh, d), dtype=torch.bfloat16, device=dev)
        B.halo_pack_mha_weights(mh, Wq, Wo, Wp)
        K = torch.randn((H, Lmax, dh), device=dev).to(torch.bfloat16)
        V = torch.randn((H, Lmax, dh), device=dev).to(torch.bfloat16)
        sets.append((Wp, Wk, Wv, K, V))
    ws = torch.empty(B.halo_group_mha_workspace_bytes(mh), dtype=torch.uint8, device=dev)
    P = torch.empty((4, d), dtype=torch.float32, device=dev)
    dg = torch.as_tensor([(-1, 0, 1, 2)[h % 4] for h in range(H)], dtype=torch.int32, device=dev)
    kl = torch.arange(H, dtype=torch.int32, device=dev)
    nk = torch.tensor([H], dtype=torch.int32, device=dev)
    j = [0]

    def mha_call():
        Wp, Wk, Wv, K, V = sets[j[0] % 6]
        j[0] += 1
        B.halo_mha_block(mh, Wp, Wk, Wv, x, K, V, pos, kl, nk, dg, 3, P, status)

    def mha_two_calls():
        Wp, Wk, Wv, K, V = sets[j[0] % 6]
        j[0] += 1
        B.halo_mha_kv_append(mh, Wk, Wv, x, pos, K, V)
        B.halo_group_mha(mh, Wp, x, K, V, pos, kl, nk, dg, 3, P, ws, status)

    mha_us = timed(mha_call)
    mha_two_us = timed(mha_two_calls)
    mha_bytes = 2 * d * d * 2 + H * (2 * dh * d * 2 + 2 * (pos + 1) * dh * 2)
    # the same block on int4 weights (caches stay bf16)
    def qrows(W2d):
        rows = W2d.shape[0]
        q = torch.empty((rows, d // 2), dtype=torch.uint8, device=dev)
        sc = torch.empty((rows, d // 128), dtype=torch.bfloat16, device=dev)
        B.halo_quantize_rows_i4(d, rows, B.BF16, W2d, q, sc)
        return q, sc
    sets4 = [(qrows(Wp.view(-1, d)), qrows(Wk), qrows(Wv), K, V) for (Wp, Wk, Wv, K, V) in sets]
    torch.cuda.synchronize()
    del sets

    def mha_i4_call():
        (Qp, Sp), (Qk, Sk), (Qv, Sv), K, V = sets4[j[0] % 6]
        j[0] += 1
        B.halo_mha_block_i4(mh, Qp, Sp, Qk, Sk, Qv, Sv, x, K, V, pos, kl, nk, dg, 3, P, status)

    mha_i4_us = timed(mha_i4_call)
    wb4 = 0.5 + 2.0 / 128.0
    mha_i4_bytes = 2 * d * d * wb4 + H * (2 * dh * d * wb4 + 2 * (pos + 1) * dh * 2)
    del sets4
    # the FFN of one 7B-shaped block on int4 group-quantised weights, all groups kept
    fw = synth.workload("llama2-7b-decode")
    G, S = fw.n_groups, fw.group_size
    fsh = B.ffn_shape(d, fw.d_ffn, S, B.BF16)
    quant = []
    for l in range(8):
        Wf = synth.packed_layer(fw, l, dev)
        Q = torch.empty((G, 3, S, d // 2), dtype=torch.uint8, device=dev)
        Sc = torch.empty((G, 3, S, d // 128), dtype=torch.bfloat16, device=dev)
        B.halo_quantize_weights_i4(fsh, Wf, Q, Sc)
        quant.append((Q, Sc))
        del Wf
    fkl = torch.arange(G, dtype=torch.int32, device=dev)
    fnk = torch.tensor([G], dtype=torch.int32, device=dev)
    fdg = torch.as_tensor([(-1, 0, 1, 2)[g % 4] for g in range(G)], dtype=torch.int32, device=dev)
    FP = torch.empty((4, 1, d), dtype=torch.float32, device=dev)
    k = [0]

    def i4_call():
        Q, Sc = quant[k[0] % 8]
        k[0] += 1
        B.halo_group_ffn_i4(fsh, Q, Sc, x, 1, fkl, fnk, fdg, 3, FP, status)

    i4_us = timed(i4_call)
    i4_bytes = G * 3 * S * (d // 2 + (d // 128) * 2)
    return {"lm_head": {"shape": "32000 x 4096 bf16, 125 groups of 256 rows", "us_per_token": lm_us,
                        "achieved_gbs": lm_bytes / lm_us / 1e3, "frac_of_peak": lm_bytes / lm_us / 1e3 / peak},
            "lm_head_int4": {"shape": "32000 x 4096 int4 rows + bf16 scales per 128", "us_per_token": lm_i4_us,
                             "achieved_gbs": lm_i4_bytes / lm_i4_us / 1e3,
                             "frac_of_peak": lm_i4_bytes / lm_i4_us / 1e3 / peak},
            "mha_groups": {"shape": "32 heads x 128, d 4096, 1024 cached positions, all heads kept; halo_mha_block "
                                    "(K/V append + attention + output projection in one launch)",
                           "us_per_block": mha_us, "achieved_gbs": mha_bytes / mha_us / 1e3,
                           "frac_of_peak": mha_bytes / mha_us / 1e3 / peak,
                           "us_per_block_as_two_calls": mha_two_us},
            "mha_groups_int4": {"shape": "the same block on int4 weights, bf16 caches; halo_mha_block_i4",
                                "us_per_block": mha_i4_us, "achieved_gbs": mha_i4_bytes / mha_i4_us / 1e3,
                                "frac_of_peak": mha_i4_bytes / mha_i4_us / 1e3 / peak},
            "ffn_int4": {"shape": "one 7B block, 86 groups of 128, int4 weights + bf16 scales per 128, all kept",
                         "us_per_block": i4_us, "achieved_gbs": i4_bytes / i4_us / 1e3,
                         "frac_of_peak": i4_bytes / i4_us / 1e3 / peak,
                         "bf16_equivalent_gbs": G * 3 * S * d * 2 / i4_us / 1e3},
            "device_status": int(status.item())}


def _timed_decode(stack, wl, dev, steps, warm, reps=3):
    """Median milliseconds of `steps` tokens through `stack` (one decode call), and the kept groups of those steps."""
    from paper_2601_11676_b200 import binding as B
    L = wl.n_layers
    total = warm + steps
    h0 = torch.stack([synth.stream_input(wl, s, dev) for s in range(total)])
    out = torch.empty_like(h0)
    nk = torch.zeros((total, L), dtype=torch.int32, device=dev)
    stack.decode(h0, total, 0, out, B.Taps(None, None, None, None, None, nk.data_ptr(), None))
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        stack.decode(h0[warm:], steps, warm, out[warm:])
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    return sorted(ts)[len(ts) // 2], int(nk[warm:].sum().item())


def keep_sweep(dev, peak, steps=48, warm=4):
    """The 7B-shaped stack at the keep ratios of its configuration, with the stated loss rates and - supplementary -
    with every virtual device always lost, where the kept fraction is the keep ratio itself (the predictor's top-k
    alone decides what is read).  Bytes are counted over the kept groups of the timed steps."""
    from paper_2601_11676_b200 import binding as B
    base = synth.workload("llama2-7b-decode")
    Wp = [synth.packed_layer(base, l, dev) for l in range(base.n_layers)]
    preds = [synth.predictor(base, l, dev) for l in range(base.n_layers)]
    ffn = B.ffn_shape(base.d_model, base.d_ffn, base.group_size, B.BF16)
    pred = B.pred_shape(base.d_model, base.pred_rank, base.n_groups, B.BF16)
    rows = []
    for lost in (False, True):
        for permille in (300, 500, 700, 1000):
            wl = synth.workload("llama2-7b-decode", keep_permille=permille,
                                loss_rate=(1.0,) * base.n_dev if lost else base.loss_rate)
            plan = B.Plan(wl.n_groups, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
            stack = B.Stack(ffn, pred, 1, plan, Wp, [p[0] for p in preds], [p[1] for p in preds])
            ms, kept = _timed_decode(stack, wl, dev, steps, warm)
            byts = kept * wl.group_bytes + steps * (wl.n_layers - 1) * wl.pred_bytes
            gbs = byts / (ms * 1e-3) / 1e9
            rows.append({"keep_permille": permille, "devices": "all lost (supplementary)" if lost else "as configured",
                         "kept_fraction": kept / float(steps * wl.n_layers * wl.n_groups),
                         "tokens_per_s": steps / (ms * 1e-3), "achieved_gbs": gbs,
                         "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS, "frac_of_peak": gbs / peak,
                         "device_status": stack.status()})
            stack.close()
    return {"workload": "llama2-7b-decode", "steps": steps, "rows": rows}


def overlap_ablation(dev, steps=48, warm=4):
    """The arms of the paper's overlap ablation (Table V) restated for one GPU, all inside the persistent kernel:
    predictor + selection beside the previous block's stream or in front of the block's own; first weights of the
    next block fetched during the merge or not; and, for scale, one launch per step of the path."""
    from paper_2601_11676_b200 import binding as B
    out = []
    for name in ("llama2-7b-decode", "tinyllama-1.1b-decode"):
        wl = synth.workload(name)
        stack, Wp, preds, plan, ffn = build_stack(wl, dev)
        arms = [("both overlaps (default)", 0), ("Pred overlapped only", B.STACK_LOAD_SERIAL),
                ("Load overlapped only", B.STACK_PRED_SERIAL), ("no overlap", B.STACK_PRED_SERIAL | B.STACK_LOAD_SERIAL),
                ("one launch per step of the path", B.STACK_PER_STEP_LAUNCHES)]
        ms_of = {}
        for label, mode in arms:
            stack.set_mode(mode)
            ms_of[label], _ = _timed_decode(stack, wl, dev, steps, warm)
        base = ms_of["no overlap"]
        out.append({"workload": name, "steps": steps,
                    "arms": [{"arm": label, "ms_per_token": ms_of[label] / steps, "tokens_per_s": steps / (ms_of[label] * 1e-3),
                              "speedup_over_no_overlap": base / ms_of[label]} for label, _ in arms]})
        stack.close()
        del stack, Wp, preds
        torch.cuda.empty_cache()
    return out


def int4_stack_report(dev, peak, steps=32, warm=4):
    """The 7B-shaped FFN stack on int4 group-quantised weights (the paper's models are 4-bit): tokens/s and GB/s over the
    int4 bytes of the kept groups (codes + scales) and the predictors.  One persistent launch (the int4 form of the
    decode kernel)."""
    from paper_2601_11676_b200 import binding as B
    wl = synth.workload("llama2-7b-decode")
    L, G, S, d = wl.n_layers, wl.n_groups, wl.group_size, wl.d_model
    fsh = B.ffn_shape(d, wl.d_ffn, S, B.BF16)
    Q, Sc = [], []
    for l in range(L):
        Wf = synth.packed_layer(wl, l, dev)
        q = torch.empty((G, 3, S, d // 2), dtype=torch.uint8, device=dev)
        sc = torch.empty((G, 3, S, d // 128), dtype=torch.bfloat16, device=dev)
        B.halo_quantize_weights_i4(fsh, Wf, q, sc)
        torch.cuda.synchronize()
        Q.append(q); Sc.append(sc)
        del Wf
    preds = [synth.predictor(wl, l, dev) for l in range(L)]
    plan = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    stack = B.Stack(fsh, B.pred_shape(d, wl.pred_rank, G, B.BF16), 1, plan, Q, [p[0] for p in preds], [p[1] for p in preds],
                    i4_scales=Sc)
    ms, kept = _timed_decode(stack, wl, dev, steps, warm)
    group_bytes_i4 = 3 * S * (d // 2 + (d // 128) * 2)
    byts = kept * group_bytes_i4 + steps * (L - 1) * wl.pred_bytes
    gbs = byts / (ms * 1e-3) / 1e9
    res = {"workload": "llama2-7b-decode on int4 weights (one bf16 scale per 128 elements)", "steps": steps,
           "tokens_per_s": steps / (ms * 1e-3), "ms_per_token": ms / steps,
           "kept_fraction": kept / float(steps * L * G), "achieved_gbs": gbs, "frac_of_peak": gbs / peak,
           "bf16_equivalent_gbs": (kept * wl.group_bytes + steps * (L - 1) * wl.pred_bytes) / (ms * 1e-3) / 1e9,
           "weights_gb": L * G * group_bytes_i4 / 1e9, "gpu_launches_per_token": stack.last_launches() / steps,
           "device_status": stack.status()}
    stack.close()
    res["prefill"] = _int4_prompt_timing(wl, fsh, plan, Q, Sc, preds, dev)
    return res


def block_stack_report(dev, peak, steps=24, warm=4, context=1024, int4=False):
    """The paper's generation loop over whole layers at the 7B shape: per layer the MHA block (keys / values of all 32
    heads appended, kept heads attend over `context` cached positions) and the MLP block, each with its predictor,
    selection and merge, and the LM-head groups at the end (32000 x 4096).  One launch per step of the path.
    Bytes: kept FFN groups + kept heads' query / output rows + K/V projections + K/V cache rows read + predictors +
    LM head.  int4: every weight matrix as int4 codes + one bf16 scale per 128 elements (the paper's models are 4-bit);
    activations, caches and predictors stay bf16."""
    from paper_2601_11676_b200 import binding as B
    wl = synth.workload("llama2-7b-decode")
    L, d, G, H, dh, vocab, r_mha = wl.n_layers, wl.d_model, wl.n_groups, 32, 128, 32000, 64
    fsh = B.ffn_shape(d, wl.d_ffn, wl.group_size, B.BF16)

    def qrows(W2d):
        rows = W2d.shape[0]
        q = torch.empty((rows, d // 2), dtype=torch.uint8, device=dev)
        sc = torch.empty((rows, d // 128), dtype=torch.bfloat16, device=dev)
        B.halo_quantize_rows_i4(d, rows, B.BF16, W2d, q, sc)
        torch.cuda.synchronize()
        return q, sc
    max_len = context + warm + steps + 1
    mh = B.mha_shape(d, H, dh, max_len, B.BF16)
    mw = synth.Workload("mha-pred", L, d, H * 8, 8, r_mha, "bf16", (), (), 500, 1, seed=wl.seed + 1)
    blocks = []
    g = torch.Generator(device=dev).manual_seed(5)
    for l in range(L):
        Wq, Wk, Wv, Wo = synth.mha_matrices(wl, l, H, dev)
        Wp = torch.empty((H, 2, dh, d), dtype=torch.bfloat16, device=dev)
        B.halo_pack_mha_weights(mh, Wq, Wo, Wp)
        torch.cuda.synchronize()
        del Wq, Wo
        K = torch.zeros((H, max_len, dh), dtype=torch.bfloat16, device=dev)
        V = torch.zeros((H, max_len, dh), dtype=torch.bfloat16, device=dev)
        K[:, :context] = torch.randn((H, context, dh), generator=g, device=dev).to(torch.bfloat16)
        V[:, :context] = torch.randn((H, context, dh), generator=g, device=dev).to(torch.bfloat16)
        blk = dict(W_ffn=synth.packed_layer(wl, l, dev), W_mha=Wp, Wk=Wk, Wv=Wv, K=K, V=V)
        if int4:
            blk["W_ffn"], blk["S_ffn"] = qrows(blk["W_ffn"].view(-1, d))
            blk["W_mha"], blk["S_mha"] = qrows(Wp.view(-1, d))
            blk["Wk"], blk["Sk"] = qrows(Wk)
            blk["Wv"], blk["Sv"] = qrows(Wv)
            del Wp, Wk, Wv
        if l > 0:
            blk["W1_ffn"], blk["W2_ffn"] = synth.predictor(wl, l, dev)
            blk["W1_mha"], blk["W2_mha"] = synth.predictor(mw, l, dev)
        blocks.append(blk)
    gc = torch.Generator(device="cpu").manual_seed(17)
    W_lm = (torch.randn((vocab, d), generator=gc) / 64).to(torch.bfloat16).to(dev)
    plan_f = B.Plan(G, wl.loss_rate, wl.share_weight, B.SEL_TOPK, B.k_of(wl), 0.0, wl.seed)
    plan_a = B.Plan(H, wl.loss_rate, wl.share_weight, B.SEL_TOPK, H // 2, 0.0, wl.seed + 1)
    S_lm = None
    if int4:
        W_lm, S_lm = qrows(W_lm)
    stack = B.BlockStack(fsh, mh, B.lm_shape(d, vocab, 256, B.BF16),
                         B.pred_shape(d, wl.pred_rank, G, B.BF16), B.pred_shape(d, r_mha, H, B.BF16), plan_f, plan_a,
                         blocks, W_lm, S_lm)
    total = warm + steps
    h0 = torch.stack([synth.stream_input(wl, 500 + s, dev)[0] for s in range(total)])
    logits = torch.empty((total, vocab), dtype=torch.float32, device=dev)
    nk_a = torch.zeros((total, L), dtype=torch.int32, device=dev)
    nk_f = torch.zeros((total, L), dtype=torch.int32, device=dev)
    taps = B.BlockTaps(B.Taps(None, None, None, None, None, nk_a.data_ptr(), None),
                       B.Taps(None, None, None, None, None, nk_f.data_ptr(), None))
    stack.decode(h0, total, context, 0, logits, None, taps)          # records the kept sets; also the warm-up
    torch.cuda.synchronize()
    ts = []
    for _ in range(3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        stack.decode(h0[warm:], steps, context + warm, warm, logits[warm:])
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ms = sorted(ts)[1]
    kept_f, kept_a = int(nk_f[warm:].sum().item()), int(nk_a[warm:].sum().item())
    pos_sum = sum(context + warm + s + 1 for s in range(steps))
    wb = (0.5 + 2.0 / 128.0) if int4 else 2.0                    # bytes per weight element
    byts = (kept_f * wl.group_bytes / 2 * wb + steps * (L - 1) * (wl.pred_bytes + (d * r_mha + r_mha * H) * 2)
            + steps * L * 2 * d * d * wb + kept_a * 2 * dh * d * wb
            + sum(int(nk_a[warm + s].sum().item()) * 2 * (context + warm + s + 1) * dh * 2 for s in range(steps))
            + steps * vocab * d * wb)
    gbs = byts / (ms * 1e-3) / 1e9
    res = {"shape": "32 layers x (32 heads of 128 + 86 FFN groups of 128), d 4096, %d cached positions, LM head 32000%s"
                    % (context, ", int4 weights" if int4 else ""),
           "steps": steps, "tokens_per_s": steps / (ms * 1e-3), "ms_per_token": ms / steps,
           "kept_fraction_ffn": kept_f / float(steps * L * G), "kept_fraction_heads": kept_a / float(steps * L * H),
           "algorithmic_gb_per_token": byts / steps / 1e9, "achieved_gbs": gbs, "frac_of_peak": gbs / peak,
           "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS, "gpu_launches_per_token": stack.last_launches() / steps,
           "device_status": stack.status()}
    stack.close()
    return res


def decode_brief(name, dev, peak, steps=64, warm=4):
    """tokens/s and algorithmic GB/s of another decode workload (one persistent launch over `steps` tokens)."""
    from paper_2601_11676_b200 import binding as B
    wl = synth.workload(name)
    stack, Wp, preds, plan, ffn = build_stack(wl, dev)
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
    gbs = byts / (ms * 1e-3) / 1e9
    res = {"workload": name, "steps": steps, "tokens_per_s": steps / (ms * 1e-3), "ms_per_step": ms / steps,
           "kept_fraction": kept / float(steps * L * G), "achieved_gbs": gbs, "frac_of_peak": gbs / peak,
           "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS, "gpu_launches": stack.last_launches(),
           "device_status": stack.status()}
    stack.close()
    return res


def _int4_prompt_timing(wl, fsh, plan, Q, Sc, preds, dev, n_tok=512, prompts=8, warm=3):
    """512-token prompts through the int4 stack: per block the kept groups are turned back into bf16 in a scratch
    block (on the side stream, under the previous block's FFN) and the tensor-core FFN reads those.  FLOPs as for the
    bf16 prompt."""
    from paper_2601_11676_b200 import binding as B
    L, G, d = wl.n_layers, wl.n_groups, wl.d_model
    stack = B.Stack(fsh, B.pred_shape(d, wl.pred_rank, G, B.BF16), n_tok, plan, Q, [p[0] for p in preds],
                    [p[1] for p in preds], i4_scales=Sc)
    pw = synth.workload(wl.name, n_tok=n_tok)
    total = warm + prompts
    h0 = torch.stack([synth.stream_input(pw, 1000 + s, dev) for s in range(total)])
    h_out = torch.empty_like(h0)
    nk_rec = torch.zeros((total, L), dtype=torch.int32, device=dev)
    stack.decode(h0, total, 0, h_out, B.Taps(None, None, None, None, None, nk_rec.data_ptr(), None))
    torch.cuda.synchronize()
    reps = []
    for _ in range(3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        stack.decode(h0[warm:], prompts, warm, h_out[warm:])
        b.record()
        torch.cuda.synchronize()
        reps.append(a.elapsed_time(b))
    ms = sorted(reps)[1]
    kept = int(nk_rec[warm:].sum().item())
    flops = 6.0 * n_tok * kept * wl.group_size * d + prompts * (L - 1) * 2.0 * n_tok * (d * wl.pred_rank + wl.pred_rank * G)
    out = {"prompt_tokens": n_tok, "prompts_timed": prompts, "ms_per_prompt": ms / prompts,
           "ms_per_prompt_runs": [r / prompts for r in reps], "tflops": flops / (ms * 1e-3) / 1e12,
           "gpu_launches": int(stack.last_launches()), "device_status": stack.status()}
    stack.close()
    return out


def prefill_report(wl, Wp, preds, plan, ffn, dev, n_tok=512, prompts=16, warm=3):
    """The same stack run on a 512-token prompt (tensor-core form of the masked FFN), weights shared with the decode
    run: milliseconds per prompt and achieved bf16 TFLOP/s over the kept groups' FLOPs."""
    from paper_2601_11676_b200 import binding as B
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peaks = json.load(open(pk)) if os.path.exists(pk) else {}
    burst, sustained = float(peaks.get("bf16_tflops", 1590.0)), float(peaks.get("bf16_tflops_sustained", 1400.0))
    L, G, d = wl.n_layers, wl.n_groups, wl.d_model
    pred = B.pred_shape(d, wl.pred_rank, G, B.BF16)
    stack = B.Stack(ffn, pred, n_tok, plan, Wp, [p[0] for p in preds], [p[1] for p in preds])
    pw = synth.workload(wl.name, n_tok=n_tok)
    total = warm + prompts
    h0 = torch.stack([synth.stream_input(pw, 1000 + s, dev) for s in range(total)])
    h_out = torch.empty_like(h0)
    nk_rec = torch.zeros((total, L), dtype=torch.int32, device=dev)
    taps = B.Taps(None, None, None, None, None, nk_rec.data_ptr(), None)
    stack.decode(h0, total, 0, h_out, taps)     # records the kept sets; also the warm-up
    torch.cuda.synchronize()
    status = stack.status()
    reps = []
    for _ in range(3):      # the same prompts three times; the median run is reported, all three are listed
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        stack.decode(h0[warm:], prompts, warm, h_out[warm:])
        b.record()
        torch.cuda.synchronize()
        reps.append(a.elapsed_time(b))
    ms = sorted(reps)[1]
    launches = stack.last_launches()
    # the same prompts through the one-launch-per-prompt kernel (not the default: see the header), for the record
    stack.set_mode(B.STACK_PROMPT_ONE_LAUNCH)
    stack.decode(h0[:warm], warm, 0, h_out[:warm])
    one = []
    for _ in range(3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        stack.decode(h0[warm:], prompts, warm, h_out[warm:])
        b.record()
        torch.cuda.synchronize()
        one.append(a.elapsed_time(b))
    one_launches = stack.last_launches()
    status |= stack.status()
    kept = int(nk_rec[warm:].sum().item())
    flops = 6.0 * n_tok * kept * wl.group_size * d + prompts * (L - 1) * 2.0 * n_tok * (d * wl.pred_rank + wl.pred_rank * G)
    tflops = flops / (ms * 1e-3) / 1e12
    stack.close()
    return {"workload": wl.name.replace("decode", "prefill"), "prompt_tokens": n_tok, "prompts_timed": prompts,
            "ms_per_prompt": ms / prompts, "ms_per_prompt_runs": [r / prompts for r in reps], "tokens_per_s": prompts * n_tok / (ms * 1e-3), "tflops": tflops,
            "bound": "tensor", "peak_burst_tflops": burst, "frac_of_burst_peak": tflops / burst,
            "peak_sustained_tflops": sustained, "frac_of_sustained_peak": tflops / sustained,
            "kept_fraction": kept / float(prompts * L * G), "gpu_launches": int(launches), "device_status": status,
            "one_launch_per_prompt": {"ms_per_prompt": sorted(one)[1] / prompts, "gpu_launches": int(one_launches),
                                      "tflops": flops / (sorted(one)[1] * 1e-3) / 1e12}}


# ----------------------------------------------------------------------------------------------------------------
# the oracle arm (CPU, fp64): reported baseline
# ----------------------------------------------------------------------------------------------------------------

def _oracle_layer_inputs(wl, layer):
    hb = synth.host_bits
    Wp = hb(synth.packed_layer(wl, layer, "cpu"))
    w1, w2 = (hb(t) for t in synth.predictor(wl, layer, "cpu"))
    feat = hb(synth.activation(wl, 2 * layer, "cpu"))
    x = hb(synth.activation(wl, 2 * layer + 1, "cpu"))
    return Wp, w1, w2, feat, x


def cpu_baseline(wl, budget_s=15.0):
    """Times the oracle as it stands on a bounded sample: whole blocks (predict, select, kept-group FFN, merge) of
    one token, as many as fit the time budget; tokens/s is that block rate divided by the blocks per token."""
    from oracle import halo_ref as R
    cores = os.cpu_count() or 1
    R.set_threads(cores)
    R.lib()
    done, spent = 0, 0.0
    inputs = _oracle_layer_inputs(wl, 1)  # same shapes for every block; generated outside the timed part
    while spent < budget_s and done < 64 * wl.n_layers:
        Wp, w1, w2, feat, x = inputs
        t0 = time.perf_counter()
        R.layer(Wp, w1, w2, feat, x, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed,
                done // wl.n_layers, 1 + done % max(wl.n_layers - 1, 1))
        spent += time.perf_counter() - t0
        done += 1
    value = (done / wl.n_layers) / spent
    return {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"{done} blocks ({done / wl.n_layers:.2f} tokens of {wl.n_layers} blocks, {wl.name}), "
                      f"{spent:.1f} s of CPU time; tokens/s = tokens / time"}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    from oracle import halo_ref as R
    wl = synth.workload(args.workload, keep_permille=args.keep_permille)
    cores = os.cpu_count() or 1
    R.set_threads(cores)
    K, W = args.steps, args.warmup
    Wp, w1, w2, feat, x = _oracle_layer_inputs(wl, 1)
    G = wl.n_groups
    scores = R.predict(w1, w2, feat)

    def one_step(step, n_groups_sample):
        # a bounded sample of one block: predictor, selection, and the FFN of the first n kept groups
        s = R.predict(w1, w2, feat)
        sel = R.select(s, wl.loss_rate, wl.share_weight, R.SEL_TOPK, R.k_of(wl), 0.0, wl.seed, step, 1)
        keep = sel["keep_list"][: min(sel["n_keep"], n_groups_sample)]
        P = R.group_ffn(Wp, x, keep, sel["dev_of_group"], wl.n_dev)
        R.merge(P)
        return len(keep), sel["n_keep"]

    # size the per-step sample so that W + K steps end within about two minutes
    t0 = time.perf_counter()
    g_done, _ = one_step(0, 4)
    per_group = max((time.perf_counter() - t0) / max(g_done, 1), 1e-6)
    budget_per_step = 120.0 / max(K + W, 1)
    n_sample = int(max(1, min(G, budget_per_step / per_group)))
    for s in range(W):
        one_step(s, n_sample)
    groups, kept_total = 0, 0
    t0 = time.perf_counter()
    for s in range(K):
        g, nk = one_step(W + s, n_sample)
        groups += g
        kept_total += nk
    dt = time.perf_counter() - t0
    # tokens/s: a token costs (average kept groups per block) x (blocks) group evaluations
    groups_per_token = (kept_total / K) * wl.n_layers
    value = (groups / groups_per_token) / dt
    sample = (f"each step = predictor + selection + FFN of {n_sample} kept groups of one block ({wl.name}); "
              f"tokens/s extrapolated by groups per token ({groups_per_token:.0f})")
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": dt * 1e3 / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, 1 if world <= 1 else world),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="halo", choices=["halo", "reference"])
    ap.add_argument("--workload", default="llama2-7b-decode", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--keep-permille", type=int, default=500)
    ap.add_argument("--layers", type=int, default=0, help="use only this many blocks (small profiling cases)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true", help="skip the 512-token prompt report")
    ap.add_argument("--no-extra", action="store_true", help="skip the brief runs of the other decode workloads")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="halo_set_option before anything is created (tuning sweeps), e.g. --option cross_stages=4")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "halo" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        res = run_reference(args, rank, world)
        if res is not None:
            print(json.dumps(res), flush=True)
        return 0

    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    try:
        res = run_halo(args, rank, world, local_rank)
        if res is not None:
            print(json.dumps(res), flush=True)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
