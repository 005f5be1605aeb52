#!/usr/bin/env python
"""Benchmark of the EfQAT layer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--frac R]

Headline workload: the two largest shapes of the GEMM-shape sweep, M = 16384 tokens with
(K, N) = (8192, 8192) and (4096, 16384), bf16 activations, W8A8, per-layer channel selection,
5 % of the channels unfrozen.  One step = one pass of the whole path over one batch:
importance + Top-K selection for both layers, then for each layer the fake-quantised forward
and the partial backward (dX, dS_x, dZ_x, db, and dW / dS_w of the selected channels only)
with the fused SGD-momentum update of the unfrozen rows.

The printed JSON line reports the step throughput in algorithmic TFLOP/s
(2MNK forward + 2MNK(1 + k/N) backward), the backward-only sweep over the unfrozen
fractions with its speed-up over the library's own full-QAT backward, the tensor-core
roofline of the dominant GEMM kernel and of each GEMM kind, the oracle's CPU time on a
bounded sample of the same workload and the end-to-end number with host buffers.  The
BERT-base-shaped linears at M = 4096 are measured the same way under the key "bert_base".
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2411_11038_b200 import inputs as I  # noqa: E402
from paper_2411_11038_b200.clocks import ClockSampler, physical_gpu_index  # noqa: E402

FRACS = (0.0, 0.05, 0.25, 1.0)
METRIC = ("fq-linear backward TFLOP/s & speedup vs full-QAT bwd per unfrozen %; roofline frac "
          "[value: TFLOP/s of one step of the whole path = select + fwd + partial bwd + fused sparse SGD; "
          "backward-only ms, TFLOP/s and speedups per unfrozen % under 'bwd']")
WORKLOAD_NAME = ("configs[4]: GEMM-shape sweep, M=16384 tokens, (K,N) = (8192,8192) and (4096,16384), "
                 "bf16 activations, W8A8, CWPL, selection recomputed every step")
L2_FLUSH_BYTES = 256 << 20
SGD_LR = 1e-9
# ncu capture of the dominant kernel on the first layer of the headline workload: the file states
# the DRAM bytes per launch and the hash of the kernel sources it was taken from.
TRAFFIC_FILE = os.path.join("profiles", "gemm_kernel_dx_cfg5_8192x8192.txt")
KERNEL_SOURCES = ("gemm.cu", "ptx.cuh", "common.cuh")
# bounded sample of the headline workload for the oracle: leading tokens and output channels
REF_SAMPLE = dict(tokens=256, channels=1024)
CPU_SAMPLE = dict(tokens=512, channels=2048)


def headline_cases():
    c = I.config5()
    return [c[3], c[2]]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(tflops=float(d["bf16_tflops"]), tflops_sustained=float(d.get("bf16_tflops_sustained", 0)),
                    hbm_gbs=float(d["hbm_gbs"]), source="measured")
    return dict(tflops=1590.0, tflops_sustained=1400.0, hbm_gbs=6650.0, source="fallback")


def kernel_source_hash():
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2411_11038_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic():
    """DRAM bytes per launch of the dominant kernel from the kept ncu summary; None once the
    kernel sources differ from those the capture was taken from."""
    path = os.path.join(ROOT, TRAFFIC_FILE)
    if not os.path.exists(path):
        return None, "no capture kept"
    txt = open(path).read()
    m = re.search(r"^dram_bytes_per_launch:\s*([0-9.eE+]+)", txt, re.M)
    h = re.search(r"^kernel_source_hash:\s*([0-9a-f]+)", txt, re.M)
    if not m or not h:
        return None, "capture summary has no traffic line"
    if h.group(1) != kernel_source_hash():
        return None, "kernel changed since the capture"
    return float(m.group(1)), TRAFFIC_FILE


# ----------------------------------------------------------------------------------------
class Workload:
    """Device-resident tensors and pre-marshalled calls of a list of layers."""

    def __init__(self, ctx, device, cases, fracs, e2e_frac=None, keep_sample=None):
        from paper_2411_11038_b200 import binding as B
        self.B, self.ctx, self.device = B, ctx, device
        self.cases = cases
        self.layers = []
        self.samples = []
        for c in self.cases:
            T = I.make_tensors(c)
            D = {k: v.to(device) for k, v in T.items()}
            D["s_w"] = B.init_weight_scales(ctx, D["W"], c.w_bits)
            D["s_x"], D["z_x"] = B.init_act_qparams(ctx, D["X"], c.x_bits, c.x_symmetric)
            if e2e_frac is not None:
                D["host_X"] = T["X"].pin_memory()
                D["host_dY"] = T["dY"].pin_memory()
                k_e = max(B.ratio_to_k(e2e_frac, c.N), 1)
                D["host_dW"] = torch.empty((k_e, c.K), dtype=torch.float32).pin_memory()
                D["host_small"] = torch.empty(2 * c.N + 2, dtype=torch.float32).pin_memory()
            if keep_sample:
                self.samples.append(sample_of(c, T, **keep_sample))
            plan = B.LayerPlan(ctx, c.M, c.N, c.K, c.act_dtype, c.w_bits, c.x_bits, c.x_symmetric, c.N, device)
            # fused sparse SGD-momentum of Algorithm 1 on the unfrozen rows (momentum and weight decay
            # of Section 4).  The learning rate is scaled down: the synthetic dY has unit variance,
            # a real loss gradient is orders of magnitude smaller, and the weights must stay put
            # over hundreds of timed steps; the arithmetic and the traffic are those of any rate.
            D["mom"] = torch.zeros_like(D["W"])
            D["sgd"] = B.make_sgd(SGD_LR, 0.9, 1e-4, D["W"], D["mom"])
            self.layers.append((c, D, plan))
            del T
        self.sel = {}
        for f in fracs:
            ks = [B.ratio_to_k(f, c.N) for c in self.cases]
            plan = B.SelectPlan(ctx, B.CWPL, [D["W"] for _, D, _ in self.layers], ks)
            offs = np.concatenate([[0], np.cumsum(ks)]).astype(int)
            views = [plan.idx[offs[i]:offs[i + 1]] if ks[i] else None for i in range(len(ks))]
            self.sel[f] = (plan, ks, views)
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
        self.copy_stream = None
        self.side_stream = None

    def flops(self, frac, fwd=True, bwd=True):
        tot = 0.0
        _, ks, _ = self.sel[frac]
        for (c, _, _), k in zip(self.layers, ks):
            g = 2.0 * c.M * c.N * c.K
            if fwd:
                tot += g
            if bwd:
                tot += g + 2.0 * c.M * k * c.K
        return tot

    def gemm_flops(self, frac):
        """Algorithmic FLOPs of the three GEMM kinds per step: fwd, dX, dW."""
        _, ks, _ = self.sel[frac]
        full = sum(2.0 * c.M * c.N * c.K for c, _, _ in self.layers)
        dw = sum(2.0 * c.M * k * c.K for (c, _, _), k in zip(self.layers, ks))
        return [full, full, dw]

    def select(self, frac):
        self.sel[frac][0].run()

    def backward(self, frac):
        _, ks, views = self.sel[frac]
        for (c, D, plan), k, idx in zip(self.layers, ks, views):
            plan.bwd(D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx, k, want_db=True, sgd=D["sgd"])

    def step(self, frac):
        """Selection only reads the weights and only the backward needs its result, so it runs
        on a second stream beside the forward launches and is joined before the backward."""
        cur = torch.cuda.current_stream()
        if self.side_stream is None:
            self.side_stream = torch.cuda.Stream()
        self.side_stream.wait_stream(cur)
        with torch.cuda.stream(self.side_stream):
            self.select(frac)
            joined = self.side_stream.record_event()
        for c, D, plan in self.layers:
            plan.fwd(D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], D["bias"])
        cur.wait_event(joined)
        self.backward(frac)

    def step_e2e(self, frac):
        """Same step with this step's activations coming from pinned host memory and the
        parameter gradients going back to it.  The host-to-device copies run on a second
        stream in the order the layers need them, so a layer's kernels start as soon as its
        own inputs have landed; everything is ordered back into the timed stream."""
        _, ks, views = self.sel[frac]
        cur = torch.cuda.current_stream()
        if self.copy_stream is None:
            self.copy_stream = torch.cuda.Stream()
        self.copy_stream.wait_stream(cur)          # the previous step has finished with the buffers
        ev_x, ev_dy = [], []
        with torch.cuda.stream(self.copy_stream):
            for c, D, plan in self.layers:
                D["X"].copy_(D["host_X"], non_blocking=True)
                ev_x.append(self.copy_stream.record_event())
            for c, D, plan in self.layers:
                D["dY"].copy_(D["host_dY"], non_blocking=True)
                ev_dy.append(self.copy_stream.record_event())
        self.select(frac)
        for (c, D, plan), e in zip(self.layers, ev_x):
            cur.wait_event(e)
            plan.fwd(D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], D["bias"])
        for (c, D, plan), k, idx, e in zip(self.layers, ks, views, ev_dy):
            cur.wait_event(e)
            plan.bwd(D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx, k, want_db=True, sgd=D["sgd"])
        for (c, D, plan), k in zip(self.layers, ks):
            if k:
                D["host_dW"][:k].copy_(plan.dW_sel[:k], non_blocking=True)
                D["host_small"][:k].copy_(plan.dS_w_sel[:k], non_blocking=True)
            D["host_small"][c.N:2 * c.N].copy_(plan.db, non_blocking=True)
            D["host_small"][2 * c.N:2 * c.N + 1].copy_(plan.dS_x, non_blocking=True)
            D["host_small"][2 * c.N + 1:].copy_(plan.dZ_x, non_blocking=True)

    def e2e_bytes(self, frac):
        _, ks, _ = self.sel[frac]
        bi = sum(D["host_X"].numel() * 2 + D["host_dY"].numel() * 2 for _, D, _ in self.layers)
        bo = sum(k * c.K * 4 + k * 4 + c.N * 4 + 8 for (c, _, _), k in zip(self.layers, ks))
        return bi, bo


def timed(fn, steps, warmup, flush, sync_all=None, after_warmup=None):
    """Sum of per-step device durations (ms); L2 is flushed, untimed, before every step."""
    for _ in range(warmup):
        flush.zero_()
        fn()
    if sync_all:
        sync_all()
    torch.cuda.synchronize()
    if after_warmup:
        after_warmup()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for i in range(steps):
        flush.zero_()
        starts[i].record()
        fn()
        ends[i].record()
    torch.cuda.synchronize()
    if sync_all:
        sync_all()
    return sum(s.elapsed_time(e) for s, e in zip(starts, ends))


# ----------------------------------------------------------------------------------------
# the oracle on the host cores
# ----------------------------------------------------------------------------------------
def sample_of(case, T, tokens, channels):
    """Leading `tokens` rows and `channels` output channels of a layer's tensors (CPU, fp64)."""
    t, n = min(tokens, case.M), min(channels, case.N)
    return dict(name=case.name, K=case.K, tokens=t, channels=n, w_bits=case.w_bits, x_bits=case.x_bits,
                x_symmetric=case.x_symmetric,
                X=I.as_f64(T["X"][:t]), W=I.as_f64(T["W"][:n]), dY=I.as_f64(T["dY"][:t, :n]),
                bias=I.as_f64(T["bias"][:n]))


def oracle_sample_seconds(samples, frac):
    """One pass of the oracle, as it stands, over the sampled layers: MinMax scales, selection,
    forward, EfQAT backward, SGD on the unfrozen rows.  Returns (seconds, algorithmic FLOPs)."""
    from oracle import efqat_oracle as O
    flops = 0.0
    t0 = time.perf_counter()
    for s in samples:
        X, W, dY, b = s["X"], s["W"], s["dY"], s["bias"]
        s_w = O.init_minmax_w(W, s["w_bits"])
        s_x, z_x = O.init_minmax_x(X, s["x_bits"], s["x_symmetric"])
        k = O.ratio_to_k(frac, s["channels"])
        idx = O.select_cwpl([W], [k])[0]
        O.forward(X, W, s_w, s_x, z_x, b, s["w_bits"], s["x_bits"], s["x_symmetric"])
        g = O.backward_efqat(dY, X, W, s_w, s_x, z_x, idx, s["w_bits"], s["x_bits"], s["x_symmetric"])
        O.sgd_rows(W, np.zeros_like(W), g["dW_sel"], idx, SGD_LR, 0.9, 1e-4)
        flops += 2.0 * s["tokens"] * s["channels"] * s["K"] * 2 + 2.0 * s["tokens"] * k * s["K"]
    return time.perf_counter() - t0, flops


def sample_text(samples, frac):
    per = ", ".join(f"{s['name']} [{s['tokens']} tokens x {s['channels']} channels x K={s['K']}]" for s in samples)
    return (f"oracle (fp64 numpy: MinMax scales, selection, forward, EfQAT backward, SGD rows) on the leading tokens "
            f"and output channels of each layer of the workload: {per}; {int(frac * 100)}% unfrozen")


def workload_config(frac, world):
    return {"workload": WORKLOAD_NAME, "unfrozen": frac,
            "l2": "inputs exceed L2; a 256 MiB buffer is also written between timed steps",
            "arithmetic": "forward: 8-bit codes on the integer tensor cores, int32 accumulate; "
                          "backward contractions: bf16 operands, fp32 accumulate",
            "optimizer": "fused SGD-momentum on the unfrozen rows (momentum 0.9, weight decay 1e-4, "
                         f"lr {SGD_LR:g} scaled for unit-variance synthetic dY)",
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    frac = args.frac
    samples = []
    for c in headline_cases():
        T = I.make_tensors(c)
        samples.append(sample_of(c, T, **REF_SAMPLE))
        del T
    for _ in range(min(args.warmup, 2)):
        oracle_sample_seconds(samples, frac)
    tot, fl = 0.0, 0.0
    for _ in range(args.steps):
        s, f = oracle_sample_seconds(samples, frac)
        tot += s
        fl += f
    val = fl / tot / 1e12
    cores = os.cpu_count()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(frac, world),
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": sample_text(samples, frac)},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------------------
def measure(wl, ctx, frac, steps, warmup, peaks, sync_all, max_over_ranks, world, sampler=None, extras=True):
    """Headline pass, per-kernel pass and backward sweep of one workload."""
    B = wl.B
    mark = {}

    def start_counting():
        mark["launches"] = ctx.launch_count()
        if sampler is not None:
            sampler.start()

    total_ms = timed(lambda: wl.step(frac), steps, warmup, wl.flush, sync_all, start_counting)
    if sampler is not None:
        sampler.stop_flag = True
    launches = ctx.launch_count() - mark["launches"]
    if sampler is not None:
        sampler.join(timeout=2)
    ms_per_step = max_over_ranks(total_ms) / steps
    value = world * wl.flops(frac) / (ms_per_step * 1e-3) / 1e12

    # The same K steps once more with a pair of CUDA events around every GEMM launch.  The events
    # serialise launches that otherwise overlap their set-up with the previous kernel's tail, so
    # they stay out of the headline pass above.
    prof_ms = timed(lambda: wl.step(frac), steps, 3, wl.flush, sync_all, lambda: ctx.profile_enable(True))
    kinds = [ctx.profile_read(i) for i in range(3)]      # (total ms, launches) of the K profiled steps
    ctx.profile_enable(False)
    gf = wl.gemm_flops(frac)
    names = ["gemm_kernel<fwd epilogue>", "gemm_kernel<dX epilogue>", "gemm_kernel<dW partial epilogue>"]
    # forward: 8-bit integer tensor-core operations, nominal rate twice the bf16 one
    kind_peak = [2.0 * peaks["tflops"], peaks["tflops"], peaks["tflops"]]
    per_kind = {}
    for i, n in enumerate(names):
        ms_i, n_i = kinds[i]
        ach = (gf[i] * steps) / (ms_i * 1e-3) / 1e12 if n_i and ms_i > 0 else None
        per_kind[n] = {"ms_per_step": ms_i / steps, "launches_per_step": n_i / steps,
                       "achieved": ach, "unit": "Top/s (int8)" if i == 0 else "TFLOP/s (bf16)",
                       "peak": kind_peak[i], "frac": (ach / kind_peak[i]) if ach else None}
    dom = max(range(3), key=lambda i: kinds[i][0])
    dom_ms, dom_n = kinds[dom]
    achieved = per_kind[names[dom]]["achieved"]
    traffic, traffic_src = recorded_traffic() if wl.cases[0].name.startswith("cfg5") else (None, "not captured")
    roofline = {"bound": "tensor", "kernel": names[dom], "achieved": achieved, "peak": kind_peak[dom],
                "unit": "TFLOP/s", "frac": (achieved / kind_peak[dom]) if achieved else None,
                "traffic": traffic, "traffic_source": traffic_src,
                "peak_source": f"{peaks['source']} burst bf16 GEMM" + (" x 2 (int8 nominal ratio)" if dom == 0 else ""),
                "launches": dom_n, "avg_launch_ms": dom_ms / max(dom_n, 1),
                "timed_in": "second pass of the same K steps with per-kernel CUDA events",
                "ms_per_step_with_kernel_events": max_over_ranks(prof_ms) / steps,
                "per_kind": per_kind}

    bwd_report, sel_ms = {}, None
    if extras:
        sweep_steps = max(20, steps // 4)
        bwd = {}
        for f in sorted(wl.sel):
            wl.select(f)
            bwd[f] = max_over_ranks(timed(lambda: wl.backward(f), sweep_steps, 5, wl.flush, sync_all) / sweep_steps)
        for f in sorted(wl.sel):
            fl = wl.flops(f, fwd=False)
            tf = fl / (bwd[f] * 1e-3) / 1e12
            bwd_report[f"{int(round(f * 100))}%"] = {
                "ms": bwd[f], "tflops": tf, "frac_of_sustained_peak": tf / peaks["tflops_sustained"],
                "speedup_vs_full_qat": bwd[1.0] / bwd[f], "ideal_speedup": 2.0 / (1.0 + f)}
        sel_ms = max_over_ranks(timed(lambda: wl.select(frac), sweep_steps, 5, wl.flush, sync_all) / sweep_steps)
        roofline["whole_backward"] = {
            "tflops": bwd_report[f"{int(round(frac * 100))}%"]["tflops"], "peak": peaks["tflops_sustained"],
            "frac": bwd_report[f"{int(round(frac * 100))}%"]["frac_of_sustained_peak"],
            "peak_source": f"{peaks['source']} sustained bf16 GEMM",
            "what": "prepare + dX GEMM + partial dW GEMM + finalize (with SGD) on the algorithmic FLOPs 2MNK(1+k/N)"}
    return dict(ms_per_step=ms_per_step, value=value, launches=int(launches), roofline=roofline, bwd=bwd_report,
                select_ms=sel_ms)


def measure_network(ctx, dev, sync_all, max_over_ranks):
    """The BERT-large-shaped stack (configs[3]): 144 quantized linears at M = 9216 tokens, W4A8,
    chained on one stream through efqat_network_fwd / _bwd with a weight-operand cache per layer,
    network-wide (CWPN) and layer-wise (LWPN) selection, and the freezing frequency f of
    Section 3.2.  Reported: ms per network backward per unfrozen ratio, the selection cost and
    its share when amortised over f samples, cached against uncached calls."""
    import math
    from paper_2411_11038_b200 import binding as B
    from paper_2411_11038_b200 import network as NW
    cases = I.config4()
    batch = 24                                       # sequences of 384 tokens per step
    pools = {}

    def pool(width, count, seed):
        if width not in pools:
            g = torch.Generator().manual_seed(seed)
            pools[width] = [torch.randn((cases[0].M, width), generator=g).to(torch.bfloat16).to(dev)
                            for _ in range(count)]
        return pools[width]

    p1, p4 = pool(1024, 8, 4901), pool(4096, 4, 4902)     # 151 MB each: rotating through them defeats L2
    states = []
    for i, c in enumerate(cases):
        g = torch.Generator().manual_seed(c.seed)
        W = (torch.randn((c.N, c.K), generator=g) * math.sqrt(2.0 / c.K)).to(dev)
        X = (p1 if c.K == 1024 else p4)[i % (8 if c.K == 1024 else 4)]
        dY = (p1 if c.N == 1024 else p4)[(i + 3) % (8 if c.N == 1024 else 4)]
        states.append(NW.LayerState(c, W, X, dY, None))
    total = sum(c.N for c in cases)
    net = NW.EfqatNetwork(ctx, states, B.CWPN, B.ratio_to_k(0.1, total), f_samples=batch, batch_samples=batch,
                          use_cache=True, sgd=(SGD_LR, 0.9, 1e-4), adam=dict(lr=1e-6))
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    gemm = sum(2.0 * c.M * c.N * c.K for c in cases)

    def t(fn, steps=10, warm=3):
        return max_over_ranks(timed(fn, steps, warm, flush, sync_all) / steps)

    out = {"workload": "configs[3]: BERT-large-shaped stack, 24 blocks x (4 x 1024->1024, 1024->4096, 4096->1024) = "
                       "144 layers, M=9216 tokens, W4A8, bf16 activations, inputs rotate through pools larger than L2",
           "layers": len(cases), "channels": total, "samples_per_step": batch}
    rows = {}
    for mode, name, ratios in ((B.CWPN, "CWPN", (0.0, 0.05, 0.10, 0.25, 1.0)), (B.LWPN, "LWPN", (0.05, 0.10, 0.25))):
        for r in ratios:
            budget = B.ratio_to_k(r, total) if mode == B.CWPN else int(r * len(cases))
            net.use_selection(mode, budget)
            net.reselect()
            ks = net.counts()
            fl = sum(2.0 * c.M * c.K * (c.N + k) for c, k in zip(cases, ks))
            ms = t(net.backward)
            rows[f"{name} {int(round(r * 100))}%"] = {
                "bwd_ms": ms, "tflops": fl / (ms * 1e-3) / 1e12, "unfrozen_channels": int(sum(ks)),
                "layers_with_unfrozen_channels": int(sum(1 for k in ks if k))}
    full = rows["CWPN 100%"]["bwd_ms"]
    for v in rows.values():
        v["speedup_vs_full_qat"] = full / v["bwd_ms"]
    out["backward"] = rows
    # the schedule's own costs at the 10 % network-wide budget
    net.use_selection(B.CWPN, B.ratio_to_k(0.1, total))
    sel_ms = t(net.reselect)                              # importance + ranking + counts to the host
    net.reselect()
    fwd_ms = t(net.forward)
    tail_ms = t(net.optimizer_tail)
    bwd_ms = rows["CWPN 10%"]["bwd_ms"]
    unc = NW.EfqatNetwork(ctx, states, B.CWPN, B.ratio_to_k(0.1, total), f_samples=batch, batch_samples=batch,
                          use_cache=False, sgd=(SGD_LR, 0.9, 1e-4), adam=None)
    unc.reselect()
    out["uncached"] = {"fwd_ms": t(unc.forward), "bwd_ms": t(unc.backward)}
    del unc
    out["cached"] = {"fwd_ms": fwd_ms, "bwd_ms": bwd_ms, "adam_and_cache_refresh_ms": tail_ms}
    out["fwd_tops"] = gemm / (fwd_ms * 1e-3) / 1e12
    out["select_ms"] = sel_ms
    out["freezing_frequency"] = {
        str(f): {"selections_per_step": min(1.0, batch / f),
                 "amortised_select_ms_per_step": sel_ms * min(1.0, batch / f),
                 "share_of_backward": sel_ms * min(1.0, batch / f) / (bwd_ms + sel_ms * min(1.0, batch / f))}
        for f in (batch, 4096, 16384)}
    # whole training steps under the real schedule: every step, and f = 4096 samples (171 steps apart)
    for f, steps in ((batch, 24), (4096, 172)):
        net.schedule = NW.FreezeSchedule(f, batch)
        net.train_step()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(steps):
            net.train_step()
        torch.cuda.synchronize()
        out["freezing_frequency"][str(f)]["train_step_ms_wall"] = 1e3 * (time.perf_counter() - t0) / steps
        out["freezing_frequency"][str(f)]["selections_in_run"] = net.schedule.selections
    out["paper_context"] = ("Table 5 (A100, BERT-base, f=4096): CWPN backward 1.36x / 1.33x / 1.23x faster than QAT at "
                            "5 / 10 / 25 %, LWPN 1.49x / 1.48x / 1.44x, 0 % 1.55x")
    return out


def measure_convnet(ctx, dev, sync_all, max_over_ranks, cases, workload, paper_context):
    """A convolutional network's quantized layers through the network calls: forward and backward per
    unfrozen ratio, network-wide (CWPN) and layer-wise (LWPN).  Each layer has its own input and
    output-gradient tensors, so nothing a layer reads is left in L2 by the one before it."""
    import math
    from paper_2411_11038_b200 import binding as B
    from paper_2411_11038_b200 import network as NW
    gen = torch.Generator(device=dev)
    states = []
    for c in cases:
        gen.manual_seed(c.seed)
        wshape = (c.N, c.R, c.S, c.Cin) if c.conv else (c.N, c.K)
        xshape = (c.B, c.H, c.Wd, c.Cin) if c.conv else (c.M, c.K)
        ho = (c.H + 2 * c.pad - c.R) // c.stride + 1
        yshape = (c.B, ho, ho, c.N) if c.conv else (c.M, c.N)
        W = torch.randn(wshape, generator=gen, device=dev) * math.sqrt(2.0 / c.K)
        X = torch.randn(xshape, generator=gen, device=dev).abs().to(torch.bfloat16)
        dY = torch.randn(yshape, generator=gen, device=dev).to(torch.bfloat16)
        states.append(NW.LayerState(c, W, X, dY, None))
    total = sum(c.N for c in cases)
    batch = cases[0].B
    net = NW.EfqatNetwork(ctx, states, B.CWPN, B.ratio_to_k(0.1, total), f_samples=batch, batch_samples=batch,
                          use_cache=True, sgd=(SGD_LR, 0.9, 1e-4), adam=dict(lr=1e-6), share_outputs=False)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def t(fn, steps=8, warm=3):
        return max_over_ranks(timed(fn, steps, warm, flush, sync_all) / steps)

    gemm = sum(2.0 * c.M * c.N * c.K for c in cases)
    out = {"workload": workload, "layers": len(cases), "channels": total, "fwd_gflop": gemm / 1e9}
    rows = {}
    for mode, name, ratios in ((B.CWPN, "CWPN", (0.0, 0.05, 0.10, 0.25, 1.0)), (B.LWPN, "LWPN", (0.05, 0.10, 0.25))):
        for r in ratios:
            budget = B.ratio_to_k(r, total) if mode == B.CWPN else int(r * len(cases))
            net.use_selection(mode, budget)
            net.reselect()
            ks = net.counts()
            fl = sum(2.0 * c.M * c.K * (c.N + k) for c, k in zip(cases, ks))
            ms = t(net.backward)
            rows[f"{name} {int(round(r * 100))}%"] = {
                "bwd_ms": ms, "tflops": fl / (ms * 1e-3) / 1e12, "unfrozen_channels": int(sum(ks)),
                "layers_with_unfrozen_channels": int(sum(1 for k in ks if k))}
    full = rows["CWPN 100%"]["bwd_ms"]
    for v in rows.values():
        v["speedup_vs_full_qat"] = full / v["bwd_ms"]
    out["backward"] = rows
    net.use_selection(B.CWPN, B.ratio_to_k(0.1, total))
    out["select_ms"] = t(net.reselect)
    net.reselect()
    out["fwd_ms"] = t(net.forward)
    out["fwd_tflops"] = gemm / (out["fwd_ms"] * 1e-3) / 1e12
    out["adam_and_cache_refresh_ms"] = t(net.optimizer_tail)
    out["paper_context"] = paper_context
    return out


def measure_resnet50(ctx, dev, sync_all, max_over_ranks, batch=64):
    """Every quantized layer of ResNet-50 (53 convolutions and the classifier) at 224 x 224, batch 64,
    W4A8 (2.8 GB of activations and gradients, one pair per layer)."""
    return measure_convnet(
        ctx, dev, sync_all, max_over_ranks, I.resnet50(batch),
        f"ResNet-50 at 224x224, batch {batch}: 53 convolutions (7x7 stride-2 input layer on 8 stored channels, "
        "bottleneck blocks 3-4-6-3, stride on the 3x3, shortcuts) + classifier, W4A8, NHWC bf16, synthetic |N(0,1)| "
        "activations, one tensor pair per layer",
        "Table 5 (A100, ResNet-50, f=12288): CWPN backward 0.87x / 0.86x / 0.80x of QAT speed at 5 / 10 / 25 % (slower "
        "than QAT), LWPN 1.55x / 1.49x / 1.36x, 0 % 1.56x")


def measure_resnet20(ctx, dev, sync_all, max_over_ranks, batch=128):
    """The CIFAR-10 ResNet-20 (19 convolutions of 16 / 32 / 64 channels and the classifier) at 32 x 32,
    batch 128, W4A8."""
    return measure_convnet(
        ctx, dev, sync_all, max_over_ranks, I.resnet20(batch),
        f"ResNet-20 at 32x32, batch {batch}: 3x3 input layer on 8 stored channels, 3 stages x 3 basic blocks with 16 / 32 "
        "/ 64 channels, parameter-free shortcuts, classifier stored with 16 outputs; W4A8, NHWC bf16, synthetic "
        "|N(0,1)| activations, one tensor pair per layer",
        "Table 5 (A100, ResNet-20, f=16384): CWPN backward 1.09x / 0.88x / 0.62x of QAT speed at 5 / 10 / 25 %, LWPN "
        "1.55x / 1.52x / 1.28x, 0 % 1.67x")


def run_capture(args):
    """Short run for a profiler: the first layer of the headline workload alone, a few steps."""
    from paper_2411_11038_b200 import binding as B
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = B.Context(0)
    wl = Workload(ctx, dev, headline_cases()[:1], (args.frac,))
    for _ in range(3):
        wl.flush.zero_()
        wl.step(args.frac)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    print(json.dumps({"capture": wl.cases[0].name, "kernel_source_hash": kernel_source_hash()}))


def run_ours(args):
    from paper_2411_11038_b200 import binding as B
    from paper_2411_11038_b200.replicas import Replicas, env_ranks
    rank, local, world = env_ranks()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    reps = Replicas(backend="nccl", device=dev)       # replicas only: no data-path collective
    sync_all = reps.barrier
    max_over_ranks = reps.max_over_ranks

    ctx = B.Context(local)
    frac = args.frac
    peaks = load_peaks()
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline and not args.skip_extras
    wl = Workload(ctx, dev, headline_cases(), FRACS if not args.skip_extras else (frac, 1.0), e2e_frac=frac,
                  keep_sample=CPU_SAMPLE if want_cpu else None)

    # ---- headline: K steps of the whole path, device-resident inputs
    sampler = ClockSampler(physical_gpu_index(local))
    all_clock = ClockSampler(physical_gpu_index(local), period_s=0.02)
    all_clock.start()
    head = measure(wl, ctx, frac, args.steps, args.warmup, peaks, sync_all, max_over_ranks, world, sampler,
                   extras=not args.skip_extras)

    # ---- end to end: inputs from pinned host memory, parameter gradients back to it
    e2e_steps = 3 if args.skip_extras else max(10, args.steps // 4)
    e2e_ms = max_over_ranks(timed(lambda: wl.step_e2e(frac), e2e_steps, 3, wl.flush, sync_all) / e2e_steps)
    bi, bo = wl.e2e_bytes(frac)
    e2e_val = world * wl.flops(frac) / (e2e_ms * 1e-3) / 1e12
    status = ctx.device_status()
    samples = wl.samples
    del wl
    torch.cuda.empty_cache()

    # ---- the BERT-base-shaped linears (M = 4096), measured the same way
    bert = None
    if not args.skip_extras:
        wl2 = Workload(ctx, dev, I.config2(), FRACS)
        b = measure(wl2, ctx, frac, max(args.steps, 50), max(args.warmup, 5), peaks, sync_all, max_over_ranks, world)
        bert = {"workload": "configs[1]: BERT-base-shaped linears 768->2304, 768->768, 768->3072, 3072->768 at "
                            "M=4096, bf16 activations, W8A8, CWPL",
                "ms_per_step": b["ms_per_step"], "value": b["value"], "unit": "TFLOP/s", "bwd": b["bwd"],
                "select_ms": b["select_ms"], "roofline": b["roofline"]}
        status = status or ctx.device_status()
        del wl2
        torch.cuda.empty_cache()
    # ---- the 144-layer stack: whole-network backward, weight-operand cache, freezing frequency
    network = None
    if not args.skip_extras and not args.no_network:
        network = measure_network(ctx, dev, sync_all, max_over_ranks)
        status = status or ctx.device_status()
        torch.cuda.empty_cache()
    # ---- ResNet-50, every quantized layer: the convolutional counterpart
    resnet = resnet20 = None
    if not args.skip_extras and not args.no_network:
        resnet = measure_resnet50(ctx, dev, sync_all, max_over_ranks)
        status = status or ctx.device_status()
        torch.cuda.empty_cache()
        resnet20 = measure_resnet20(ctx, dev, sync_all, max_over_ranks)
        status = status or ctx.device_status()
        torch.cuda.empty_cache()
    all_clock.stop_flag = True
    all_clock.join(timeout=2)

    # ---- the oracle on this machine's host cores (rank 0, single GPU only)
    cpu = None
    if want_cpu:
        s, fl = oracle_sample_seconds(samples, frac)
        cpu = {"value": fl / s / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
               "seconds": s, "sample": sample_text(samples, frac)}

    if rank == 0:
        clocks = sampler.summary()
        clocks["whole_run"] = all_clock.summary()
        clocks["time_x_mhz"] = (head["ms_per_step"] * clocks["sm_mhz"]) if clocks["sm_mhz"] else None
        print(json.dumps({
            "metric": METRIC, "value": head["value"], "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(frac, world),
            "clocks": clocks,
            "e2e": {"value": e2e_val, "unit": "TFLOP/s", "ms_per_step": e2e_ms, "h2d_bytes_per_step": bi,
                    "d2h_bytes_per_step": bo},
            "gpu_launches": head["launches"],
            "roofline": head["roofline"],
            "cpu_baseline": cpu,
            "bwd": head["bwd"],
            "select_ms": head["select_ms"],
            "bert_base": bert,
            "network": network,
            "resnet50": resnet,
            "resnet20": resnet20,
            "device_status": status,
            "paper_context": "paper reports 1.44-1.64x backward speed-up on A10/A100 (whole network)",
        }))
    reps.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--frac", type=float, default=0.05, choices=list(FRACS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--skip-extras", action="store_true",
                    help="only the headline timed steps and a 3-step end-to-end leg")
    ap.add_argument("--no-network", action="store_true", help="skip the 144-layer stack and the ResNet-50 stack")
    ap.add_argument("--capture", action="store_true",
                    help="three steps of the first headline layer alone (small run for a profiler)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.capture:
        run_capture(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
