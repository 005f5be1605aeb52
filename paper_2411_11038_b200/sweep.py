"""Per-layer timing sweep over the five workload families (single GPU).

    python -m paper_2411_11038_b200.sweep [--configs 1,2,3,4,5] [--iters 30] [--out file.jsonl]

For every layer: forward ms, backward ms at each unfrozen fraction, algorithmic TFLOP/s
(2MNK forward, 2MNK(1 + k/N) backward, Eq. 7-8 of the paper), the speed-up of the partial
backward over this library's own full-QAT backward next to the ideal 2/(1+r), and the
selection time.  Every number is the median over `iters` runs timed with CUDA events, with a
256 MiB buffer written between runs so that nothing is served from a warm L2.  Each record
carries the SM clock (median, minimum) and the clock-event reasons sampled through NVML while
that record's measurements ran.
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys

import torch

from . import binding as B
from . import inputs as I
from .clocks import ClockSampler, physical_gpu_index

FRACS = {1: (0.0, 26 / 512, 1.0), 2: (0.0, 0.05, 0.25, 1.0), 3: (0.0, 0.10, 1.0), 4: (0.0, 0.10, 1.0),
         5: (0.0, 0.01, 0.05, 0.10, 0.25, 0.50, 1.0), 6: (0.0, 0.10, 1.0)}
SGD = (1e-9, 0.9, 1e-4)      # fused update of the unfrozen rows, as in bench.py (rate scaled for unit-variance dY)


def load_peaks():
    """Measured peaks of this machine (burst bf16 GEMM TFLOP/s, copy GB/s); the recipe's fallback otherwise."""
    import os
    p = os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["bf16_tflops"]), float(d["hbm_gbs"]), "measured"
    return 1590.0, 6650.0, "fallback"


def bounds(case, k, peaks, fwd_int8=False):
    """Roofline time (ms) of the forward and of the backward with k unfrozen channels:
    max(algorithmic flops / tensor peak, algorithmic bytes / copy bandwidth)."""
    tf, gbs, _ = peaks
    e = 2 if case.act_dtype == torch.bfloat16 else 4
    g = 2.0 * case.M * case.N * case.K
    x_elems = case.B * case.H * case.Wd * case.Cin if case.conv else case.M * case.K
    fwd_bytes = x_elems * e + case.N * case.K * 4 + case.M * case.N * e
    bwd_bytes = case.M * case.N * e + x_elems * e + case.N * case.K * 4 + x_elems * e + k * case.K * 4
    fwd = max(g / (tf * (2.0 if fwd_int8 else 1.0) * 1e9), fwd_bytes / (gbs * 1e6))
    bwd = max((g + 2.0 * case.M * k * case.K) / (tf * 1e9), bwd_bytes / (gbs * 1e6))
    return fwd, bwd, fwd_bytes, bwd_bytes


class Timer:
    def __init__(self, iters: int, device):
        self.iters = iters
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)

    def ms(self, fn, warmup: int = 5) -> float:
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        out = []
        for _ in range(self.iters):
            self.flush.zero_()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            fn()
            e.record()
            torch.cuda.synchronize()
            out.append(s.elapsed_time(e))
        return statistics.median(out)


def layer_on_device(ctx, case: I.LayerCase, dev):
    T = I.make_tensors(case)
    D = {k: (v.to(dev) if v is not None else None) for k, v in T.items()}
    D["s_w"] = B.init_weight_scales(ctx, D["W"], case.w_bits)
    D["s_x"], D["z_x"] = B.init_act_qparams(ctx, D["X"], case.x_bits, case.x_symmetric)
    conv = B.ConvGeom(case.B, case.H, case.Wd, case.Cin, case.R, case.S, case.stride, case.pad) if case.conv else None
    if conv is not None:
        Ho = (case.H + 2 * case.pad - case.R) // case.stride + 1
        Wo = (case.Wd + 2 * case.pad - case.S) // case.stride + 1
        plan = B.LayerPlan(ctx, case.M, case.N, case.K, case.act_dtype, case.w_bits, case.x_bits, case.x_symmetric,
                           case.N, dev, conv, x_shape=D["X"].shape, y_shape=(case.B, Ho, Wo, case.N))
    else:
        plan = B.LayerPlan(ctx, case.M, case.N, case.K, case.act_dtype, case.w_bits, case.x_bits, case.x_symmetric,
                           case.N, dev)
    return D, plan


def clocked(fn):
    """Runs a record-producing function with the clock sampler on and attaches its summary."""
    def wrapper(*args, **kwargs):
        sampler = ClockSampler(physical_gpu_index(0), period_s=0.005)
        sampler.start()
        try:
            rec = fn(*args, **kwargs)
        finally:
            sampler.stop_flag = True
            sampler.join(timeout=2)
        for r in (rec if isinstance(rec, list) else [rec]):
            r.setdefault("clocks", sampler.summary())
        return rec
    return wrapper


@clocked
def sweep_layer(ctx, case, fracs, timer, dev, ks=None):
    D, plan = layer_on_device(ctx, case, dev)
    g = 2.0 * case.M * case.N * case.K
    rec = {"layer": case.name, "M": case.M, "N": case.N, "K": case.K, "w_bits": case.w_bits, "x_bits": case.x_bits}
    peaks = load_peaks()
    int8 = (not case.conv) and case.K >= 512 and case.K % 16 == 0 and case.N % 32 == 0
    t = timer.ms(lambda: plan.fwd(D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], D["bias"]))
    fb, _, fbytes, _ = bounds(case, 0, peaks, int8)
    rec["fwd_ms"], rec["fwd_tflops"], rec["fwd_int8"] = t, g / t / 1e9, int8
    rec["fwd_bound_ms"], rec["fwd_frac_of_bound"], rec["fwd_bytes"] = fb, fb / t, fbytes
    rec["peaks"] = {"tflops": peaks[0], "hbm_gbs": peaks[1], "source": peaks[2]}
    rec["bwd"] = {}
    full_ms = None
    mom = torch.zeros_like(D["W"])
    sgd = B.make_sgd(SGD[0], SGD[1], SGD[2], D["W"], mom)
    for f in sorted(set(fracs), reverse=True):
        k = B.ratio_to_k(f, case.N) if ks is None else ks[f]
        sel = B.SelectPlan(ctx, B.CWPL, [D["W"]], [k])
        sel.run()
        idx = sel.idx[:k] if 0 < k < case.N else None
        t = timer.ms(lambda: plan.bwd(D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx, k, want_db=True,
                                      sgd=sgd))
        if f == 1.0:
            full_ms = t
        _, bb, _, bbytes = bounds(case, k, peaks)
        rec["bwd"][f"{f:.4g}"] = {"k_sel": k, "ms": t, "tflops": (g + 2.0 * case.M * k * case.K) / t / 1e9,
                                  "speedup_vs_full_qat": (full_ms / t) if full_ms else None,
                                  "ideal": 2.0 / (1.0 + k / case.N), "bound_ms": bb, "frac_of_bound": bb / t,
                                  "bytes": bbytes}
    sel = B.SelectPlan(ctx, B.CWPL, [D["W"]], [B.ratio_to_k(0.05, case.N)])
    t = timer.ms(sel.run)
    rec["select_ms"], rec["select_gbs"] = t, case.N * case.K * 4 / t / 1e6
    return rec


@clocked
def sweep_network(ctx, timer, dev):
    """Config 4: one global ranking over the 144 layers, then the per-layer steps with the
    counts that ranking assigns (the 4096->1024 layers end up fully frozen)."""
    cases = I.config4()
    Ws = []
    for c in cases:
        g = torch.Generator().manual_seed(c.seed)
        Ws.append((torch.randn((c.N, c.K), generator=g) * (2.0 / c.K) ** 0.5).to(dev))
    total = sum(c.N for c in cases)
    budget = B.ratio_to_k(0.1, total)
    plan = B.SelectPlan(ctx, B.CWPN, Ws, [budget])
    t = timer.ms(plan.run)
    nbytes = sum(w.numel() * 4 for w in Ws)
    counts = (plan.offsets[1:] - plan.offsets[:-1]).cpu().tolist()
    out = [{"layer": "cfg4_cwpn_selection_144_layers", "select_ms": t, "select_gbs": nbytes / t / 1e6,
            "channels": total, "budget": budget, "per_layer_counts_block0": counts[:6]}]
    del Ws, plan
    torch.cuda.empty_cache()
    for j in (0, 4, 5):                       # one of each shape: 1024->1024, 1024->4096, 4096->1024
        c = cases[j]
        ks = {0.0: 0, 0.10: counts[j], 1.0: c.N}
        out.append(sweep_layer(ctx, c, (0.0, 0.10, 1.0), timer, dev, ks))
    return out


@clocked
def sweep_layerwise(ctx, timer, dev):
    """Layer-wise mode (LWPN) over the four W8A8 sweep shapes as one stack: the selection kernel
    ranks whole layers by mean |w| and unfreezes the top half; a frozen layer then runs the 0 %
    backward and an unfrozen one the 100 % backward of the per-layer records above."""
    cases = I.config5()
    g = torch.Generator().manual_seed(5000)
    Ws = [(torch.randn((c.N, c.K), generator=g) * 0.02).to(dev) for c in cases]
    k_l = len(cases) // 2
    plan = B.SelectPlan(ctx, B.LWPN, Ws, [k_l])
    plan.run()
    torch.cuda.synchronize()
    t = timer.ms(plan.run)
    counts = (plan.offsets[1:] - plan.offsets[:-1]).cpu().tolist()
    nbytes = sum(w.numel() * 4 for w in Ws)
    return {"layer": "cfg5_lwpn_selection_4_layers", "select_ms": t, "select_gbs": nbytes / t / 1e6,
            "layers": [c.name for c in cases], "unfrozen_layers": k_l, "channels_per_layer": counts}


def print_markdown(path):
    """Results table of a finished sweep: one row per layer, times in ms, fractions of the
    roofline bound max(flops / tensor peak, bytes / copy bandwidth) of the measured peaks."""
    recs = [json.loads(l) for l in open(path) if l.strip()]
    print("| config | layer (M, N, K) | fwd ms (TFLOP/s; of bound) | bwd ms by unfrozen % (TFLOP/s; of bound) | "
          "speed-up vs own full-QAT bwd (ideal) | SM MHz median (min); reasons |")
    print("|---|---|---|---|---|---|")
    for r in recs:
        if "bwd" not in r:
            continue
        b = r["bwd"]
        keys = sorted(b, key=float)
        bw = " · ".join(f"{float(f) * 100:.3g}%: {b[f]['ms']:.3f} ({b[f]['tflops']:.0f}; {b[f]['frac_of_bound']:.2f})"
                        for f in keys)
        sp = " · ".join(f"{float(f) * 100:.3g}%: {b[f]['speedup_vs_full_qat']:.2f}x ({b[f]['ideal']:.2f})"
                        for f in keys if float(f) < 1.0 and b[f]["speedup_vs_full_qat"])
        c = r.get("clocks", {})
        clk = f"{c.get('sm_mhz')} ({c.get('sm_min_mhz')}); {','.join(c.get('reasons', [])) or 'none'}"
        tag = " int8" if r.get("fwd_int8") else ""
        print(f"| {r['config']} | {r['layer']} ({r['M']}, {r['N']}, {r['K']}) | {r['fwd_ms']:.3f} ({r['fwd_tflops']:.0f}{tag}; "
              f"{r['fwd_frac_of_bound']:.2f}) | {bw} | {sp} | {clk} |")
    for r in recs:
        if "bwd" not in r:
            print()
            print(json.dumps({k: v for k, v in r.items() if k != "clocks"}), "clocks:", json.dumps(r.get("clocks")))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,6,4,5", help="6 = the stride-2 layers of ResNet-50")
    ap.add_argument("--markdown", default=None, help="print the results table of a finished sweep (JSONL file) and exit")
    ap.add_argument("--iters", type=int, default=30)
    ap.add_argument("--out", default=None)
    ap.add_argument("--only", default=None, help="run only layers whose name contains this string")
    args = ap.parse_args()
    if args.markdown:
        print_markdown(args.markdown)
        return
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    ctx = B.Context(0)
    timer = Timer(args.iters, dev)
    sink = open(args.out, "w") if args.out else sys.stdout
    for cfg in (int(c) for c in args.configs.split(",")):
        if cfg == 4:
            recs = sweep_network(ctx, timer, dev)
        else:
            cases = {1: I.config1, 2: I.config2, 3: I.config3, 5: I.config5, 6: I.config3_strided}[cfg]()
            if cfg == 5:
                cases = cases + I.config5(4, 4)
            recs = []
            if args.only:
                cases = [c for c in cases if args.only in c.name]
            for c in cases:
                recs.append(sweep_layer(ctx, c, FRACS[cfg], timer, dev))
                torch.cuda.empty_cache()
            if cfg == 5 and not args.only:
                recs.append(sweep_layerwise(ctx, timer, dev))
                torch.cuda.empty_cache()
        for r in recs:
            r["config"] = cfg
            sink.write(json.dumps(r) + "\n")
            sink.flush()
    assert ctx.device_status() == 0


if __name__ == "__main__":
    main()
