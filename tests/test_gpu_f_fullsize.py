"""Full-size parity of the workload families whose numbers are quoted: the ResNet-50-shaped
convolutions at batch 64 (W4A8, 10 % unfrozen) and the GEMM-sweep shapes at M = 16384
(W8A8 and W4A4, 5 % unfrozen and the full-QAT backward), in the launch configuration the
benchmark and the sweep time.

Where the fp64 oracle of the whole layer would take minutes, it is evaluated on what it can
compute alone:
  * images of a convolution batch (or rows of a linear layer) are independent in Y and dX, so
    the oracle runs on sampled images / rows and every element of those is compared;
  * the weight gradient contracts over all rows: sampled selected channels are compared
    against the oracle's restricted loop (Algorithm 1's wording) over the whole batch, and a
    second backward with dY zeroed outside the sampled images / rows (one row in every tile of
    128) makes every output -- all of dW_sel, dS_w, dS_x, dZ_x, db -- a function of the sampled
    part alone, which the oracle then checks completely.
Tolerances are those of tests/parity_util.py.
"""
import numpy as np
import pytest
import torch

from oracle import efqat_oracle as O
from paper_2411_11038_b200 import binding as B
from paper_2411_11038_b200 import inputs as I
from tests import parity_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    return B.Context(0)


def _np(t):
    return t.detach().float().cpu().numpy()


# ------------------------------------------------------------------------------------------
# ResNet-50-shaped convolutions, batch 64
# ------------------------------------------------------------------------------------------
def _conv_sub(case, T, images):
    c = I.LayerCase(**{k: v for k, v in case.__dict__.items() if k != "tensors"})
    c.B = len(images)
    c.M = case.M // case.B * len(images)
    return c, dict(X=T["X"][images].contiguous(), W=T["W"], dY=T["dY"][images].contiguous(), bias=T["bias"])


def _batch64_cases():
    """The eight ResNet-50-shaped layers of configs[2], then layers of the real network that take
    other launch forms: the 7x7 stride-2 input layer on 8 stored channels (filter rows as
    contraction blocks, grad-input on strips of 8 pixels), the first stage's 3x3 64 -> 64 (taps of a
    filter column sharing one box, weights resident in shared memory) and the stride-2 3x3 that
    opens the second stage."""
    rn = {c.name: c for c in I.resnet50(64)}
    r20 = {c.name: c for c in I.resnet20(64)}
    # ... and two layers of the CIFAR-10 ResNet-20 (16 channels: grad-input on strips of 4 pixels)
    return I.config3() + [rn["rn50_stem"], rn["rn50_s1b1_b"], rn["rn50_s2b1_b"], r20["rn20_stem"], r20["rn20_s1b1_a"]]


@pytest.mark.parametrize("li", range(13))
def test_config3_layer_batch64(ctx, li):
    case = _batch64_cases()[li]
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.6, 0.9, 0.0))       # shrunk scales: both tensors clip
    D = U.to_dev(T, s_w, s_x, z_x)
    geom = B.ConvGeom(case.B, case.H, case.Wd, case.Cin, case.R, case.S, case.stride, case.pad)
    N, K = case.N, case.K
    k = B.ratio_to_k(0.10, N)
    W64 = I.as_f64(T["W"])
    sel, _, _ = B.select_channels(ctx, B.CWPL, [D["W"]], [k])
    idx = O.select_cwpl([W64], [k])[0]
    assert sel[0].cpu().numpy().tolist() == idx.tolist()

    # whole batch when the oracle finishes in seconds, else images at both ends of the batch
    # and on either side of its middle (pixel boxes of the small feature maps span images)
    images = list(range(case.B)) if case.M <= 16384 else [0, 31, 32, 63]
    sub, Ts = _conv_sub(case, T, images)
    Xs, dYs, b64 = (I.as_f64(Ts[kk]) for kk in ("X", "dY", "bias"))
    Yabs, Gx_abs, Gw_abs = U.conv_abs_bounds(sub, Ts, s_w, s_x, z_x)

    Y = B.fq_linear_fwd(ctx, D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], D["bias"], case.w_bits, case.x_bits,
                        False, conv=geom)
    out = B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], sel[0], k, case.w_bits,
                          case.x_bits, False, want_db=True, conv=geom)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    name = case.name
    ref = O.conv_forward(Xs, W64, s_w, s_x, z_x, b64, case.w_bits, case.x_bits, case.stride, case.pad)
    got = _np(Y[images])
    U.assert_bf16_class(got, ref, name + " Y")
    U.assert_fp32_class(got, ref, Yabs + np.abs(b64), name + " Y", out_is_bf16=True)

    args = (dYs, Xs, W64, s_w, s_x, z_x, idx, case.w_bits, case.x_bits, case.stride, case.pad)
    ex = O.conv_backward_efqat(*args, operand_model="exact")
    bm = O.conv_backward_efqat(*args, operand_model="bf16")
    dX = _np(out["dX"][images])
    clip_x = O.fake_quant_x(Xs, s_x, z_x, case.x_bits)["flag"] != 0
    assert clip_x.any() and np.all(dX[clip_x] == 0)
    U.assert_bf16_class(dX, ex["dX"], name + " dX")
    U.assert_fp32_class(dX, bm["dX"], Gx_abs, name + " dX", out_is_bf16=True)
    dY_abs_cols = T["dY"].double().abs().reshape(-1, N).sum(dim=0).numpy()
    U.assert_fp32_class(_np(out["db"]), T["dY"].double().reshape(-1, N).sum(dim=0).numpy(), dY_abs_cols, name + " db")
    dW = out["dW_sel"].cpu().numpy().reshape((k,) + W64.shape[1:])
    dSw = out["dS_w_sel"].cpu().numpy()
    full_batch = len(images) == case.B
    if full_batch:
        U.assert_bf16_class(dW, ex["dW_sel"], name + " dW_sel")
        U.assert_fp32_class(dW, bm["dW_sel"], Gw_abs[idx], name + " dW_sel")
        U.assert_fp32_class(dSw, bm["dS_w_sel"], bm["dS_w_sel_abs"], name + " dS_w", atol=1e-30)
        for key in ("dS_x", "dZ_x"):
            U.assert_fp32_class(out[key].item(), bm[key], bm[key + "_abs"], name + " " + key, atol=1e-30)
        return

    # sampled selected channels over the whole batch (dY is bf16: both operand models coincide)
    rng = np.random.default_rng(li)
    pick = np.unique(np.concatenate([[0, k - 1], rng.choice(k, min(6, k), replace=False)]))
    d = O.conv_backward_efqat_direct(I.as_f64(T["dY"]), I.as_f64(T["X"]), W64, s_w, s_x, z_x, idx[pick],
                                     case.w_bits, case.x_bits, case.stride, case.pad, operand_model="bf16")
    U.assert_bf16_class(dW[pick], d["dW_sel"], name + " dW_sel sampled channels")
    U.assert_fp32_class(dW[pick], d["dW_sel"], d["G_w_sel_abs"], name + " dW_sel sampled channels")
    U.assert_fp32_class(dSw[pick], d["dS_w_sel"], d["dS_w_sel_abs"], name + " dS_w sampled channels", atol=1e-30)

    # dY zero outside the sampled images: every output is the oracle's on those images alone
    dX_dense = out["dX"][images].clone()
    dYz = torch.zeros_like(D["dY"])
    dYz[images] = D["dY"][images]
    out = B.fq_linear_bwd(ctx, dYz, D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], sel[0], k, case.w_bits,
                          case.x_bits, False, want_db=True, conv=geom)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert torch.equal(out["dX"][images], dX_dense)
    others = [b for b in range(case.B) if b not in images]
    assert not out["dX"][others].any()
    dW = out["dW_sel"].cpu().numpy().reshape((k,) + W64.shape[1:])
    U.assert_bf16_class(dW, ex["dW_sel"], name + " dW_sel (sparse dY)")
    U.assert_fp32_class(dW, bm["dW_sel"], Gw_abs[idx], name + " dW_sel (sparse dY)")
    U.assert_fp32_class(out["dS_w_sel"].cpu().numpy(), bm["dS_w_sel"], bm["dS_w_sel_abs"], name + " dS_w (sparse dY)",
                        atol=1e-30)
    for key in ("dS_x", "dZ_x"):
        U.assert_fp32_class(out[key].item(), bm[key], bm[key + "_abs"], name + " " + key + " (sparse dY)", atol=1e-30)
    U.assert_fp32_class(_np(out["db"]), bm["db"], np.abs(dYs).reshape(-1, N).sum(axis=0), name + " db (sparse dY)")


# ------------------------------------------------------------------------------------------
# GEMM-sweep shapes at M = 16384
# ------------------------------------------------------------------------------------------
def _tile_rows(M, seed):
    """One row in every tile of 128 rows, first and last row of the matrix included."""
    rng = np.random.default_rng(seed)
    rows = np.arange(0, M, 128) + rng.integers(0, 128, size=(M + 127) // 128)
    rows[0], rows[-1] = 0, M - 1
    return np.minimum(rows, M - 1)


SWEEP = [(3, 8, 8, True), (2, 8, 8, False), (3, 4, 4, False)]      # (index into the sweep, w_bits, x_bits, dense dW sample)


@pytest.mark.parametrize("si,w_bits,x_bits,dense_dw", SWEEP, ids=["8192x8192_w8a8", "4096x16384_w8a8", "8192x8192_w4a4"])
def test_config5_large_shapes(ctx, si, w_bits, x_bits, dense_dw):
    case = I.config5(w_bits, x_bits)[si]
    M, N, K = case.M, case.N, case.K
    T = I.make_tensors(case)
    W64 = I.as_f64(T["W"])
    D = {kk: v.cuda() for kk, v in T.items()}
    # MinMax initialisation on the device agrees exactly with the oracle's
    s_w = O.init_minmax_w(W64, w_bits)
    s_x, z_x = O.init_minmax_x(I.as_f64(T["X"]), x_bits, False)
    D["s_w"] = B.init_weight_scales(ctx, D["W"], w_bits)
    D["s_x"], D["z_x"] = B.init_act_qparams(ctx, D["X"], x_bits, False)
    assert np.array_equal(D["s_w"].cpu().numpy(), s_w)
    assert D["s_x"].item() == float(s_x) and D["z_x"].item() == float(z_x)
    # move the parameters off their start so that both tensors clip and Z is fractional
    s_x = np.float32(s_x * np.float32(0.8))
    s_w = (s_w * np.float32(0.85)).astype(np.float32)
    z_x = np.float32(z_x + np.float32(0.4))
    D["s_x"].fill_(float(s_x)); D["z_x"].fill_(float(z_x)); D["s_w"].copy_(torch.from_numpy(s_w))

    k5 = B.ratio_to_k(0.05, N)
    sel, _, _ = B.select_channels(ctx, B.CWPL, [D["W"]], [k5])
    idx = O.select_cwpl([W64], [k5])[0]
    assert sel[0].cpu().numpy().tolist() == idx.tolist()
    rows = _tile_rows(M, si)
    rows_t = torch.from_numpy(rows).cuda()
    Xr, dYr, b64 = I.as_f64(T["X"][rows]), I.as_f64(T["dY"][rows]), I.as_f64(T["bias"])
    name = case.name

    plan = B.LayerPlan(ctx, M, N, K, case.act_dtype, w_bits, x_bits, False, N, "cuda")
    Y = plan.fwd(D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], D["bias"])
    Yr = _np(Y[rows_t])
    sub = I.shrink(case, len(rows))
    ref, ref_abs = U.fwd_reference(sub, dict(X=T["X"][rows], W=T["W"], bias=T["bias"]), s_w, s_x, z_x)
    U.assert_bf16_class(Yr, ref, name + " Y rows")
    U.assert_fp32_class(Yr, ref, ref_abs, name + " Y rows", out_is_bf16=True)

    ex = O.backward_full(dYr, Xr, W64, s_w, s_x, z_x, w_bits, x_bits, operand_model="exact")
    bm = O.backward_full(dYr, Xr, W64, s_w, s_x, z_x, w_bits, x_bits, operand_model="bf16")
    qxr = O.fake_quant_x(Xr, s_x, z_x, x_bits)
    clip_x = qxr["flag"] != 0
    clip_w = O.fake_quant_w(W64, s_w, w_bits)["flag"] != 0
    assert clip_x.any() and clip_w.any()
    # bf16 operand rounding against the exact oracle: 1e-2 of the sum of |terms| of the whole
    # reduction (the terms of G_x included: few clipped elements make dZ_x a short sum of
    # long, cancelling dot products)
    loose = {"dS_x": U.BF16_CLASS * (ex["G_x_abs"] * np.abs(qxr["t"])).sum(),
             "dZ_x": U.BF16_CLASS * (ex["G_x_abs"] * np.abs(qxr["dz"])).sum()}
    # fp32 class: dS_x = sum_{m,k,n} dY[m,n] w^[n,k] t[m,k] is one triple sum; its sum of |terms|
    nested = {"dS_x": (bm["G_x_abs"] * np.abs(qxr["t"])).sum(), "dZ_x": (bm["G_x_abs"] * np.abs(qxr["dz"])).sum()}
    dYz = torch.zeros_like(D["dY"])
    dYz[rows_t] = D["dY"][rows_t]
    not_rows = torch.ones(M, dtype=torch.bool, device="cuda")
    not_rows[rows_t] = False
    dY_cols = T["dY"].double().sum(dim=0).numpy()
    dY_cols_abs = T["dY"].double().abs().sum(dim=0).numpy()

    dense = {}
    for k_sel in (k5, N):
        tag = f"{name} k_sel={k_sel}"
        idx_dev = sel[0] if k_sel < N else None
        chan = idx.astype(np.int64) if k_sel < N else np.arange(N)
        # dense dY: sampled rows of dX, db, and (below) sampled channels of dW
        out = plan.bwd(D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx_dev, k_sel)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        dXr_t = out["dX"][rows_t].clone()
        dXr = _np(dXr_t)
        assert np.all(dXr[clip_x] == 0), tag + " dX mask"
        U.assert_bf16_class(dXr, ex["dX"], tag + " dX rows")
        U.assert_fp32_class(dXr, bm["dX"], bm["G_x_abs"], tag + " dX rows", out_is_bf16=True)
        U.assert_fp32_class(_np(out["db"]), dY_cols, dY_cols_abs, tag + " db")
        dense[k_sel] = dict(dW=out["dW_sel"].clone(), dS_x=out["dS_x"].item(), dZ_x=out["dZ_x"].item())
        # dY zero outside the sampled rows: every output against the oracle on those rows
        out = plan.bwd(dYz, D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx_dev, k_sel)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        assert torch.equal(out["dX"][rows_t], dXr_t), tag + " dX rows differ between the two runs"
        assert not out["dX"][not_rows].any(), tag + " dX outside the sampled rows"
        dW = out["dW_sel"].cpu().numpy()
        assert np.all(dW[clip_w[chan]] == 0), tag + " dW mask"
        U.assert_bf16_class(dW, ex["dW"][chan], tag + " dW_sel (sparse dY)")
        U.assert_fp32_class(dW, bm["dW"][chan], bm["G_w_abs"][chan], tag + " dW_sel (sparse dY)")
        U.assert_fp32_class(out["dS_w_sel"].cpu().numpy(), bm["dS_w"][chan], bm["dS_w_abs"][chan], tag + " dS_w (sparse dY)",
                            atol=1e-30)
        for key in ("dS_x", "dZ_x"):
            assert abs(out[key].item() - ex[key]) <= loose[key], tag + " " + key
            U.assert_fp32_class(out[key].item(), bm[key], nested[key], tag + " " + key + " (sparse dY)", atol=1e-30)
        U.assert_fp32_class(_np(out["db"]), bm["db"], np.abs(dYr).sum(axis=0), tag + " db (sparse dY)")
        del out, dW

    # dense dY at full size: dS_x / dZ_x do not depend on the selection; the rows both backward
    # calls produce (gathered partial product vs the full weight-gradient GEMM) agree
    assert dense[k5]["dS_x"] == dense[N]["dS_x"] and dense[k5]["dZ_x"] == dense[N]["dZ_x"]
    a, b = dense[k5]["dW"], dense[N]["dW"][sel[0].long()]
    scale = b.abs().max().item()
    assert (a - b).abs().max().item() <= 1e-4 * scale, name + " partial vs full weight gradient"
    if dense_dw:
        rng = np.random.default_rng(si)
        pick5 = np.unique(np.concatenate([[0, k5 - 1], rng.choice(k5, 6, replace=False)]))
        other = rng.choice(N, 8, replace=False)
        chan = np.unique(np.concatenate([idx[pick5], other]))
        d = O.backward_efqat_direct(I.as_f64(T["dY"]), I.as_f64(T["X"]), W64, s_w, s_x, z_x, chan, w_bits, x_bits,
                                    operand_model="bf16")
        gotN = dense[N]["dW"][torch.from_numpy(chan).cuda()].cpu().numpy()
        U.assert_bf16_class(gotN, d["dW_sel"], name + " dense dW, full backward, sampled channels")
        U.assert_fp32_class(gotN, d["dW_sel"], d["G_w_sel_abs"], name + " dense dW, full backward, sampled channels")
        pos = np.searchsorted(chan, idx[pick5])
        got5 = dense[k5]["dW"][torch.from_numpy(pick5).cuda()].cpu().numpy()
        U.assert_fp32_class(got5, d["dW_sel"][pos], d["G_w_sel_abs"][pos], name + " dense dW, 5 %, sampled channels")


def test_config5_4096_dense_reductions(ctx):
    """M = 16384, K = N = 4096, dense dY: the oracle's complete backward (one fp64 pass), so that
    dS_x, dZ_x and every dS_w are compared with full reductions at the stated class."""
    case = I.config5()[1]
    M, N, K = case.M, case.N, case.K
    T = I.make_tensors(case)
    X64, W64, dY64 = (I.as_f64(T[kk]) for kk in ("X", "W", "dY"))
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.8, 0.85, 0.4))
    D = U.to_dev(T, s_w, s_x, z_x)
    k = B.ratio_to_k(0.05, N)
    idx = O.select_cwpl([W64], [k])[0]
    bm = O.backward_full(dY64, X64, W64, s_w, s_x, z_x, 8, 8, operand_model="bf16")
    plan = B.LayerPlan(ctx, M, N, K, case.act_dtype, 8, 8, False, N, "cuda")
    for k_sel in (k, N):
        tag = f"{case.name} dense k_sel={k_sel}"
        chan = idx.astype(np.int64) if k_sel < N else np.arange(N)
        idx_dev = torch.from_numpy(idx).cuda() if k_sel < N else None
        out = plan.bwd(D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx_dev, k_sel)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        U.assert_fp32_class(_np(out["dX"]), bm["dX"], bm["G_x_abs"], tag + " dX", out_is_bf16=True)
        for key in ("dS_x", "dZ_x"):
            U.assert_fp32_class(out[key].item(), bm[key], bm[key + "_abs"], tag + " " + key, atol=1e-30)
        U.assert_fp32_class(out["dW_sel"].cpu().numpy(), bm["dW"][chan], bm["G_w_abs"][chan], tag + " dW_sel")
        U.assert_fp32_class(out["dS_w_sel"].cpu().numpy(), bm["dS_w"][chan], bm["dS_w_abs"][chan], tag + " dS_w",
                            atol=1e-30)
        U.assert_fp32_class(_np(out["db"]), bm["db"], np.abs(dY64).sum(axis=0), tag + " db")


@pytest.mark.parametrize("which", ["conv_28x28_3x3", "linear_4096x4096"])
def test_backward_is_bit_reproducible_at_full_size(ctx, which):
    """Thirty backward calls on the same inputs, with host-side pauses of varying length between
    them so that the launches meet the GPU in different states: dX, dS_x, dZ_x, dW_sel and db
    must come out bit-identical every time (every reduction has a fixed order, and nothing may
    depend on timing)."""
    import time
    if which.startswith("conv"):
        case = I.config3()[3]
        geom = B.ConvGeom(case.B, case.H, case.Wd, case.Cin, case.R, case.S, 1, case.pad)
        frac = 0.10
    else:
        case, geom, frac = I.config5()[1], None, 0.05
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.6, 0.9, 0.3 if geom is None else 0.0))
    D = U.to_dev(T, s_w, s_x, z_x)
    k = B.ratio_to_k(frac, case.N)
    sel, _, _ = B.select_channels(ctx, B.CWPL, [D["W"]], [k])
    first = None
    for it in range(30):
        out = B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], sel[0], k, case.w_bits,
                              case.x_bits, False, want_db=True, conv=geom)
        torch.cuda.synchronize()
        cur = {kk: v.clone() for kk, v in out.items()}
        if first is None:
            first = cur
        for kk in first:
            assert torch.equal(cur[kk], first[kk]), f"{case.name}: {kk} differs in repeat {it}"
        time.sleep(0.002 * (it % 5))
    assert ctx.device_status() == 0
