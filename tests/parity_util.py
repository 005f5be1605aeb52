"""Shared helpers of the GPU parity tests: run a layer case through the CUDA library
and through the oracle on the same bytes, and compare under the stated tolerances.

Tolerances (written out here once):
  * integer codes, clip flags, selected index sets: bit-exact;
  * "bf16 path" outputs against the exact fp64 oracle:  max|err| <= 1e-2 * max|ref|;
  * fp32-accumulation class against the oracle run with the same bf16 operand rounding:
    |err| <= 1e-5 * (sum of |terms| of that dot product / reduction), plus one bf16
    rounding (2^-8 relative) where the output itself is stored as bf16.
"""
import numpy as np
import torch

from oracle import efqat_oracle as O
from paper_2411_11038_b200 import binding as B
from paper_2411_11038_b200.inputs import LayerCase, as_f64, make_tensors

BF16_CLASS = 1e-2
FP32_CLASS = 1e-5
BF16_ULP = 2.0 ** -8


def np32(t):
    return t.detach().float().cpu().numpy()


def oracle_qparams(case: LayerCase, T, shrink=None):
    """MinMax initialisation through the oracle; `shrink` = (fx, fw, dz) moves the
    parameters off their initial values so that both tensors clip and Z is fractional."""
    X64, W64 = as_f64(T["X"]), as_f64(T["W"])
    s_w = O.init_minmax_w(W64, case.w_bits)
    s_x, z_x = O.init_minmax_x(X64, case.x_bits, case.x_symmetric)
    if shrink is not None:
        fx, fw, dz = shrink
        s_x = np.float32(s_x * np.float32(fx))
        s_w = (s_w * np.float32(fw)).astype(np.float32)
        if not case.x_symmetric:
            z_x = np.float32(z_x + np.float32(dz))
    return s_w, np.float32(s_x), np.float32(z_x)


def to_dev(T, s_w, s_x, z_x, dev="cuda"):
    D = {k: (v.to(dev) if v is not None else None) for k, v in T.items()}
    D["s_w"] = torch.from_numpy(np.asarray(s_w, np.float32)).to(dev)
    D["s_x"] = torch.tensor([float(s_x)], dtype=torch.float32, device=dev)
    D["z_x"] = torch.tensor([float(z_x)], dtype=torch.float32, device=dev)
    return D


def assert_bf16_class(got, ref, what):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    if ref.size == 0:
        return
    err = np.abs(got - ref).max()
    bound = BF16_CLASS * max(np.abs(ref).max(), 1e-30)
    assert err <= bound, f"{what}: max|err| {err:.3e} > 1e-2*max|ref| = {bound:.3e}"


def assert_fp32_class(got, ref, abs_sum, what, out_is_bf16=False, atol=0.0):
    got, ref, abs_sum = (np.asarray(a, np.float64) for a in (got, ref, abs_sum))
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    if ref.size == 0:
        return
    bound = FP32_CLASS * abs_sum + atol
    if out_is_bf16:
        bound = bound + BF16_ULP * np.abs(ref)
    bad = np.abs(got - ref) > bound
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} beyond 1e-5*abs-sum; worst "
                           f"{np.abs(got - ref)[bad].max():.3e} vs bound {np.asarray(bound)[bad].min():.3e}")


def fwd_reference(case, T, s_w, s_x, z_x):
    X64, W64 = as_f64(T["X"]), as_f64(T["W"])
    b = as_f64(T["bias"]) if T.get("bias") is not None else None
    Y = O.forward(X64, W64, s_w, s_x, z_x, b, case.w_bits, case.x_bits, case.x_symmetric)
    qx = O.fake_quant_x(X64, s_x, z_x, case.x_bits, case.x_symmetric)
    qw = O.fake_quant_w(W64, s_w, case.w_bits)
    Yabs = np.abs(qx["deq"]) @ np.abs(qw["deq"]).T
    if b is not None:
        Yabs = Yabs + np.abs(b)[None, :]
    return Y, Yabs


def check_forward_values(case, T, Y, s_w, s_x, z_x):
    """Compares a forward output Y (device tensor) with the oracle's on the CPU tensors T."""
    ref, ref_abs = fwd_reference(case, T, s_w, s_x, z_x)
    got = np32(Y)
    is_bf16 = case.act_dtype == torch.bfloat16
    assert_bf16_class(got, ref, f"{case.name} Y")
    assert_fp32_class(got, ref, ref_abs, f"{case.name} Y", out_is_bf16=is_bf16)
    return got


def check_forward(ctx, case, T, D, s_w, s_x, z_x):
    Y = B.fq_linear_fwd(ctx, D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], D.get("bias"),
                        case.w_bits, case.x_bits, case.x_symmetric)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return check_forward_values(case, T, Y, s_w, s_x, z_x)


def check_backward(ctx, case, T, D, s_w, s_x, z_x, idx_np, sgd=None, full_ref=None):
    """Runs efqat_fq_linear_bwd for the channel set idx_np and compares every output with
    the oracle.  Returns the GPU outputs (numpy) for cross-case invariants."""
    k_sel = len(idx_np)
    N = case.N
    idx_dev = torch.from_numpy(np.asarray(idx_np, np.int32)).to("cuda") if 0 < k_sel < N else None
    out = B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx_dev, k_sel,
                          case.w_bits, case.x_bits, case.x_symmetric, want_db=True, sgd=sgd)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    X64, W64, dY64 = as_f64(T["X"]), as_f64(T["W"]), as_f64(T["dY"])
    args = (dY64, X64, W64, s_w, s_x, z_x, idx_np, case.w_bits, case.x_bits, case.x_symmetric)
    ex = O.backward_efqat(*args, operand_model="exact")
    bm = O.backward_efqat(*args, operand_model="bf16")
    is_bf16 = case.act_dtype == torch.bfloat16
    g = {k: (np32(v) if v is not None else None) for k, v in out.items()}
    name = f"{case.name} k_sel={k_sel}"
    # straight-through masks: exactly zero wherever the oracle's code was clipped
    clip_x = O.fake_quant_x(X64, s_x, z_x, case.x_bits, case.x_symmetric)["flag"] != 0
    assert np.all(g["dX"][clip_x] == 0), name + " dX mask"
    assert_bf16_class(g["dX"], ex["dX"], name + " dX")
    assert_fp32_class(g["dX"], bm["dX"], bm["G_x_abs"], name + " dX", out_is_bf16=is_bf16)
    for key in ("dS_x", "dZ_x"):
        # against the exact oracle the bf16 operand rounding shows: bound by 1e-2 of the abs-sum
        assert abs(g[key][0] - ex[key]) <= BF16_CLASS * ex[key + "_abs"] + 1e-30, name + " " + key
        assert_fp32_class(g[key][0], bm[key], bm[key + "_abs"], name + " " + key, atol=1e-30)
    assert_fp32_class(g["db"], bm["db"], np.abs(dY64).sum(axis=0), name + " db")
    assert g["dW_sel"].shape == (k_sel, case.K)
    if k_sel:
        assert_bf16_class(g["dW_sel"], ex["dW_sel"], name + " dW_sel")
        assert_fp32_class(g["dW_sel"], bm["dW_sel"], bm["G_w_sel_abs"], name + " dW_sel")
        assert_fp32_class(g["dS_w_sel"], bm["dS_w_sel"], bm["dS_w_sel_abs"], name + " dS_w_sel", atol=1e-30)
        clip_w = O.fake_quant_w(W64, s_w, case.w_bits)["flag"][np.asarray(idx_np, np.int64)] != 0
        assert np.all(g["dW_sel"][clip_w] == 0), name + " dW mask"
    return g


def conv_abs_bounds(case, T, s_w, s_x, z_x):
    """Sum of |terms| of every output of the three contractions (same loops as the definition)."""
    X64, W64, dY64 = (as_f64(T[k]) for k in ("X", "W", "dY"))
    qx = O.fake_quant_x(X64, s_x, z_x, case.x_bits)
    qw = O.fake_quant_w(W64, s_w, case.w_bits)
    N, R, S, C = W64.shape
    Bn, H, Wd, _ = X64.shape
    Ho, Wo = dY64.shape[1:3]
    pad, st = case.pad, case.stride
    P = O._patches(np.abs(qx["deq"]), R, S, st, pad).reshape(-1, R * S * C)
    Yabs = (P @ np.abs(qw["deq"]).reshape(N, -1).T).reshape(Bn, Ho, Wo, N)
    dY2 = np.abs(dY64).reshape(-1, N)
    Pc = O._patches(np.abs(qx["c0"]), R, S, st, pad).reshape(-1, R * S * C)
    Gw_abs = (float(s_x) * (dY2.T @ Pc)).reshape(N, R, S, C)
    Gp = (dY2 @ np.abs(qw["deq"]).reshape(N, -1)).reshape(Bn, Ho, Wo, R, S, C)
    Gxp = np.zeros((Bn, H + 2 * pad + st, Wd + 2 * pad + st, C))
    for r in range(R):
        for s in range(S):
            Gxp[:, r:r + st * Ho:st, s:s + st * Wo:st, :] += Gp[:, :, :, r, s, :]
    return Yabs, Gxp[:, pad:pad + H, pad:pad + Wd, :], Gw_abs
