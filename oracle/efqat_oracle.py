"""fp64 CPU oracle for the EfQAT fake-quantized linear / conv training step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition of what the
CUDA library computes.  It shares no code with the CUDA path and is imported only
by the tests, the smoke check and the CPU-baseline leg of the benchmark.  The
product never routes through it.

Every function follows a passage of the EfQAT paper (arxiv 2411.11038):

  Eq. 1   asymmetric b-bit activation quantizer
  Eq. 2   MinMax activation scale / zero point
  Eq. 3   symmetric b-bit per-channel weight quantizer (restricted range, Z_w = 0)
  Eq. 4   weight scale from the channel's absolute maximum
  Eq. 5   the two backward contractions  dX^ = dY W^,  dW^ = dY^T X^
  Eq. 6   block importance = mean |w| of the block
  Table 2 modes CWPL / CWPN / LWPN, all three using Top-K
  Algorithm 1  partial weight gradient on the unfrozen channels only
  Section 4 "Setup"  straight-through estimator for the rounding, SGD momentum,
                     Adam for the quantization parameters
  Appendix A.2  optional log2 parameterisation of the scales

Readings of points the paper leaves open (rounding ties, how x/s is evaluated,
gradient of the quantizer w.r.t. scale and zero point, tie-breaks in Top-K, the
budget unit of CWPN / LWPN) are stated where they are used.

Parity pins: every function here is pinned by tests/test_oracle_pins.py except the
budget rules of `select_cwpn` (budget counted in channels) and `select_lwpn`
(budget counted in layers), for which the paper prints no example:
"parity unpinned" for those two budget rules; their ranking/tie-break logic is
pinned by brute force.

All floating point is fp64 except the one step the method fixes in fp32: the
integer code is decided from  u32 = fl32(x * fl32(1/s))  (one fp32 reciprocal per
scale, one fp32 multiply per element, both round-to-nearest-even), so that an
fp32 device implementation can reproduce the codes bit for bit.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
F64 = np.float64


# ----------------------------------------------------------------------------
# small helpers
# ----------------------------------------------------------------------------
def qmax_w(bits: int) -> int:
    """Largest weight code, 2^(b-1) - 1 (Eq. 3 / Eq. 4 denominator)."""
    return (1 << (bits - 1)) - 1


def qmax_x(bits: int) -> int:
    """Largest activation code, 2^b - 1 (Eq. 1)."""
    return (1 << bits) - 1


def ratio_to_k(ratio: float, n: int) -> int:
    """Number of unfrozen channels floor(r * C_out) (Eq. 7)."""
    return int(np.floor(F64(ratio) * n))


def _rne(v):
    """Round to nearest, ties to even (the reading taken for the paper's
    round-to-nearest operator)."""
    return np.rint(v)


def _u32(x, s):
    """fp32 evaluation of x/s that decides the integer code:
    fl32(x * fl32(1/s)).  The quotient of two floats and the product of two
    floats are formed in fp64 (exact or correctly rounded there) and rounded
    once to fp32."""
    x = np.asarray(x)
    r = (F64(1.0) / np.asarray(s, dtype=F32).astype(F64)).astype(F32)
    return (x.astype(F32).astype(F64) * r.astype(F64)).astype(F32)


def bf16_rne(v):
    """Round fp32 values to the bfloat16 grid (8-bit significand), ties to even;
    returned as fp64.  Used only by the 'bf16' operand model."""
    a = np.ascontiguousarray(np.asarray(v, dtype=F32))
    b = a.view(np.uint32).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) & 0xFFFF0000
    return b.astype(np.uint32).view(F32).astype(F64).reshape(a.shape)


# ----------------------------------------------------------------------------
# Eq. 6 importance and Top-K selection (Table 2 modes)
# ----------------------------------------------------------------------------
def importance_rows(W):
    """I[n] = (1/K) sum_k |W[n,k]|, block = output channel (row).  Eq. 6.
    fp64 accumulation, key stored as fp32.  Conv weights [N,R,S,C] are viewed as
    [N, R*S*C]."""
    W2 = np.asarray(W, dtype=F64).reshape(W.shape[0], -1)
    return (np.abs(W2).sum(axis=1) / W2.shape[1]).astype(F32)


def importance_layer(W):
    """I_layer = mean |w| over the whole layer, block = layer (LWPN).  Eq. 6."""
    W2 = np.asarray(W, dtype=F64).reshape(-1)
    return F32(np.abs(W2).sum() / W2.size)


def select_topk(keys, k):
    """Top-K of fp32 keys: larger key first, equal keys by smaller index; the k
    winners are returned in ascending index order."""
    keys = np.asarray(keys, dtype=F32)
    n = keys.shape[0]
    k = int(k)
    assert 0 <= k <= n
    order = sorted(range(n), key=lambda i: (-float(keys[i]), i))
    return np.array(sorted(order[:k]), dtype=np.int32)


def select_cwpl(weights, ks):
    """Channel-wise, per-layer: Top-k_l inside every layer."""
    return [select_topk(importance_rows(W), k) for W, k in zip(weights, ks)]


def select_cwpn(weights, k_total):
    """Channel-wise, per-network: one ranking over all layers' channels (global id
    = layer offset + channel; ties by smaller global id), budget counted in
    channels, winners split back per layer."""
    keys = [importance_rows(W) for W in weights]
    offs = np.concatenate([[0], np.cumsum([len(kk) for kk in keys])])
    g = select_topk(np.concatenate(keys) if keys else np.zeros(0, F32), k_total)
    out = []
    for l in range(len(weights)):
        m = (g >= offs[l]) & (g < offs[l + 1])
        out.append((g[m] - offs[l]).astype(np.int32))
    return out


def select_lwpn(weights, k_layers):
    """Layer-wise, per-network: Top-k over the layers' importances; a selected
    layer has all its channels unfrozen, the others none."""
    keys = np.array([importance_layer(W) for W in weights], dtype=F32)
    chosen = set(select_topk(keys, k_layers).tolist())
    return [np.arange(W.shape[0], dtype=np.int32) if l in chosen
            else np.zeros(0, np.int32) for l, W in enumerate(weights)]


# ----------------------------------------------------------------------------
# Eq. 2 / Eq. 4 MinMax initialisation
# ----------------------------------------------------------------------------
def init_minmax_w(W, bits):
    """s_w[n] = max_k |W[n,k]| / (2^(b-1)-1), stored fp32 (Eq. 4).  An all-zero
    channel gets scale 1."""
    W2 = np.asarray(W, dtype=F64).reshape(W.shape[0], -1)
    s = np.abs(W2).max(axis=1) / qmax_w(bits)
    s = s.astype(F32)
    s[s == 0] = F32(1.0)
    return s


def init_minmax_x(X, bits, symmetric=False):
    """Asymmetric: s = (beta-alpha)/(2^b-1), Z = -rne(alpha/s) (Eq. 2) with
    [alpha,beta] = [min X, max X].  Symmetric variant: s = max|X|/(2^(b-1)-1),
    Z = 0.  Both returned as fp32; a degenerate range gets scale 1."""
    Xd = np.asarray(X, dtype=F64)
    if symmetric:
        s = F32(np.abs(Xd).max() / qmax_w(bits))
        if s == 0:
            s = F32(1.0)
        return s, F32(0.0)
    a, b = Xd.min(), Xd.max()
    s = F32((b - a) / qmax_x(bits))
    if s == 0:
        s = F32(1.0)
    z = F32(-_rne(a / F64(s)))
    return s, z


# ----------------------------------------------------------------------------
# Eq. 1 / Eq. 3 fake quantisation
# ----------------------------------------------------------------------------
def fake_quant_w(W, s_w, bits):
    """Symmetric per-channel weight quantizer (Eq. 3, read as a clamp to
    [-(2^(b-1)-1), 2^(b-1)-1]).

    Returns dict: q (int32 codes), flag (uint8: 0 in range, 1 clipped low,
    2 clipped high, decided on the pre-clamp integer, boundaries inclusive),
    deq (fp64 s*q), t (fp64 d(deq)/d(s) under the straight-through estimator:
    q - w/s in range, q when clipped)."""
    Q = qmax_w(bits)
    shape = np.asarray(W).shape
    W2 = np.asarray(W).reshape(shape[0], int(np.prod(shape[1:])))
    s = np.asarray(s_w, dtype=F32).reshape(-1, 1)
    c = _rne(_u32(W2, s).astype(F64))
    q = np.clip(c, -Q, Q)
    flag = np.where(c < -Q, 1, np.where(c > Q, 2, 0)).astype(np.uint8)
    sd = s.astype(F64)
    u = W2.astype(F64) / sd
    t = np.where(flag == 0, q - u, q)
    return dict(q=q.astype(np.int32).reshape(shape), flag=flag.reshape(shape),
                deq=(sd * q).reshape(shape), t=t.reshape(shape))


def fake_quant_x(X, s_x, z_x, bits, symmetric=False):
    """Per-tensor activation quantizer.

    Asymmetric (Eq. 1): Zr = clamp(rne(Z),0,Qx); c = rne(x/s)+Zr; q = clamp(c,0,Qx);
    x^ = s (q - Zr).  Symmetric variant: Zr = 0 and range [-Qs,Qs], Qs=2^(b-1)-1.

    Returns dict: q, flag (as for weights), c0 = q - Zr (the centred integer that
    enters the contractions), deq (fp64 s*c0), t = d(deq)/d(s) (STE: c0 - x/s in
    range, c0 when clipped), dz = d(deq)/d(Z) (0 in range, -s when clipped), Zr."""
    Xa = np.asarray(X)
    s32 = F32(s_x)
    sd = F64(s32)
    if symmetric:
        lo, hi, Zr = -qmax_w(bits), qmax_w(bits), 0.0
    else:
        lo, hi = 0, qmax_x(bits)
        Zr = float(np.clip(_rne(F64(F32(z_x))), lo, hi))
    c = _rne(_u32(Xa, s32).astype(F64)) + Zr
    q = np.clip(c, lo, hi)
    flag = np.where(c < lo, 1, np.where(c > hi, 2, 0)).astype(np.uint8)
    c0 = q - Zr
    u = Xa.astype(F64) / sd
    t = np.where(flag == 0, c0 - u, c0)
    dz = np.where(flag == 0, 0.0, -sd)
    return dict(q=q.astype(np.int32), flag=flag, c0=c0, deq=sd * c0, t=t, dz=dz, Zr=Zr)


# ----------------------------------------------------------------------------
# forward and backward of the fake-quantised linear layer
# ----------------------------------------------------------------------------
def forward(X, W, s_w, s_x, z_x, bias, w_bits, x_bits, x_symmetric=False):
    """Y = X^ W^^T + b in fp64 (Section 3.1; PyTorch Linear convention
    [M,K] x [N,K]^T).  Integer operands are exact in bf16, so there is no
    separate operand model for the forward."""
    qx = fake_quant_x(X, s_x, z_x, x_bits, x_symmetric)
    qw = fake_quant_w(W, s_w, w_bits)
    Y = qx["deq"] @ qw["deq"].T
    if bias is not None:
        Y = Y + np.asarray(bias, dtype=F64)[None, :]
    return Y


def backward_full(dY, X, W, s_w, s_x, z_x, w_bits, x_bits, x_symmetric=False,
                  operand_model="exact"):
    """Ordinary QAT backward of the layer (Eq. 5 + STE).

    G_x = dY W^          dX = G_x * [x not clipped]
    G_w = dY^T X^        dW = G_w * [w not clipped]
    dS_x = sum G_x t_x   dZ_x = sum G_x dz_x   dS_w[n] = sum_k G_w[n,k] t_w[n,k]
    db[n] = sum_m dY[m,n]

    operand_model 'exact': fp64 operands as defined.  'bf16': the operands a
    bf16 tensor-core contraction sees -- dY rounded to bf16 and, in G_x only,
    W^ replaced by bf16(fl32(s_w q_w)); the integer operands are exact either
    way and s_x multiplies G_w afterwards.  Also returns the absolute sums that
    bound the rounding error of the three reductions."""
    dYd = np.asarray(dY, dtype=F64)
    qx = fake_quant_x(X, s_x, z_x, x_bits, x_symmetric)
    qw = fake_quant_w(W, s_w, w_bits)
    What = qw["deq"]
    dYo = dYd
    if operand_model == "bf16":
        dYo = bf16_rne(dYd)
        s = np.asarray(s_w, dtype=F32).reshape(-1, 1)
        What = bf16_rne((s.astype(F64) * qw["q"]).astype(F32))
    elif operand_model != "exact":
        raise ValueError(operand_model)
    G_x = dYo @ What                                   # [M,N] x [N,K]
    G_w = F64(F32(s_x)) * (dYo.T @ qx["c0"])           # [N,M] x [M,K]
    in_x = qx["flag"] == 0
    in_w = qw["flag"] == 0
    out = dict(
        dX=np.where(in_x, G_x, 0.0),
        dW=np.where(in_w, G_w, 0.0),
        dS_x=(G_x * qx["t"]).sum(), dS_x_abs=np.abs(G_x * qx["t"]).sum(),
        dZ_x=(G_x * qx["dz"]).sum(), dZ_x_abs=np.abs(G_x * qx["dz"]).sum(),
        dS_w=(G_w * qw["t"]).sum(axis=1), dS_w_abs=np.abs(G_w * qw["t"]).sum(axis=1),
        db=dYd.sum(axis=0),
        G_x_abs=np.abs(dYo) @ np.abs(What),
        G_w_abs=F64(F32(s_x)) * (np.abs(dYo).T @ np.abs(qx["c0"])),
    )
    return out


def backward_efqat(dY, X, W, s_w, s_x, z_x, idx, w_bits, x_bits, x_symmetric=False,
                   operand_model="exact"):
    """EfQAT backward (Algorithm 1): dX, dS_x, dZ_x, db as in the full backward;
    weight gradient and weight-scale gradient only for the unfrozen channels,
    dW_sel[i,:] = rows idx[i] of the full dW (read as dY[:,idx]^T X^)."""
    full = backward_full(dY, X, W, s_w, s_x, z_x, w_bits, x_bits, x_symmetric,
                         operand_model)
    idx = np.asarray(idx, dtype=np.int64)
    out = {k: full[k] for k in ("dX", "dS_x", "dS_x_abs", "dZ_x", "dZ_x_abs", "db",
                                "G_x_abs")}
    out["dW_sel"] = full["dW"][idx]
    out["dS_w_sel"] = full["dS_w"][idx]
    out["dS_w_sel_abs"] = full["dS_w_abs"][idx]
    out["G_w_sel_abs"] = full["G_w_abs"][idx]
    return out


def backward_efqat_direct(dY, X, W, s_w, s_x, z_x, idx, w_bits, x_bits,
                          x_symmetric=False, operand_model="exact"):
    """The same partial weight gradient computed the way Algorithm 1 words it:
    take the columns idx of dY, contract them with X^, never forming the other
    rows.  Must agree with `backward_efqat` (self-check of the indexing).

    operand_model as in `backward_full` (only the rounding of dY to bf16 touches
    this contraction; the integer operand is exact either way).  Also returns
    the sums of absolute terms that bound the rounding error of the
    contraction and of the weight-scale reduction."""
    idx = np.asarray(idx, dtype=np.int64)
    dYd = np.asarray(dY, dtype=F64)[:, idx]
    if operand_model == "bf16":
        dYd = bf16_rne(dYd)
    elif operand_model != "exact":
        raise ValueError(operand_model)
    qx = fake_quant_x(X, s_x, z_x, x_bits, x_symmetric)
    qw = fake_quant_w(np.asarray(W)[idx], np.asarray(s_w)[idx], w_bits)
    G = F64(F32(s_x)) * (dYd.T @ qx["c0"])
    return dict(dW_sel=np.where(qw["flag"] == 0, G, 0.0),
                dS_w_sel=(G * qw["t"]).sum(axis=1),
                dS_w_sel_abs=np.abs(G * qw["t"]).sum(axis=1),
                G_w_sel_abs=F64(F32(s_x)) * (np.abs(dYd).T @ np.abs(qx["c0"])))


def sgd_rows(W, V, dW_sel, idx, lr, momentum, weight_decay):
    """SGD with momentum on the unfrozen rows only (Algorithm 1 optimizer step;
    hyper-parameters of Section 4): v <- mu v + (g + lambda w); w <- w - lr v.
    Frozen rows of W and V are returned untouched.  fp64."""
    W2 = np.array(W, dtype=F64)
    V2 = np.array(V, dtype=F64)
    for i, n in enumerate(np.asarray(idx)):
        g = np.asarray(dW_sel[i], dtype=F64) + weight_decay * W2[n]
        V2[n] = momentum * V2[n] + g
        W2[n] = W2[n] - lr * V2[n]
    return W2, V2


def adam_qparams(p, m, v, grad, idx, step, lr, beta1=0.9, beta2=0.999, eps=1e-8,
                 theta=None):
    """Adam step (Kingma & Ba, as cited in Section 4 "Setup" for the quantization
    parameters) on the entries idx of the parameter vector p with the compact
    gradient grad[i] = dL/dp[idx[i]]; entries outside idx and their moments are
    returned untouched (a frozen channel's scale is not updated, Algorithm 1).

        m <- b1 m + (1-b1) g      v <- b2 v + (1-b2) g^2
        p <- p - lr (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps),   t = step >= 1

    theta given (Appendix A.2, scales only): the optimised variable is
    theta = log2(p); its gradient is dL/dp * p * ln 2 by the chain rule through
    p = 2^theta, the same step is taken on theta and p <- 2^theta.  Zero points
    are always trained raw.  Returns new (p, m, v) or (p, m, v, theta).  fp64."""
    p2, m2, v2 = (np.array(a, dtype=F64).reshape(-1) for a in (p, m, v))
    th2 = None if theta is None else np.array(theta, dtype=F64).reshape(-1)
    g = np.asarray(grad, dtype=F64).reshape(-1)
    idx = np.arange(p2.size) if idx is None else np.asarray(idx, dtype=np.int64)
    bc1 = 1.0 - beta1 ** step
    bc2 = 1.0 - beta2 ** step
    for i, n in enumerate(idx):
        gi = g[i] if th2 is None else g[i] * p2[n] * np.log(2.0)
        m2[n] = beta1 * m2[n] + (1.0 - beta1) * gi
        v2[n] = beta2 * v2[n] + (1.0 - beta2) * gi * gi
        upd = lr * (m2[n] / bc1) / (np.sqrt(v2[n] / bc2) + eps)
        if th2 is None:
            p2[n] = p2[n] - upd
        else:
            th2[n] = th2[n] - upd
            p2[n] = 2.0 ** th2[n]
    return (p2, m2, v2) if th2 is None else (p2, m2, v2, th2)


# ----------------------------------------------------------------------------
# convolution (NHWC activations, [N,R,S,C] weights, zero padding of x^)
# ----------------------------------------------------------------------------
def _patches(A, R, S, stride, pad):
    """[B,H,W,C] -> [B,Ho,Wo,R,S,C] of the zero-padded tensor."""
    B, H, Wd, C = A.shape
    Ho = (H + 2 * pad - R) // stride + 1
    Wo = (Wd + 2 * pad - S) // stride + 1
    Ap = np.zeros((B, H + 2 * pad, Wd + 2 * pad, C), dtype=F64)
    Ap[:, pad:pad + H, pad:pad + Wd, :] = A
    P = np.zeros((B, Ho, Wo, R, S, C), dtype=F64)
    for r in range(R):
        for s in range(S):
            P[:, :, :, r, s, :] = Ap[:, r:r + stride * Ho:stride, s:s + stride * Wo:stride, :]
    return P


def conv_forward(X, W, s_w, s_x, z_x, bias, w_bits, x_bits, stride=1, pad=0,
                 x_symmetric=False):
    """Y[b,ho,wo,n] = sum_{r,s,c} x^[b,ho*st+r-pad,wo*st+s-pad,c] w^[n,r,s,c] (+b[n]);
    padded positions contribute x^ = 0."""
    N, R, S, C = W.shape
    qx = fake_quant_x(X, s_x, z_x, x_bits, x_symmetric)
    qw = fake_quant_w(W, s_w, w_bits)
    P = _patches(qx["deq"], R, S, stride, pad)
    B, Ho, Wo = P.shape[:3]
    Y = P.reshape(B * Ho * Wo, R * S * C) @ qw["deq"].reshape(N, -1).T
    if bias is not None:
        Y = Y + np.asarray(bias, dtype=F64)[None, :]
    return Y.reshape(B, Ho, Wo, N)


def conv_backward_full(dY, X, W, s_w, s_x, z_x, w_bits, x_bits, stride=1, pad=0,
                       x_symmetric=False, operand_model="exact"):
    """Backward of the fake-quantised convolution: the two contractions of Eq. 5
    in their convolution form (input gradient = scatter of dY w^ back onto the
    padded input; weight gradient = dY^T patches(x^)), then the same masks and
    reductions as the linear layer."""
    N, R, S, C = W.shape
    B, H, Wd, _ = np.asarray(X).shape
    dYd = np.asarray(dY, dtype=F64)
    qx = fake_quant_x(X, s_x, z_x, x_bits, x_symmetric)
    qw = fake_quant_w(W, s_w, w_bits)
    What = qw["deq"]
    dYo = dYd
    if operand_model == "bf16":
        dYo = bf16_rne(dYd)
        s = np.asarray(s_w, dtype=F32).reshape(-1, 1, 1, 1)
        What = bf16_rne((s.astype(F64) * qw["q"]).astype(F32))
    Ho, Wo = dYd.shape[1:3]
    dY2 = dYo.reshape(B * Ho * Wo, N)
    # weight gradient
    P = _patches(qx["c0"], R, S, stride, pad).reshape(B * Ho * Wo, R * S * C)
    G_w = (F64(F32(s_x)) * (dY2.T @ P)).reshape(N, R, S, C)
    # input gradient: every output pixel adds dY w^ onto the input positions it read
    Gp = (dY2 @ What.reshape(N, -1)).reshape(B, Ho, Wo, R, S, C)
    G_xp = np.zeros((B, H + 2 * pad, Wd + 2 * pad, C), dtype=F64)
    for r in range(R):
        for s_ in range(S):
            G_xp[:, r:r + stride * Ho:stride, s_:s_ + stride * Wo:stride, :] += Gp[:, :, :, r, s_, :]
    G_x = G_xp[:, pad:pad + H, pad:pad + Wd, :]
    in_x = qx["flag"] == 0
    in_w = qw["flag"] == 0
    ax = tuple(range(1, 4))
    return dict(
        dX=np.where(in_x, G_x, 0.0), dW=np.where(in_w, G_w, 0.0),
        dS_x=(G_x * qx["t"]).sum(), dS_x_abs=np.abs(G_x * qx["t"]).sum(),
        dZ_x=(G_x * qx["dz"]).sum(), dZ_x_abs=np.abs(G_x * qx["dz"]).sum(),
        dS_w=(G_w * qw["t"]).sum(axis=ax), dS_w_abs=np.abs(G_w * qw["t"]).sum(axis=ax),
        db=dYd.reshape(-1, N).sum(axis=0),
    )


def conv_backward_efqat(dY, X, W, s_w, s_x, z_x, idx, w_bits, x_bits, stride=1, pad=0,
                        x_symmetric=False, operand_model="exact"):
    """EfQAT backward of the convolution: rows idx (output channels) of dW, dS_w."""
    full = conv_backward_full(dY, X, W, s_w, s_x, z_x, w_bits, x_bits, stride, pad,
                              x_symmetric, operand_model)
    idx = np.asarray(idx, dtype=np.int64)
    out = {k: full[k] for k in ("dX", "dS_x", "dS_x_abs", "dZ_x", "dZ_x_abs", "db")}
    out["dW_sel"] = full["dW"][idx]
    out["dS_w_sel"] = full["dS_w"][idx]
    out["dS_w_sel_abs"] = full["dS_w_abs"][idx]
    return out


def conv_backward_efqat_direct(dY, X, W, s_w, s_x, z_x, idx, w_bits, x_bits, stride=1, pad=0,
                               x_symmetric=False, operand_model="exact"):
    """Partial weight gradient of the convolution the way Algorithm 1 words it:
    take the output channels idx of dY and contract them with the patches of
    x^, never forming the other channels' rows.  Must agree with
    `conv_backward_efqat`.  Also returns the sums of absolute terms of the
    contraction and of the weight-scale reduction."""
    idx = np.asarray(idx, dtype=np.int64)
    Wa = np.asarray(W)
    N, R, S, C = Wa.shape
    dYd = np.asarray(dY, dtype=F64)[..., idx]
    if operand_model == "bf16":
        dYd = bf16_rne(dYd)
    elif operand_model != "exact":
        raise ValueError(operand_model)
    qx = fake_quant_x(X, s_x, z_x, x_bits, x_symmetric)
    qw = fake_quant_w(Wa[idx], np.asarray(s_w)[idx], w_bits)
    P = _patches(qx["c0"], R, S, stride, pad).reshape(-1, R * S * C)
    dY2 = dYd.reshape(int(np.prod(dYd.shape[:3])), len(idx))
    G = (F64(F32(s_x)) * (dY2.T @ P)).reshape(len(idx), R, S, C)
    G_abs = (F64(F32(s_x)) * (np.abs(dY2).T @ np.abs(P))).reshape(len(idx), R, S, C)
    ax = tuple(range(1, 4))
    return dict(dW_sel=np.where(qw["flag"] == 0, G, 0.0),
                dS_w_sel=(G * qw["t"]).sum(axis=ax),
                dS_w_sel_abs=np.abs(G * qw["t"]).sum(axis=ax),
                G_w_sel_abs=G_abs)
