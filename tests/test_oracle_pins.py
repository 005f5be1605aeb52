"""Pins for the fp64 oracle: each check ties one oracle function to something other
than itself -- hand-worked values (tests/golden), closed forms, brute-force loops,
invariants the paper states, or an independent library routine (torch autograd,
torch fake-quantize, torch SGD, torch conv2d, numpy argsort)."""
import os

import numpy as np
import pytest
import torch

from oracle import efqat_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quantizer_worked_example.txt")
rng = np.random.default_rng


# ---------------------------------------------------------------------------
# quantizer: hand-worked fixture, closed forms, ranges
# ---------------------------------------------------------------------------
def _golden_rows(tag):
    for line in open(GOLDEN):
        if line.startswith(tag + " "):
            yield [np.array(p.split(), dtype=np.float64) for p in line[1:].split("|")]


def test_golden_weight_rows():
    for w, s, q in _golden_rows("W"):
        W = w.astype(np.float32)[None, :]
        s_w = O.init_minmax_w(W, 8)
        assert s_w[0] == np.float32(s[0])
        out = O.fake_quant_w(W, s_w, 8)
        assert out["q"][0].tolist() == q.astype(int).tolist()
        assert not out["flag"].any()


def test_golden_activation_rows():
    for x, s, z, q in _golden_rows("X"):
        X = x.astype(np.float32)[None, :]
        s_x, z_x = O.init_minmax_x(X, 8)
        assert s_x == np.float32(s[0]) and z_x == np.float32(z[0])
        out = O.fake_quant_x(X, s_x, z_x, 8)
        assert out["q"][0].tolist() == q.astype(int).tolist()
        np.testing.assert_allclose(out["deq"][0], x, atol=1e-6)


def test_golden_clip_rows():
    for x, s, z, q, f in _golden_rows("C"):
        out = O.fake_quant_x(x.astype(np.float32), np.float32(s[0]), np.float32(z[0]), 4)
        assert out["q"].tolist() == q.astype(int).tolist()
        assert out["flag"].tolist() == f.astype(int).tolist()


@pytest.mark.parametrize("bits", [4, 8])
def test_power_of_two_scale_closed_form(bits):
    # x = s (j + delta): delta = .25 -> j, delta = +-.5 -> even neighbour
    s = np.float32(2.0 ** -5)
    Q = O.qmax_w(bits)
    j = np.arange(-Q + 1, Q - 1, dtype=np.float64)
    for delta, expect in ((0.25, j), (-0.25, j),
                          (0.5, np.where(j % 2 == 0, j, j + 1)),
                          (-0.5, np.where(j % 2 == 0, j, j - 1))):
        W = (float(s) * (j + delta)).astype(np.float32)[None, :]
        out = O.fake_quant_w(W, np.array([s]), bits)
        assert np.array_equal(out["q"][0], expect.astype(np.int32))
        np.testing.assert_array_equal(out["deq"][0], float(s) * expect)
    # beyond the range: boundary code and flag
    W = np.array([[-(Q + 3) * float(s), (Q + 0.6) * float(s), Q * float(s)]], dtype=np.float32)
    out = O.fake_quant_w(W, np.array([s]), bits)
    assert out["q"][0].tolist() == [-Q, Q, Q]
    assert out["flag"][0].tolist() == [1, 2, 0]


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("sym", [False, True])
def test_code_ranges_and_minmax_endpoints(bits, sym):
    r = rng(1)
    X = r.standard_normal((37, 29)).astype(np.float32) * 3
    W = r.standard_normal((11, 29)).astype(np.float32) * 0.02
    s_w = O.init_minmax_w(W, bits)
    qw = O.fake_quant_w(W, s_w, bits)
    Qw = O.qmax_w(bits)
    assert qw["q"].min() >= -Qw and qw["q"].max() <= Qw
    assert -(1 << (bits - 1)) <= qw["q"].min() and qw["q"].max() <= (1 << (bits - 1)) - 1
    # Eq. 4: the arg-max element of every row lands exactly on +-Qw and nothing clips
    am = np.abs(W).argmax(axis=1)
    assert np.all(np.abs(qw["q"][np.arange(11), am]) == Qw)
    assert not qw["flag"].any()
    s_x, z_x = O.init_minmax_x(X, bits, sym)
    qx = O.fake_quant_x(X, s_x, z_x, bits, sym)
    if sym:
        assert qx["q"].min() >= -Qw and qx["q"].max() <= Qw
        assert np.abs(qx["q"]).max() == Qw and z_x == 0
    else:
        # Eq. 2: min -> code 0, max -> code 2^b-1
        assert qx["q"].min() == 0 and qx["q"].max() == O.qmax_x(bits)
        assert qx["q"].flat[X.argmin()] == 0 and qx["q"].flat[X.argmax()] == O.qmax_x(bits)
    assert not qx["flag"].any()


def test_idempotence():
    r = rng(2)
    X = r.standard_normal((16, 24)).astype(np.float32)
    s_x, z_x = O.init_minmax_x(X, 8)
    a = O.fake_quant_x(X, s_x, z_x, 8)
    b = O.fake_quant_x(a["deq"].astype(np.float32), s_x, z_x, 8)
    assert np.array_equal(a["q"], b["q"]) and not b["flag"].any()


def test_u32_and_bf16_against_torch():
    r = rng(3)
    x = r.standard_normal(4096).astype(np.float32) * 7
    for s in (np.float32(0.0371), np.float32(1.0 / 3.0), np.float32(0.0101)):
        ours = O._u32(x, s)
        ref = (torch.from_numpy(x) * (torch.tensor(1.0, dtype=torch.float32) / torch.tensor(s))).numpy()
        assert np.array_equal(ours.view(np.uint32), ref.view(np.uint32))
    v = (r.standard_normal(8192) * np.exp(r.standard_normal(8192) * 4)).astype(np.float32)
    v[:4] = [1.00390625, 1.01171875, -1.00390625, 255.5]        # exact ties
    ref = torch.from_numpy(v).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.bf16_rne(v), ref)


def test_code_rule_against_literal_division_on_workload_inputs():
    """Eq. 1 / Eq. 3 write round(x / s).  The oracle (and the CUDA path) decide the code from
    fl32(x * fl32(1/s)) instead.  On the seeded inputs of the first two workload families the two
    rules may differ only where x/s sits within an fp32 rounding of a tie: at most one code in
    1e5, and never by more than one step."""
    from paper_2411_11038_b200 import inputs as I
    for case in I.config1() + I.config2()[:2]:
        T = I.make_tensors(case)
        X, W = I.as_f64(T["X"]), I.as_f64(T["W"])
        s_w = O.init_minmax_w(W, case.w_bits)
        s_x, z_x = O.init_minmax_x(X, case.x_bits, case.x_symmetric)
        for fx, fw in ((1.0, 1.0), (0.8, 0.85)):          # at the MinMax start and after the scales moved
            sx = np.float32(s_x * np.float32(fx))
            sw = (s_w * np.float32(fw)).astype(np.float32)
            qx = O.fake_quant_x(X, sx, z_x, case.x_bits, case.x_symmetric)
            lo, hi = (-O.qmax_w(case.x_bits), O.qmax_w(case.x_bits)) if case.x_symmetric else (0, O.qmax_x(case.x_bits))
            lit = np.clip(np.rint(X / np.float64(sx)) + qx["Zr"], lo, hi)
            d = np.abs(qx["q"] - lit)
            assert d.max() <= 1 and (d != 0).mean() <= 1e-5, (case.name, "x", d.max(), (d != 0).mean())
            qw = O.fake_quant_w(W, sw, case.w_bits)
            Q = O.qmax_w(case.w_bits)
            lit = np.clip(np.rint(W / sw.astype(np.float64)[:, None]), -Q, Q)
            d = np.abs(qw["q"] - lit)
            assert d.max() <= 1 and (d != 0).mean() <= 1e-5, (case.name, "w", d.max(), (d != 0).mean())


def test_fake_quant_matches_torch_fake_quantize():
    r = rng(4)
    X = torch.from_numpy(r.standard_normal((33, 17)).astype(np.float32) * 2)
    s, z = np.float32(0.03), np.float32(117)
    ref = torch.fake_quantize_per_tensor_affine(X, float(s), int(z), 0, 255).numpy()
    out = O.fake_quant_x(X.numpy(), s, z, 8)
    np.testing.assert_allclose(out["deq"], ref, rtol=0, atol=1e-6)
    assert out["flag"].any()            # the case does clip
    W = torch.from_numpy(r.standard_normal((9, 17)).astype(np.float32))
    sw = torch.from_numpy((r.random(9).astype(np.float32) + 0.5) * 0.01)
    ref = torch.fake_quantize_per_channel_affine(W, sw, torch.zeros(9, dtype=torch.int32), 0, -7, 7).numpy()
    out = O.fake_quant_w(W.numpy(), sw.numpy(), 4)
    np.testing.assert_allclose(out["deq"], ref, rtol=0, atol=1e-7)


# ---------------------------------------------------------------------------
# importance and selection
# ---------------------------------------------------------------------------
def test_importance_closed_forms():
    W = np.full((3, 64), -0.375, dtype=np.float32)
    assert np.all(O.importance_rows(W) == np.float32(0.375))
    W = np.where(rng(5).random((4, 33)) < 0.5, -1.0, 1.0).astype(np.float32)
    assert np.all(O.importance_rows(W) == 1.0)
    W = rng(6).standard_normal((5, 7)).astype(np.float32)
    brute = [sum(abs(float(v)) for v in row) / 7 for row in W]
    np.testing.assert_allclose(O.importance_rows(W), brute, rtol=1e-7)
    assert O.importance_layer(W) == np.float32(sum(sum(abs(float(v)) for v in row) for row in W) / 35)
    # a 4-d conv weight is ranked by output channel over all of R*S*C
    Wc = rng(7).standard_normal((6, 3, 3, 4)).astype(np.float32)
    np.testing.assert_array_equal(O.importance_rows(Wc), O.importance_rows(Wc.reshape(6, 36)))


def _brute_topk(keys, k):
    # repeated arg-max with smallest-index tie-break
    left = list(range(len(keys)))
    out = []
    for _ in range(k):
        best = left[0]
        for i in left:
            if keys[i] > keys[best]:
                best = i
        out.append(best)
        left.remove(best)
    return sorted(out)


def test_select_topk_brute_force_with_ties():
    r = rng(8)
    for n in (1, 2, 7, 16, 33):
        keys = r.integers(0, 5, n).astype(np.float32) / 4          # many ties
        for k in range(n + 1):
            got = O.select_topk(keys, k)
            assert got.tolist() == _brute_topk(keys.tolist(), k)
            assert got.dtype == np.int32
    assert O.select_topk(np.ones(9, np.float32), 4).tolist() == [0, 1, 2, 3]
    assert O.select_topk(np.ones(9, np.float32), 0).tolist() == []
    assert O.select_topk(np.ones(9, np.float32), 9).tolist() == list(range(9))


def test_select_topk_matches_argsort_on_distinct_keys():
    r = rng(9)
    keys = r.permutation(200).astype(np.float32) / 7
    for k in (1, 10, 199):
        ref = np.sort(np.argsort(-keys, kind="stable")[:k])
        assert np.array_equal(O.select_topk(keys, k), ref)
    # invariance under a common positive factor (Eq. 6 is homogeneous)
    W = r.standard_normal((40, 16)).astype(np.float32)
    assert np.array_equal(O.select_cwpl([W], [7])[0], O.select_cwpl([2 * W], [7])[0])


def test_modes():
    r = rng(10)
    Ws = [r.standard_normal((n, k)).astype(np.float32) * sc
          for n, k, sc in ((8, 16, 1.0), (12, 8, 1.5), (6, 32, 0.5))]
    # CWPN with a single layer is CWPL
    assert np.array_equal(O.select_cwpn([Ws[0]], 3)[0], O.select_cwpl([Ws[0]], [3])[0])
    # CWPN = global top-k on the concatenated keys, split per layer
    keys = np.concatenate([O.importance_rows(W) for W in Ws])
    g = _brute_topk(keys.tolist(), 9)
    got = O.select_cwpn(Ws, 9)
    offs = [0, 8, 20, 26]
    flat = [int(i) + offs[l] for l in range(3) for i in got[l]]
    assert flat == g and sum(len(x) for x in got) == 9
    # the large-scale layer wins most channels, the small-scale layer none
    assert len(got[1]) > len(got[0]) >= len(got[2])
    # LWPN: whole layers, ranked by the layer mean
    lw = O.select_lwpn(Ws, 1)
    assert [len(x) for x in lw] == [0, 12, 0] and lw[1].tolist() == list(range(12))
    assert [len(x) for x in O.select_lwpn(Ws, 0)] == [0, 0, 0]
    assert [len(x) for x in O.select_lwpn(Ws, 3)] == [8, 12, 6]
    assert O.ratio_to_k(0.05, 512) == 25 and O.ratio_to_k(0.1, 221184) == 22118
    assert O.ratio_to_k(1.0, 768) == 768 and O.ratio_to_k(0.0, 768) == 0


# ---------------------------------------------------------------------------
# forward / backward contractions
# ---------------------------------------------------------------------------
def _tiny(seed, M=5, K=6, N=4, clip=False):
    r = rng(seed)
    X = r.standard_normal((M, K)).astype(np.float32)
    W = (r.standard_normal((N, K)) * 0.05).astype(np.float32)
    dY = r.standard_normal((M, N)).astype(np.float32)
    s_w = O.init_minmax_w(W, 8)
    s_x, z_x = O.init_minmax_x(X, 8)
    if clip:                       # shrink the ranges so that both tensors clip
        s_w = (s_w * 0.6).astype(np.float32)
        s_x = np.float32(s_x * 0.7)
        z_x = np.float32(z_x + 9.3)          # non-integer learnt zero point
    return X, W, dY, s_w, s_x, z_x


def test_forward_is_plain_matmul_on_grid():
    # inputs on the quantisation grid with power-of-two scales: fake-quant is the identity
    r = rng(11)
    s_x, s_w = np.float32(2.0 ** -4), np.full(7, 2.0 ** -6, np.float32)
    X = (r.integers(0, 256, (9, 12)) - 100).astype(np.float32) * s_x
    W = r.integers(-127, 128, (7, 12)).astype(np.float32) * s_w[0]
    b = r.standard_normal(7).astype(np.float32)
    Y = O.forward(X, W, s_w, s_x, np.float32(100), b, 8, 8)
    np.testing.assert_array_equal(Y, X.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64))


def test_forward_backward_brute_force_loops():
    X, W, dY, s_w, s_x, z_x = _tiny(12, clip=True)
    M, K = X.shape
    N = W.shape[0]
    qx = O.fake_quant_x(X, s_x, z_x, 8)
    qw = O.fake_quant_w(W, s_w, 8)
    assert qx["flag"].any() and qw["flag"].any()
    Y = O.forward(X, W, s_w, s_x, z_x, None, 8, 8)
    full = O.backward_full(dY, X, W, s_w, s_x, z_x, 8, 8)
    for m in range(M):
        for n in range(N):
            y = sum(qx["deq"][m, k] * qw["deq"][n, k] for k in range(K))
            assert abs(Y[m, n] - y) < 1e-12
    dS_x = dZ_x = 0.0
    for m in range(M):
        for k in range(K):
            g = sum(float(dY[m, n]) * qw["deq"][n, k] for n in range(N))
            assert abs(full["dX"][m, k] - (g if qx["flag"][m, k] == 0 else 0.0)) < 1e-12
            dS_x += g * qx["t"][m, k]
            dZ_x += g * qx["dz"][m, k]
    assert abs(full["dS_x"] - dS_x) < 1e-10 and abs(full["dZ_x"] - dZ_x) < 1e-10
    for n in range(N):
        ds = 0.0
        for k in range(K):
            g = sum(float(dY[m, n]) * qx["deq"][m, k] for m in range(M))
            assert abs(full["dW"][n, k] - (g if qw["flag"][n, k] == 0 else 0.0)) < 1e-12
            ds += g * qw["t"][n, k]
        assert abs(full["dS_w"][n] - ds) < 1e-10
        assert abs(full["db"][n] - sum(float(dY[m, n]) for m in range(M))) < 1e-12


def test_backward_matches_torch_autograd_through_learnable_fake_quant():
    """Independent library routine: torch's learnable fake-quantize ops carry the
    straight-through gradient for the input, the scale and the zero point."""
    X, W, dY, s_w, s_x, z_x = _tiny(13, M=12, K=10, N=6, clip=True)
    z_int = np.float32(np.clip(np.rint(z_x), 0, 255))
    Xt = torch.tensor(X, dtype=torch.float32, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.float32, requires_grad=True)
    sx = torch.tensor([float(s_x)], requires_grad=True)
    zx = torch.tensor([float(z_int)], requires_grad=True)
    sw = torch.tensor(s_w, requires_grad=True)
    zw = torch.zeros(6, requires_grad=True)
    Xh = torch._fake_quantize_learnable_per_tensor_affine(Xt, sx, zx, 0, 255, 1.0)
    Wh = torch._fake_quantize_learnable_per_channel_affine(Wt, sw, zw, 0, -127, 127, 1.0)
    Y = Xh @ Wh.T
    Y.backward(torch.tensor(dY))
    full = O.backward_full(dY, X, W, s_w, s_x, z_int, 8, 8)
    tol = dict(rtol=2e-5, atol=2e-5)
    np.testing.assert_allclose(O.forward(X, W, s_w, s_x, z_int, None, 8, 8), Y.detach().numpy(), **tol)
    np.testing.assert_allclose(full["dX"], Xt.grad.numpy(), **tol)
    np.testing.assert_allclose(full["dW"], Wt.grad.numpy(), **tol)
    np.testing.assert_allclose(full["dS_x"], sx.grad.item(), rtol=1e-4, atol=1e-3)
    np.testing.assert_allclose(full["dZ_x"], zx.grad.item(), rtol=1e-4, atol=1e-4)
    np.testing.assert_allclose(full["dS_w"], sw.grad.numpy(), rtol=1e-4, atol=1e-2)
    assert np.count_nonzero(full["dX"] == 0) > 0 and np.count_nonzero(full["dW"] == 0) > 0


def test_ste_surrogate_finite_differences():
    """dS and dZ against central differences of the straight-through surrogate:
    the rounding residual rho = rne(u0) - u0 is frozen at the base point."""
    X, W, dY, s_w, s_x, z_x = _tiny(14, M=9, K=8, N=5, clip=True)
    X64, W64, dY64 = X.astype(np.float64), W.astype(np.float64), dY.astype(np.float64)
    Zr = float(np.clip(np.rint(z_x), 0, 255))
    rho_x = np.rint(X64 / float(s_x)) - X64 / float(s_x)
    sw64 = s_w.astype(np.float64)[:, None]
    rho_w = np.rint(W64 / sw64) - W64 / sw64

    def xhat(s, Z):
        return s * (np.clip(X64 / s + rho_x + Z, 0, 255) - Z)

    def what(sv):
        return sv * np.clip(W64 / sv + rho_w, -127, 127)

    def loss(s, Z, sv):
        return float((dY64 * (xhat(s, Z) @ what(sv).T)).sum())

    full = O.backward_full(dY, X, W, s_w, s_x, z_x, 8, 8)
    h = 1e-7
    fd = (loss(float(s_x) + h, Zr, sw64) - loss(float(s_x) - h, Zr, sw64)) / (2 * h)
    assert abs(fd - full["dS_x"]) <= 1e-5 * full["dS_x_abs"] + 1e-6
    hz = 1e-4
    fd = (loss(float(s_x), Zr + hz, sw64) - loss(float(s_x), Zr - hz, sw64)) / (2 * hz)
    assert abs(fd - full["dZ_x"]) <= 1e-6 * full["dZ_x_abs"] + 1e-8
    for n in range(5):
        e = np.zeros_like(sw64)
        e[n] = 1e-9
        fd = (loss(float(s_x), Zr, sw64 + e) - loss(float(s_x), Zr, sw64 - e)) / 2e-9
        assert abs(fd - full["dS_w"][n]) <= 1e-4 * full["dS_w_abs"][n] + 1e-5
    # all weights exactly on the grid -> in-range t_w = q - u = 0 -> dS_w = 0
    Wg = (np.rint(W64 / sw64) * sw64).astype(np.float32)
    s2 = np.full(5, 2.0 ** -8, np.float32)
    Wg = (rng(0).integers(-100, 100, W.shape) * 2.0 ** -8).astype(np.float32)
    assert np.all(O.backward_full(dY, X, Wg, s2, s_x, z_x, 8, 8)["dS_w"] == 0)


def test_efqat_invariants():
    X, W, dY, s_w, s_x, z_x = _tiny(15, M=14, K=9, N=8, clip=True)
    full = O.backward_full(dY, X, W, s_w, s_x, z_x, 8, 8)
    idx_all = np.arange(8)
    a = O.backward_efqat(dY, X, W, s_w, s_x, z_x, idx_all, 8, 8)
    # 100 % unfrozen is ordinary QAT backward
    assert np.array_equal(a["dW_sel"], full["dW"]) and np.array_equal(a["dS_w_sel"], full["dS_w"])
    # 0 %: only dX and the activation quantisation parameters (and db) remain
    z = O.backward_efqat(dY, X, W, s_w, s_x, z_x, [], 8, 8)
    assert z["dW_sel"].shape == (0, 9) and z["dS_w_sel"].shape == (0,)
    for idx in ([], [3], [0, 5, 7], idx_all):
        e = O.backward_efqat(dY, X, W, s_w, s_x, z_x, idx, 8, 8)
        d = O.backward_efqat_direct(dY, X, W, s_w, s_x, z_x, idx, 8, 8)
        # rows of the brute-force full dW, and the "extract columns of dY" wording agree
        assert np.array_equal(e["dW_sel"], full["dW"][list(idx)])
        np.testing.assert_allclose(d["dW_sel"], e["dW_sel"], rtol=0, atol=1e-12)
        np.testing.assert_allclose(d["dS_w_sel"], e["dS_w_sel"], rtol=0, atol=1e-12)
        # the input gradient and the activation-parameter gradients never depend on idx
        assert np.array_equal(e["dX"], full["dX"])
        assert e["dS_x"] == full["dS_x"] and e["dZ_x"] == full["dZ_x"]
    # linear in dY
    b = O.backward_full(2.0 * dY, X, W, s_w, s_x, z_x, 8, 8)
    np.testing.assert_allclose(b["dX"], 2 * full["dX"], rtol=1e-13)
    np.testing.assert_allclose(b["dW"], 2 * full["dW"], rtol=1e-13)


def test_ste_mask_extremes():
    X, W, dY, s_w, s_x, z_x = _tiny(16, M=6, K=7, N=5)
    # every activation out of range -> dX = 0 and dS_x = sum G_x (boundary - Zr)
    Xbig = (np.abs(X) + 1.0).astype(np.float32) * 1e3
    full = O.backward_full(dY, Xbig, W, s_w, s_x, z_x, 8, 8)
    assert np.all(full["dX"] == 0)
    G = dY.astype(np.float64) @ O.fake_quant_w(W, s_w, 8)["deq"]
    Zr = float(np.clip(np.rint(z_x), 0, 255))
    np.testing.assert_allclose(full["dS_x"], (G * (255 - Zr)).sum(), rtol=1e-12)
    np.testing.assert_allclose(full["dZ_x"], (G * -float(s_x)).sum(), rtol=1e-12)
    # nothing clipped -> dX = G_x, dZ_x = 0
    full = O.backward_full(dY, X, W, s_w, s_x, z_x, 8, 8)
    np.testing.assert_array_equal(full["dX"], G)
    assert full["dZ_x"] == 0


def test_bf16_operand_model_is_close_and_distinct():
    X, W, dY, s_w, s_x, z_x = _tiny(17, M=32, K=24, N=16)
    e = O.backward_full(dY, X, W, s_w, s_x, z_x, 8, 8, operand_model="exact")
    b = O.backward_full(dY, X, W, s_w, s_x, z_x, 8, 8, operand_model="bf16")
    assert np.abs(b["dX"] - e["dX"]).max() <= 1e-2 * np.abs(e["dX"]).max()
    assert np.abs(b["dW"] - e["dW"]).max() <= 1e-2 * np.abs(e["dW"]).max()
    assert not np.array_equal(b["dX"], e["dX"])
    # bf16 inputs make the two models agree on G_w exactly (dY already on the grid)
    dYb = torch.tensor(dY).to(torch.bfloat16).to(torch.float32).numpy()
    e = O.backward_full(dYb, X, W, s_w, s_x, z_x, 8, 8, operand_model="exact")
    b = O.backward_full(dYb, X, W, s_w, s_x, z_x, 8, 8, operand_model="bf16")
    assert np.array_equal(b["dW"], e["dW"])


def test_direct_partial_backward_operand_model_and_abs_sums():
    """The restricted loop of Algorithm 1 under the bf16 operand model and its abs-sums equal
    the matching rows of the full backward under the same model."""
    X, W, dY, s_w, s_x, z_x = _tiny(31, M=40, K=24, N=16, clip=True)
    idx = [1, 4, 5, 11, 15]
    for model in ("exact", "bf16"):
        e = O.backward_efqat(dY, X, W, s_w, s_x, z_x, idx, 8, 8, operand_model=model)
        d = O.backward_efqat_direct(dY, X, W, s_w, s_x, z_x, idx, 8, 8, operand_model=model)
        for key in ("dW_sel", "dS_w_sel", "dS_w_sel_abs", "G_w_sel_abs"):
            np.testing.assert_allclose(d[key], e[key], rtol=1e-13, atol=1e-13, err_msg=f"{model} {key}")
    # the abs-sums are what they say: sums of |terms| of the plain loops
    c0 = O.fake_quant_x(X, s_x, z_x, 8)["c0"]
    brute = np.array([[sum(abs(float(dY[m, n]) * c0[m, k]) for m in range(40)) for k in range(24)] for n in idx])
    exact = O.backward_efqat_direct(dY, X, W, s_w, s_x, z_x, idx, 8, 8)
    np.testing.assert_allclose(exact["G_w_sel_abs"], float(s_x) * brute, rtol=1e-12)


def test_sgd_rows_against_torch_sgd():
    r = rng(18)
    W = r.standard_normal((7, 5))
    V = r.standard_normal((7, 5)) * 0.1
    idx = [1, 4, 6]
    g = r.standard_normal((3, 5))
    W2, V2 = O.sgd_rows(W, V, g, idx, lr=0.1, momentum=0.9, weight_decay=1e-4)
    frozen = [0, 2, 3, 5]
    assert np.array_equal(W2[frozen], W[frozen]) and np.array_equal(V2[frozen], V[frozen])
    # hand recurrence
    v = 0.9 * V[4] + g[1] + 1e-4 * W[4]
    np.testing.assert_allclose(V2[4], v, rtol=1e-15)
    np.testing.assert_allclose(W2[4], W[4] - 0.1 * v, rtol=1e-15)
    # torch.optim.SGD on the selected rows alone
    p = torch.tensor(W[idx], dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=0.1, momentum=0.9, weight_decay=1e-4)
    opt.state[p]["momentum_buffer"] = torch.tensor(V[idx], dtype=torch.float64)
    p.grad = torch.tensor(g, dtype=torch.float64)
    opt.step()
    np.testing.assert_allclose(W2[idx], p.detach().numpy(), rtol=1e-14)


def test_adam_qparams_against_torch_adam():
    """Three Adam steps on a subset of entries equal torch.optim.Adam on those entries alone;
    the other entries and their moments never move.  With the log2 parameterisation the same
    holds for theta with the gradient that autograd sends through p = 2^theta."""
    r = rng(51)
    p0 = r.random(9) * 0.05 + 0.01
    idx = [0, 3, 4, 8]
    frozen = [1, 2, 5, 6, 7]
    grads = [r.standard_normal(4) * 10 ** r.uniform(-3, 2) for _ in range(3)]
    kw = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)
    # raw parameters
    p, m, v = p0.copy(), np.zeros(9), np.zeros(9)
    tp = torch.tensor(p0[idx], dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([tp], lr=1e-3, betas=(0.9, 0.999), eps=1e-8)
    for t, g in enumerate(grads, 1):
        p, m, v = O.adam_qparams(p, m, v, g, idx, t, **kw)
        tp.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(p[idx], tp.detach().numpy(), rtol=1e-12)
        np.testing.assert_allclose(m[idx], opt.state[tp]["exp_avg"].numpy(), rtol=1e-12)
        np.testing.assert_allclose(v[idx], opt.state[tp]["exp_avg_sq"].numpy(), rtol=1e-12)
        assert np.array_equal(p[frozen], p0[frozen]) and not m[frozen].any() and not v[frozen].any()
    # first step by hand: m^ = g, v^ = g^2, so the step is lr * sign(g) up to eps
    p1, _, _ = O.adam_qparams(p0, np.zeros(9), np.zeros(9), grads[0], idx, 1, **kw)
    np.testing.assert_allclose(p1[idx], p0[idx] - 1e-3 * grads[0] / (np.abs(grads[0]) + 1e-8), rtol=1e-12)
    # log2 parameterisation: torch differentiates through p = 2^theta
    p, m, v, th = p0.copy(), np.zeros(9), np.zeros(9), np.log2(p0)
    tth = torch.tensor(np.log2(p0[idx]), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([tth], lr=1e-3, betas=(0.9, 0.999), eps=1e-8)
    for t, g in enumerate(grads, 1):
        p, m, v, th = O.adam_qparams(p, m, v, g, idx, t, theta=th, **kw)
        opt.zero_grad()
        (torch.pow(2.0, tth) * torch.tensor(g, dtype=torch.float64)).sum().backward()     # dL/dp = g
        opt.step()
        np.testing.assert_allclose(th[idx], tth.detach().numpy(), rtol=1e-12)
        np.testing.assert_allclose(p[idx], 2.0 ** tth.detach().numpy(), rtol=1e-12)
        assert np.array_equal(p[frozen], p0[frozen]) and np.all(p > 0)
    # scalar form (activation scale / zero point): idx = None updates every entry
    q, mq, vq = O.adam_qparams([0.02], [0.0], [0.0], [3.0], None, 1, **kw)
    np.testing.assert_allclose(q, [0.02 - 1e-3 * 3.0 / (3.0 + 1e-8)], rtol=1e-12)


# ---------------------------------------------------------------------------
# convolution
# ---------------------------------------------------------------------------
def _conv_case(seed, B=2, H=5, Wd=6, C=3, N=4, R=3, clip=True):
    r = rng(seed)
    X = np.abs(r.standard_normal((B, H, Wd, C))).astype(np.float32)
    W = (r.standard_normal((N, R, R, C)) * 0.1).astype(np.float32)
    s_w = O.init_minmax_w(W, 4)
    s_x, z_x = O.init_minmax_x(X - 0.3, 8)              # asymmetric: Z != 0, and X clips
    if clip:
        s_w = (s_w * 0.8).astype(np.float32)
    return X, W, s_w, s_x, z_x


def test_conv_1x1_is_linear():
    X, W, s_w, s_x, z_x = _conv_case(19, R=1)
    B, H, Wd, C = X.shape
    dY = rng(20).standard_normal((B, H, Wd, 4)).astype(np.float32)
    Yc = O.conv_forward(X, W, s_w, s_x, z_x, None, 4, 8)
    Yl = O.forward(X.reshape(-1, C), W.reshape(4, C), s_w, s_x, z_x, None, 4, 8)
    assert np.array_equal(Yc.reshape(-1, 4), Yl)
    bc = O.conv_backward_full(dY, X, W, s_w, s_x, z_x, 4, 8)
    bl = O.backward_full(dY.reshape(-1, 4), X.reshape(-1, C), W.reshape(4, C), s_w, s_x, z_x, 4, 8)
    np.testing.assert_allclose(bc["dX"].reshape(-1, C), bl["dX"], atol=1e-12)
    np.testing.assert_allclose(bc["dW"].reshape(4, C), bl["dW"], atol=1e-12)
    np.testing.assert_allclose(bc["dS_x"], bl["dS_x"], atol=1e-10)
    np.testing.assert_allclose(bc["dS_w"], bl["dS_w"], atol=1e-10)


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 1), (1, 0)])
def test_conv_3x3_against_torch_conv2d_and_adjointness(stride, pad):
    X, W, s_w, s_x, z_x = _conv_case(21)
    qx = O.fake_quant_x(X, s_x, z_x, 8)
    qw = O.fake_quant_w(W, s_w, 4)
    assert qx["Zr"] != 0 and qx["flag"].any() and qw["flag"].any()
    xh = torch.tensor(qx["deq"]).permute(0, 3, 1, 2).requires_grad_(True)       # NCHW
    wh = torch.tensor(qw["deq"]).permute(0, 3, 1, 2).requires_grad_(True)       # N C R S
    Yt = torch.nn.functional.conv2d(xh, wh, stride=stride, padding=pad)
    Y = O.conv_forward(X, W, s_w, s_x, z_x, None, 4, 8, stride, pad)
    np.testing.assert_allclose(Y, Yt.detach().permute(0, 2, 3, 1).numpy(), atol=1e-12)
    dY = rng(22).standard_normal(Y.shape)
    Yt.backward(torch.tensor(dY).permute(0, 3, 1, 2))
    full = O.conv_backward_full(dY, X, W, s_w, s_x, z_x, 4, 8, stride, pad)
    Gx = xh.grad.permute(0, 2, 3, 1).numpy()
    Gw = wh.grad.permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(full["dX"], np.where(qx["flag"] == 0, Gx, 0), atol=1e-12)
    np.testing.assert_allclose(full["dW"], np.where(qw["flag"] == 0, Gw, 0), atol=1e-12)
    np.testing.assert_allclose(full["dS_x"], (Gx * qx["t"]).sum(), atol=1e-10)
    np.testing.assert_allclose(full["dS_w"], (Gw * qw["t"]).sum(axis=(1, 2, 3)), atol=1e-10)
    # adjointness <dY, conv(x^, w^)> = <dgrad, x^> = <wgrad, w^>
    lhs = (dY * Y).sum()
    np.testing.assert_allclose((Gx * qx["deq"]).sum(), lhs, rtol=1e-12)
    np.testing.assert_allclose((Gw * qw["deq"]).sum(), lhs, rtol=1e-12)
    e = O.conv_backward_efqat(dY, X, W, s_w, s_x, z_x, [0, 2], 4, 8, stride, pad)
    assert np.array_equal(e["dW_sel"], full["dW"][[0, 2]])


def test_conv_brute_force_seven_loops():
    X, W, s_w, s_x, z_x = _conv_case(23, B=1, H=4, Wd=3, C=2, N=2)
    qx = O.fake_quant_x(X, s_x, z_x, 8)["deq"]
    qw = O.fake_quant_w(W, s_w, 4)["deq"]
    Y = O.conv_forward(X, W, s_w, s_x, z_x, None, 4, 8, 1, 1)
    for h in range(4):
        for w in range(3):
            for n in range(2):
                acc = 0.0
                for r in range(3):
                    for s in range(3):
                        hh, ww = h + r - 1, w + s - 1
                        if 0 <= hh < 4 and 0 <= ww < 3:
                            for c in range(2):
                                acc += qx[0, hh, ww, c] * qw[n, r, s, c]
                assert abs(Y[0, h, w, n] - acc) < 1e-12


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 1)])
def test_conv_bf16_operand_model_against_torch_on_rounded_operands(stride, pad):
    """The 'bf16' operand model of the convolution backward = the exact backward evaluated by an
    independent routine (torch conv2d autograd, fp64) on operands rounded by torch itself: dY to
    bf16 and, for the input gradient only, w^ to bf16(fl32(s_w q_w)) with s_w per OUTPUT channel."""
    X, W, s_w, s_x, z_x = _conv_case(41, B=2, H=6, Wd=5, C=4, N=6)
    s_w = (s_w * (1.0 + 0.37 * np.arange(6))).astype(np.float32)      # distinct scales: a wrong axis shows
    qx = O.fake_quant_x(X, s_x, z_x, 8)
    qw = O.fake_quant_w(W, s_w, 4)
    Y = O.conv_forward(X, W, s_w, s_x, z_x, None, 4, 8, stride, pad)
    dY = rng(42).standard_normal(Y.shape)
    b = O.conv_backward_full(dY, X, W, s_w, s_x, z_x, 4, 8, stride, pad, operand_model="bf16")
    e = O.conv_backward_full(dY, X, W, s_w, s_x, z_x, 4, 8, stride, pad, operand_model="exact")
    dYb = torch.tensor(dY, dtype=torch.float32).to(torch.bfloat16).to(torch.float64)
    wb = (torch.tensor(s_w).reshape(-1, 1, 1, 1) * torch.tensor(qw["q"], dtype=torch.float32)) \
        .to(torch.bfloat16).to(torch.float64)
    # input gradient: dY_b against the rounded dequantised weights
    xh = torch.tensor(qx["deq"]).permute(0, 3, 1, 2).requires_grad_(True)
    torch.nn.functional.conv2d(xh, wb.permute(0, 3, 1, 2), stride=stride, padding=pad) \
        .backward(dYb.permute(0, 3, 1, 2))
    Gx = xh.grad.permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(b["dX"], np.where(qx["flag"] == 0, Gx, 0), atol=1e-12)
    np.testing.assert_allclose(b["dS_x"], (Gx * qx["t"]).sum(), atol=1e-10)
    np.testing.assert_allclose(b["dZ_x"], (Gx * qx["dz"]).sum(), atol=1e-10)
    # weight gradient: dY_b against the exact integer activations, s_x applied afterwards
    wh = torch.zeros(W.shape, dtype=torch.float64).permute(0, 3, 1, 2).contiguous().requires_grad_(True)
    xc = torch.tensor(qx["c0"]).permute(0, 3, 1, 2)
    torch.nn.functional.conv2d(xc, wh, stride=stride, padding=pad).backward(dYb.permute(0, 3, 1, 2))
    Gw = float(s_x) * wh.grad.permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(b["dW"], np.where(qw["flag"] == 0, Gw, 0), atol=1e-12)
    np.testing.assert_allclose(b["dS_w"], (Gw * qw["t"]).sum(axis=(1, 2, 3)), atol=1e-10)
    # close to, and distinct from, the exact model; db never depends on the model
    assert np.abs(b["dX"] - e["dX"]).max() <= 1e-2 * np.abs(e["dX"]).max()
    assert not np.array_equal(b["dX"], e["dX"]) and np.array_equal(b["db"], e["db"])


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 1)])
def test_conv_direct_partial_backward_equals_rows_of_full(stride, pad):
    X, W, s_w, s_x, z_x = _conv_case(43, B=2, H=6, Wd=5, C=4, N=6)
    Y = O.conv_forward(X, W, s_w, s_x, z_x, None, 4, 8, stride, pad)
    dY = rng(44).standard_normal(Y.shape)
    for idx in ([], [2], [0, 3, 5]):
        for model in ("exact", "bf16"):
            e = O.conv_backward_efqat(dY, X, W, s_w, s_x, z_x, idx, 4, 8, stride, pad, operand_model=model)
            d = O.conv_backward_efqat_direct(dY, X, W, s_w, s_x, z_x, idx, 4, 8, stride, pad, operand_model=model)
            for key in ("dW_sel", "dS_w_sel", "dS_w_sel_abs"):
                np.testing.assert_allclose(d[key], e[key], rtol=1e-13, atol=1e-13)
            assert np.all(d["G_w_sel_abs"] >= np.abs(d["dW_sel"]) - 1e-12)
