"""GPU tests of the building blocks through the C ABI: the tensor-core contraction in its
four operand layouts, the quantizer exports (bit-exact against the oracle), the MinMax
initialisation and the Top-K selection modes (index sets bit-exact)."""
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


# ---------------------------------------------------------------------------
# tensor-core contraction: small-integer operands make every fp32 sum exact
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 1), (1, 0)])
@pytest.mark.parametrize("M,N,K,splits", [(128, 64, 64, 1), (256, 256, 512, 1), (136, 72, 200, 1),
                                           (384, 48, 1000, 3), (128, 16, 4096, 8), (520, 328, 264, 2)])
def test_gemm_core_exact_on_integers(ctx, a_mn, b_mn, M, N, K, splits):
    g = torch.Generator().manual_seed(M * 7 + N * 3 + K + a_mn * 2 + b_mn)
    A = torch.randint(-8, 9, (M, K), generator=g).float()
    Bm = torch.randint(-8, 9, (N, K), generator=g).float()
    ref = (A.double() @ Bm.double().T).numpy()                          # [M,N]
    A_st = (A.T if a_mn else A).contiguous().to(torch.bfloat16).cuda()
    B_st = (Bm.T if b_mn else Bm).contiguous().to(torch.bfloat16).cuda()
    out = B.gemm_bf16(ctx, A_st, B_st, M, N, K, a_mn, b_mn, splits)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    got = out.double().sum(dim=0).cpu().numpy().T                       # slabs are [N,M]
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("splits", [1, 3])
def test_gemm_core_cta_pairs_exact_on_integers(ctx, splits):
    """Both operands MN-major and 64 output tiles of 256 x 256: the shape class for which the
    partial-product GEMM runs on CTA pairs (cta_group::2), with and without a split contraction."""
    M, N, K = 2048, 2048, 1024
    g = torch.Generator().manual_seed(77 + splits)
    A = torch.randint(-4, 5, (M, K), generator=g).float()
    Bm = torch.randint(-4, 5, (N, K), generator=g).float()
    ref = (A.double() @ Bm.double().T).numpy()
    A_st = A.T.contiguous().to(torch.bfloat16).cuda()
    B_st = Bm.T.contiguous().to(torch.bfloat16).cuda()
    out = B.gemm_bf16(ctx, A_st, B_st, M, N, K, 1, 1, splits)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    got = out.double().sum(dim=0).cpu().numpy().T
    assert np.array_equal(got, ref)


def test_gemm_core_random_bf16(ctx):
    g = torch.Generator().manual_seed(5)
    M, N, K = 640, 392, 1096
    A = torch.randn((M, K), generator=g).to(torch.bfloat16)
    Bm = torch.randn((K, N), generator=g).to(torch.bfloat16)           # stored [K,N]: b_mn = 1
    out = B.gemm_bf16(ctx, A.cuda(), Bm.cuda(), M, N, K, 0, 1, 1)
    torch.cuda.synchronize()
    got = out[0].cpu().numpy().T.astype(np.float64)
    ref = A.double().numpy() @ Bm.double().numpy()
    abs_sum = np.abs(A.double().numpy()) @ np.abs(Bm.double().numpy())
    assert np.all(np.abs(got - ref) <= 1e-5 * abs_sum)


# ---------------------------------------------------------------------------
# quantizer exports and MinMax initialisation
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("bits,sym", [(8, False), (8, True), (4, False), (4, True)])
def test_fake_quant_act_bit_exact(ctx, dtype, bits, sym):
    g = torch.Generator().manual_seed(11 + bits + int(sym))
    x = (torch.randn((301, 77), generator=g) * 1.7).to(dtype)
    x64 = x.double().numpy()
    s, z = O.init_minmax_x(x64, bits, sym)
    for s_use, z_use in ((s, z), (np.float32(s * 0.61), np.float32(z + 3.4))):
        codes, clip = B.fake_quant_act(ctx, x.cuda(), torch.tensor([s_use]).cuda(), torch.tensor([z_use]).cuda(),
                                       bits, sym)
        ref = O.fake_quant_x(x64, s_use, z_use, bits, sym)
        assert np.array_equal(codes.cpu().numpy(), ref["q"])
        assert np.array_equal(clip.cpu().numpy(), ref["flag"])
    assert ref["flag"].any()
    assert ctx.device_status() == 0


@pytest.mark.parametrize("bits", [8, 4])
def test_fake_quant_weight_bit_exact(ctx, bits):
    g = torch.Generator().manual_seed(17 + bits)
    W = torch.randn((93, 200), generator=g) * 0.02
    W[5] = 0.0
    s = O.init_minmax_w(W.double().numpy(), bits)
    for s_use in (s, (s * np.float32(0.7)).astype(np.float32)):
        codes, clip = B.fake_quant_weight(ctx, W.cuda(), torch.from_numpy(s_use).cuda(), bits)
        ref = O.fake_quant_w(W.numpy(), s_use, bits)
        assert np.array_equal(codes.cpu().numpy(), ref["q"])
        assert np.array_equal(clip.cpu().numpy(), ref["flag"])
        Q = (1 << (bits - 1)) - 1
        assert codes.min().item() >= -Q and codes.max().item() <= Q
    assert ref["flag"].any()


def test_tie_values_round_to_even(ctx):
    s = np.float32(2.0 ** -4)
    j = np.arange(-100, 100)
    x = torch.tensor((j + 0.5) * float(s), dtype=torch.float32)
    codes, clip = B.fake_quant_act(ctx, x.cuda(), torch.tensor([s]).cuda(), torch.tensor([0.0]).cuda(), 8, True)
    want = np.where(j % 2 == 0, j, j + 1)
    assert np.array_equal(codes.cpu().numpy(), want) and not clip.any().item()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("bits,sym", [(8, False), (8, True), (4, False)])
def test_init_qparams_exact(ctx, dtype, bits, sym):
    g = torch.Generator().manual_seed(23)
    x = (torch.randn((1000, 333), generator=g) * 2 + 0.3).to(dtype)
    s, z = B.init_act_qparams(ctx, x.cuda(), bits, sym)
    rs, rz = O.init_minmax_x(x.double().numpy(), bits, sym)
    assert s.item() == float(rs) and z.item() == float(rz)
    W = torch.randn((70, 264), generator=g) * 0.02
    W[3] = 0
    sw = B.init_weight_scales(ctx, W.cuda(), bits)
    assert np.array_equal(sw.cpu().numpy(), O.init_minmax_w(W.numpy(), bits))


def test_bad_scale_is_reported_not_faulted(ctx):
    x = torch.randn(64, 64).cuda()
    B.fake_quant_act(ctx, x, torch.tensor([-1.0]).cuda(), torch.tensor([0.0]).cuda(), 8, False)
    assert ctx.device_status() == 1          # EFQAT_DEV_BAD_SCALE
    assert ctx.device_status() == 0          # reading clears it


# ---------------------------------------------------------------------------
# selection
# ---------------------------------------------------------------------------
def _weights(seed, shapes, ties=True):
    g = torch.Generator().manual_seed(seed)
    Ws = []
    for n, k, sc in shapes:
        W = torch.randn((n, k), generator=g) * sc
        if ties and n >= 8:
            W[n // 2] = W[1]            # equal importance, different index
            W[n - 1] = W[1].flip(0)     # equal |w| multiset
            W[3] = 0.0
        Ws.append(W)
    return Ws


def _same_sets(got, ref):
    assert len(got) == len(ref)
    for a, b in zip(got, ref):
        assert a.dtype == torch.int32
        assert a.cpu().numpy().tolist() == b.tolist()


SHAPES = [(64, 128, 1.0), (200, 72, 1.3), (8, 4096, 0.7), (1500, 40, 1.0), (33, 7, 2.0)]


@pytest.mark.parametrize("frac", [0.0, 0.05, 0.5, 1.0])
def test_select_cwpl(ctx, frac):
    Ws = _weights(31, SHAPES)
    ks = [int(frac * w.shape[0]) for w in Ws]
    got, offsets, imp = B.select_channels(ctx, B.CWPL, [w.cuda() for w in Ws], ks, want_importance=True)
    _same_sets(got, O.select_cwpl([w.numpy() for w in Ws], ks))
    keys = np.concatenate([O.importance_rows(w.numpy()) for w in Ws])
    assert np.array_equal(imp.cpu().numpy(), keys)
    assert offsets.cpu().tolist() == np.concatenate([[0], np.cumsum(ks)]).tolist()
    assert ctx.device_status() == 0


@pytest.mark.parametrize("budget", [0, 1, 180, 1805])
def test_select_cwpn(ctx, budget):
    Ws = _weights(37, SHAPES)
    got, offsets, _ = B.select_channels(ctx, B.CWPN, [w.cuda() for w in Ws], [budget])
    ref = O.select_cwpn([w.numpy() for w in Ws], budget)
    _same_sets(got, ref)
    assert offsets.cpu().tolist()[-1] == budget


@pytest.mark.parametrize("k_layers", [0, 2, 5])
def test_select_lwpn(ctx, k_layers):
    Ws = _weights(41, SHAPES, ties=False)
    got, offsets, imp = B.select_channels(ctx, B.LWPN, [w.cuda() for w in Ws], [k_layers], want_importance=True)
    _same_sets(got, O.select_lwpn([w.numpy() for w in Ws], k_layers))
    assert np.array_equal(imp.cpu().numpy(), np.array([O.importance_layer(w.numpy()) for w in Ws]))


def test_select_all_equal_keys_takes_lowest_indices(ctx):
    W = torch.ones((50, 16))
    got, _, _ = B.select_channels(ctx, B.CWPL, [W.cuda()], [7])
    assert got[0].cpu().tolist() == list(range(7))


def test_select_many_layers(ctx):
    # more layers than one table chunk holds
    g = torch.Generator().manual_seed(43)
    Ws = [torch.randn((16 + (i % 5) * 8, 24), generator=g) * (1 + 0.01 * i) for i in range(130)]
    ks = [w.shape[0] // 4 for w in Ws]
    got, _, _ = B.select_channels(ctx, B.CWPL, [w.cuda() for w in Ws], ks)
    _same_sets(got, O.select_cwpl([w.numpy() for w in Ws], ks))
    got, _, _ = B.select_channels(ctx, B.CWPN, [w.cuda() for w in Ws], [500])
    _same_sets(got, O.select_cwpn([w.numpy() for w in Ws], 500))


def test_bounded_wait_runs_out_and_reports(ctx):
    """A device-side wait that nothing satisfies gives up after its limit, the kernel returns,
    the status word reads EFQAT_DEV_WAIT_TIMEOUT, and the context keeps working afterwards."""
    import time
    assert ctx.device_status() == 0
    t0 = time.perf_counter()
    ctx.selftest_bounded_wait(2_000_000)            # 2 ms
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0
    assert ctx.device_status() == 3
    assert B.status_string(3) == "device: bounded wait expired"
    assert ctx.device_status() == 0                  # reading cleared it
    W = torch.randn(64, 128, device="cuda")
    s = B.init_weight_scales(ctx, W, 8)
    torch.cuda.synchronize()
    assert torch.equal(s, W.abs().amax(dim=1) / 127) or torch.allclose(s, W.abs().amax(dim=1) / 127, rtol=1e-6)
    assert ctx.device_status() == 0
    lib = B.load()
    assert lib.efqat_selftest_bounded_wait(ctx.handle, 10, None) == -2       # limit outside 1 us .. 1 s
    assert lib.efqat_selftest_bounded_wait(None, 1000000, None) == -1


@pytest.mark.parametrize("log2_scale", [False, True])
def test_qparam_adam_matches_oracle(ctx, log2_scale):
    """Three fused Adam steps on the weight scales of the selected channels, the activation scale
    and the zero point (raw and with theta = log2 s) against the fp64 oracle; the scales and
    moments of the frozen channels stay bit-identical."""
    r = np.random.default_rng(61 + int(log2_scale))
    N = 777
    idx = np.sort(r.choice(N, 123, replace=False)).astype(np.int32)
    frozen = np.setdiff1d(np.arange(N), idx)
    s_w0 = (r.random(N) * 0.05 + 0.002).astype(np.float32)
    s_x0, z_x0 = np.float32(0.0173), np.float32(117.3)
    s_w = torch.from_numpy(s_w0.copy()).cuda()
    s_x = torch.tensor([float(s_x0)], device="cuda")
    z_x = torch.tensor([float(z_x0)], device="cuda")
    lr = 1e-3
    opt = B.QParamOptimizer(ctx, s_w, s_x, z_x, lr, log2_scale=log2_scale)
    # the ABI carries the hyper-parameters as fp32: the oracle gets the same (rounded) values
    hp = dict(lr=float(np.float32(lr)), beta1=float(np.float32(0.9)), beta2=float(np.float32(0.999)),
              eps=float(np.float32(1e-8)))
    # oracle state
    pw, mw, vw = s_w0.astype(np.float64), np.zeros(N), np.zeros(N)
    px, mx, vx = np.array([s_x0], np.float64), np.zeros(1), np.zeros(1)
    pz, mz, vz = np.array([z_x0], np.float64), np.zeros(1), np.zeros(1)
    thw, thx = (np.log2(pw), np.log2(px)) if log2_scale else (None, None)
    idx_dev = torch.from_numpy(idx).cuda()
    for t in range(1, 4):
        gw = (r.standard_normal(len(idx)) * 10.0 ** r.uniform(-3, 3, len(idx))).astype(np.float32)
        gx, gz = np.float32(r.standard_normal() * 50), np.float32(r.standard_normal() * 0.01)
        opt.step(idx_dev, len(idx), torch.from_numpy(gw).cuda(), torch.tensor([float(gx)], device="cuda"),
                 torch.tensor([float(gz)], device="cuda"))
        if log2_scale:
            pw, mw, vw, thw = O.adam_qparams(pw, mw, vw, gw, idx, t, theta=thw, **hp)
            px, mx, vx, thx = O.adam_qparams(px, mx, vx, [gx], None, t, theta=thx, **hp)
        else:
            pw, mw, vw = O.adam_qparams(pw, mw, vw, gw, idx, t, **hp)
            px, mx, vx = O.adam_qparams(px, mx, vx, [gx], None, t, **hp)
        pz, mz, vz = O.adam_qparams(pz, mz, vz, [gz], None, t, **hp)
        torch.cuda.synchronize()
        np.testing.assert_allclose(s_w.cpu().numpy(), pw, rtol=1e-5)
        np.testing.assert_allclose(opt.m_sw.cpu().numpy(), mw, rtol=1e-5, atol=1e-30)
        np.testing.assert_allclose(opt.v_sw.cpu().numpy(), vw, rtol=1e-5, atol=1e-30)
        np.testing.assert_allclose(s_x.item(), px[0], rtol=1e-5)
        np.testing.assert_allclose(z_x.item(), pz[0], rtol=1e-6)
        if log2_scale:
            np.testing.assert_allclose(opt.theta_sw.cpu().numpy()[idx], thw[idx], rtol=1e-5)
        assert np.array_equal(s_w.cpu().numpy()[frozen], s_w0[frozen])
        assert not opt.m_sw.cpu().numpy()[frozen].any() and not opt.v_sw.cpu().numpy()[frozen].any()
    assert ctx.device_status() == 0
    # every selected scale moved, by about lr per step in the first steps (Adam's normalised update)
    moved = np.abs(s_w.cpu().numpy()[idx] - s_w0[idx])
    assert np.all(moved > 0)
    lib = B.load()
    import ctypes as C
    bad = B.Adam(lr, 0.9, 0.999, 1e-8, 0, 0)             # step must be >= 1
    assert lib.efqat_qparam_adam(ctx.handle, C.byref(bad), C.byref(opt.state), N, None, 0, None,
                                 C.c_void_p(s_x.data_ptr()), None, None) == -2


def test_backward_then_qparam_adam_end_to_end(ctx):
    """Gradients straight from efqat_fq_linear_bwd into efqat_qparam_adam on the device, against
    the oracle's backward followed by the oracle's Adam step."""
    case = I.LayerCase("adam_e2e", 192, 128, 96, act_dtype=torch.float32, seed=77)
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.8, 0.85, 0.4))
    D = U.to_dev(T, s_w, s_x, z_x)
    idx = O.select_cwpl([T["W"].numpy()], [12])[0]
    idx_dev = torch.from_numpy(idx).cuda()
    out = B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx_dev, 12, 8, 8, False)
    opt = B.QParamOptimizer(ctx, D["s_w"], D["s_x"], D["z_x"], 1e-4)
    opt.step(idx_dev, 12, out["dS_w_sel"], out["dS_x"], out["dZ_x"])
    torch.cuda.synchronize()
    ref = O.backward_efqat(I.as_f64(T["dY"]), I.as_f64(T["X"]), I.as_f64(T["W"]), s_w, s_x, z_x, idx, 8, 8,
                           operand_model="bf16")
    hp = dict(lr=float(np.float32(1e-4)), beta1=float(np.float32(0.9)), beta2=float(np.float32(0.999)),
              eps=float(np.float32(1e-8)))
    pw, _, _ = O.adam_qparams(s_w, np.zeros(96), np.zeros(96), ref["dS_w_sel"], idx, 1, **hp)
    px, _, _ = O.adam_qparams([s_x], [0.0], [0.0], [ref["dS_x"]], None, 1, **hp)
    pz, _, _ = O.adam_qparams([z_x], [0.0], [0.0], [ref["dZ_x"]], None, 1, **hp)
    np.testing.assert_allclose(D["s_w"].cpu().numpy(), pw, rtol=1e-5)
    np.testing.assert_allclose(D["s_x"].item(), px[0], rtol=1e-5)
    np.testing.assert_allclose(D["z_x"].item(), pz[0], rtol=1e-6)
    assert ctx.device_status() == 0
