"""GPU tests of the building blocks through the C ABI: the tensor-core contraction in its
four operand layouts, the quantizer exports (bit-exact against the oracle), the MinMax
initialisation and the Top-K selection modes (index sets bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import efqat_oracle as O
from paper_2411_11038_b200 import binding as B

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
