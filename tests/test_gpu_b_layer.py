"""GPU parity of the whole layer step (forward, partial backward) against the oracle,
element by element, on shapes that span several tiles with ragged tails."""
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


def _case(name, M, K, N, dtype, w_bits=8, x_bits=8, sym=False, seed=0):
    return I.LayerCase(name, M, K, N, act_dtype=dtype, w_bits=w_bits, x_bits=x_bits, x_symmetric=sym, seed=seed)


SMALL = [
    _case("ragged_f32", 200, 136, 72, torch.float32, seed=1),
    _case("ragged_bf16", 333, 200, 264, torch.bfloat16, seed=2),
    _case("tiles_bf16_w4", 512, 320, 520, torch.bfloat16, w_bits=4, seed=3),
    _case("sym_a4", 260, 64, 128, torch.bfloat16, w_bits=4, x_bits=4, sym=True, seed=4),
    _case("one_row", 1, 64, 8, torch.float32, seed=5),
    _case("two_bit", 160, 72, 40, torch.bfloat16, w_bits=2, x_bits=2, seed=6),
    _case("smallest", 8, 8, 8, torch.bfloat16, seed=7),
    # contractions of 512 and more with N % 32 == 0: the forward runs on the integer tensor cores
    _case("int8_asym_bf16", 333, 640, 96, torch.bfloat16, seed=8),
    _case("int8_asym_f32", 200, 512, 64, torch.float32, seed=9),
    _case("int8_sym_w4", 130, 1024, 160, torch.bfloat16, w_bits=4, x_bits=8, sym=True, seed=10),
    # contractions of 64 / 128 with N % 64 == 0: the one-launch forward with the quantizer as operand producer
    _case("short_k64_bf16", 1000, 64, 256, torch.bfloat16, w_bits=4, seed=11),
    _case("short_k128_bf16", 700, 128, 512, torch.bfloat16, w_bits=4, seed=12),
    _case("short_k64_f32", 300, 64, 64, torch.float32, seed=13),
    _case("short_k128_ragged_n", 129, 128, 320, torch.bfloat16, seed=14),
    _case("short_k64_wide", 260, 64, 832, torch.bfloat16, x_bits=4, sym=True, seed=15),
    # ... and with N = 128 / 256 the backward in one pass over dY and X
    _case("short_k64_n128", 517, 64, 128, torch.bfloat16, seed=16),
    _case("short_k64_n256_sym", 300, 64, 256, torch.bfloat16, w_bits=4, x_bits=4, sym=True, seed=17),
    _case("short_k64_many_tiles", 40000, 64, 256, torch.bfloat16, w_bits=4, seed=18),
]


@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
@pytest.mark.parametrize("clip", [False, True])
def test_forward_parity(ctx, case, clip):
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.7, 0.8, 2.3) if clip else None)
    D = U.to_dev(T, s_w, s_x, z_x)
    U.check_forward(ctx, case, T, D, s_w, s_x, z_x)


@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
@pytest.mark.parametrize("clip", [False, True])
def test_backward_parity_and_invariants(ctx, case, clip):
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.7, 0.8, 2.3) if clip else None)
    D = U.to_dev(T, s_w, s_x, z_x)
    N = case.N
    k5 = max(1, N // 20)
    sets = [np.zeros(0, np.int32), O.select_cwpl([T["W"].numpy()], [k5])[0],
            np.arange(0, N, 3, dtype=np.int32), np.arange(N, dtype=np.int32)]
    if N > 2:
        sets.insert(3, np.delete(np.arange(N, dtype=np.int32), N // 2))      # all channels but one: widest gather
    outs = [U.check_backward(ctx, case, T, D, s_w, s_x, z_x, idx) for idx in sets]
    # dX, dS_x, dZ_x, db never depend on the selection: bit-identical across idx
    for o in outs[1:]:
        for key in ("dX", "dS_x", "dZ_x", "db"):
            assert np.array_equal(o[key], outs[0][key]), key
    # 100 % unfrozen is ordinary QAT; a partial set returns the matching rows of it
    full = outs[-1]
    for idx, o in zip(sets[1:3], outs[1:3]):
        assert np.allclose(o["dW_sel"], full["dW_sel"][idx], rtol=1e-5, atol=1e-6 * np.abs(full["dW_sel"]).max())
    # determinism: same call twice -> identical bits
    again = U.check_backward(ctx, case, T, D, s_w, s_x, z_x, sets[2])
    for key in ("dX", "dW_sel", "dS_w_sel", "dS_x", "dZ_x"):
        assert np.array_equal(again[key], outs[2][key]), key


def test_config1_exact_forward_and_selected_backward(ctx):
    """The first workload: fp32 I/O, symmetric activations, 26 of 512 channels."""
    case = I.config1()[0]
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T)
    D = U.to_dev(T, s_w, s_x, z_x)
    got = U.check_forward(ctx, case, T, D, s_w, s_x, z_x)
    # all-integer operands with K*127*127 < 2^24: the contraction itself is exact, only the
    # two epilogue multiplies and the bias add round
    ref, _ = U.fwd_reference(case, T, s_w, s_x, z_x)
    assert np.abs(got - ref).max() <= 4e-7 * np.abs(ref).max()
    sel, _, _ = B.select_channels(ctx, B.CWPL, [D["W"]], [26])
    idx = sel[0].cpu().numpy()
    assert idx.tolist() == O.select_cwpl([T["W"].numpy()], [26])[0].tolist()
    U.check_backward(ctx, case, T, D, s_w, s_x, z_x, idx)


def test_fused_sgd_rows(ctx):
    case = _case("sgd", 256, 128, 96, torch.bfloat16, seed=9)
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T, (0.8, 0.85, 1.0))
    D = U.to_dev(T, s_w, s_x, z_x)
    idx = np.array([0, 5, 17, 40, 95], np.int32)
    g = torch.Generator().manual_seed(3)
    V0 = torch.randn(T["W"].shape, generator=g) * 0.01
    Wd, Vd = D["W"].clone(), V0.cuda()
    sgd = B.make_sgd(0.1, 0.9, 1e-4, Wd, Vd)
    out = U.check_backward(ctx, case, T, D, s_w, s_x, z_x, idx, sgd=sgd)
    W2, V2 = O.sgd_rows(T["W"].numpy(), V0.numpy(), out["dW_sel"], idx, 0.1, 0.9, 1e-4)
    frozen = np.setdiff1d(np.arange(case.N), idx)
    assert np.array_equal(Wd.cpu().numpy()[frozen], T["W"].numpy()[frozen])
    assert np.array_equal(Vd.cpu().numpy()[frozen], V0.numpy()[frozen])
    np.testing.assert_allclose(Wd.cpu().numpy()[idx], W2[idx], rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(Vd.cpu().numpy()[idx], V2[idx], rtol=1e-5, atol=1e-7)


def test_saturating_input_masks_everything(ctx):
    case = _case("sat", 128, 64, 64, torch.float32, seed=10)
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T)
    T["X"] = (T["X"].abs() + 1.0) * 1e3
    D = U.to_dev(T, s_w, s_x, z_x)
    out = U.check_backward(ctx, case, T, D, s_w, s_x, z_x, np.arange(8, dtype=np.int32))
    assert np.all(out["dX"] == 0)


def test_bad_index_is_reported_not_faulted(ctx):
    case = _case("badidx", 128, 64, 64, torch.float32, seed=11)
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T)
    D = U.to_dev(T, s_w, s_x, z_x)
    for bad in ([3, 2, 9], [1, 64, 70], [-4, 5, 6]):
        idx = torch.tensor(bad, dtype=torch.int32).cuda()
        B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx, 3, 8, 8, False)
        torch.cuda.synchronize()
        assert ctx.device_status() == 2      # EFQAT_DEV_BAD_INDEX


def test_host_errors(ctx):
    case = _case("err", 128, 64, 64, torch.float32, seed=12)
    T = I.make_tensors(case)
    s_w, s_x, z_x = U.oracle_qparams(case, T)
    D = U.to_dev(T, s_w, s_x, z_x)
    with pytest.raises(B.EfqatError) as e:
        B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], None, 65, 8, 8, False)
    assert e.value.code == -8
    plan = B.LayerPlan(ctx, 128, 64, 64, torch.float32, 8, 8, False, 0, "cuda")
    with pytest.raises(B.EfqatError) as e:     # workspace sized for k_sel = 0 only
        plan.bwd(D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], None, 64)
    assert e.value.code == -7
    with pytest.raises(B.EfqatError) as e:     # partial selection without indices
        B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], None, 5, 8, 8, False)
    assert e.value.code == -1


def test_backward_back_to_back_on_one_workspace(ctx):
    """Two different problems alternate through ONE plan (one workspace) without any host
    synchronisation in between.  The weight-gradient GEMM runs beside the grad-input GEMM of
    the same call; if it ever started before that call's producers had finished it would
    contract the previous problem's codes, which differ everywhere."""
    M, K, N = 512, 256, 384
    dev = torch.device("cuda", 0)
    cases = [_case("b2b_a", M, K, N, torch.bfloat16, seed=11), _case("b2b_b", M, K, N, torch.bfloat16, seed=12)]
    probs = []
    for c in cases:
        T = I.make_tensors(c)
        s_w, s_x, z_x = U.oracle_qparams(c, T, (0.8, 0.9, 1.3))
        D = U.to_dev(T, s_w, s_x, z_x)
        idx_np = np.arange(1, N, 5, dtype=np.int32)
        idx = torch.from_numpy(idx_np).to(dev)
        X64, W64, dY64 = I.as_f64(T["X"]), I.as_f64(T["W"]), I.as_f64(T["dY"])
        ref = O.backward_efqat(dY64, X64, W64, s_w, s_x, z_x, idx_np, c.w_bits, c.x_bits, c.x_symmetric,
                               operand_model="bf16")
        probs.append((D, idx, len(idx_np), ref))
    plan = B.LayerPlan(ctx, M, N, K, torch.bfloat16, 8, 8, False, N, dev)
    got = []
    for rep in range(6):
        D, idx, k, _ = probs[rep % 2]
        out = plan.bwd(D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx, k, want_db=True)
        got.append({key: out[key][:k].clone() if key in ("dW_sel", "dS_w_sel") else out[key].clone()
                    for key in ("dW_sel", "dS_w_sel", "dX", "dS_x")})
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for rep, g in enumerate(got):
        ref = probs[rep % 2][3]
        U.assert_fp32_class(U.np32(g["dW_sel"]), ref["dW_sel"], ref["G_w_sel_abs"], f"rep {rep} dW_sel")
        U.assert_fp32_class(U.np32(g["dX"]), ref["dX"], ref["G_x_abs"], f"rep {rep} dX", out_is_bf16=True)
        U.assert_fp32_class(U.np32(g["dS_x"])[0], ref["dS_x"], ref["dS_x_abs"], f"rep {rep} dS_x", atol=1e-30)
