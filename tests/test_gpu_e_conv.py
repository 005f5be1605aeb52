"""GPU parity of the convolution form of the layer step (implicit GEMM over NHWC tensors,
strides 1 and 2, channel counts that are not multiples of 64, filters up to 7 x 7) against the
oracle: forward, grad-input with the STE mask and dS_x / dZ_x, and the partial grad-weight,
including padded borders with a non-zero activation zero point.  The stride-2 cases carry the
shapes of ResNet-50's stem, of its three stride-2 3x3 convolutions and of its three stride-2
1x1 shortcut convolutions (Section 4 "Setup": every convolution is quantized, "including the
input, output, and shortcut layers")."""
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


def _case(name, Bn, H, Wd, Cin, N, R, pad, dtype=torch.bfloat16, w_bits=4, seed=0, stride=1):
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - R) // stride + 1
    return I.LayerCase(name, Bn * Ho * Wo, R * R * Cin, N, act_dtype=dtype, w_bits=w_bits, x_bits=8, w_std=None,
                       x_abs=True, seed=seed, conv=True, B=Bn, H=H, Wd=Wd, Cin=Cin, R=R, S=R, stride=stride, pad=pad)


CASES = [
    _case("c3x3_small", 2, 9, 10, 64, 72, 3, 1, seed=1),
    _case("c3x3_valid_f32", 3, 8, 8, 64, 64, 3, 0, dtype=torch.float32, seed=2),
    _case("c5x5", 2, 7, 7, 128, 136, 5, 2, w_bits=8, seed=3),
    _case("c3x3_14", 4, 14, 14, 128, 256, 3, 1, seed=4),
    _case("c1x1", 2, 12, 12, 72, 64, 1, 0, seed=5),
    _case("resnet_56_64to256_3x3_b2", 2, 56, 56, 64, 256, 3, 1, seed=6),
    # channel counts that are not multiples of 64 (zero-filled chunk tails)
    _case("c3x3_cin72", 2, 10, 9, 72, 80, 3, 1, seed=7),
    _case("c3x3_cin8_f32", 2, 12, 12, 8, 64, 3, 1, dtype=torch.float32, seed=8),
    # stride 2: odd and even extents, padded and valid
    _case("c3x3_s2_odd", 2, 9, 11, 64, 72, 3, 1, seed=9, stride=2),
    _case("c3x3_s2_valid", 3, 10, 10, 64, 64, 3, 0, seed=10, stride=2),
    _case("c5x5_s2", 2, 13, 12, 128, 64, 5, 2, w_bits=8, seed=11, stride=2),
    _case("c1x1_s2", 2, 14, 14, 64, 128, 1, 0, seed=12, stride=2),
    _case("c2x2_s2", 2, 8, 8, 64, 64, 2, 0, seed=13, stride=2),
    # ResNet-50: stem (3 input channels padded to 8), stride-2 3x3 of stages 2-4, stride-2 shortcuts
    _case("resnet_stem_7x7_s2", 1, 224, 224, 8, 64, 7, 3, w_bits=8, seed=14, stride=2),
    # few input channels: a whole filter row is one contraction block on a zero-framed copy of the codes
    _case("c3x3_cin16_s2_odd", 2, 11, 13, 16, 72, 3, 1, seed=21, stride=2),
    _case("c5x5_cin8_valid", 3, 12, 9, 8, 64, 5, 0, w_bits=8, seed=22),
    _case("c3x3_cin16_pad2", 2, 9, 9, 16, 64, 3, 2, seed=23),
    # ... and grad-input on strips of 64 / Cin pixels where the width allows it
    _case("c3x3_cin16_strip", 2, 9, 12, 16, 72, 3, 1, seed=29),
    _case("c2x2_cin32_s2_strip", 2, 8, 16, 32, 64, 2, 0, seed=30, stride=2),
    _case("c5x5_cin8_s2_strip", 2, 10, 16, 8, 64, 5, 2, w_bits=8, seed=31, stride=2),
    _case("c7x7_cin8_s2_strip_b2", 2, 30, 32, 8, 72, 7, 3, seed=32, stride=2),
    _case("c3x3_cin16_strip_f32", 1, 8, 8, 16, 64, 3, 1, dtype=torch.float32, seed=33),
    # extents that 8-, 16- or 32-pixel-wide one-image boxes tile well: the taps of a filter column share one box
    _case("c3x3_shared_30x15", 2, 15, 30, 64, 72, 3, 1, seed=24),
    _case("c3x3_shared_cin128", 2, 16, 24, 128, 136, 3, 1, seed=25),
    _case("c3x3_shared_valid_f32", 1, 16, 24, 64, 64, 3, 0, dtype=torch.float32, seed=26),
    _case("c4x4_shared_s2", 2, 32, 48, 64, 64, 4, 1, seed=27, stride=2),
    _case("c3x3_shared_resident_2chunks", 2, 16, 24, 128, 64, 3, 1, seed=40),      # resident weights over two channel chunks
    _case("c3x3_shared_two_tile_columns", 1, 16, 16, 64, 320, 3, 1, seed=41),      # several tile columns: weights staged per stage
    _case("resnet_56_64to64_3x3_b2", 2, 56, 56, 64, 64, 3, 1, seed=28),
    # the CIFAR-10 ResNet-20's layer shapes (16 / 32 / 64 channels on 32 x 32, 16 x 16 and 8 x 8 maps)
    _case("resnet20_stem", 2, 32, 32, 8, 16, 3, 1, seed=34),
    _case("resnet20_stage1", 2, 32, 32, 16, 16, 3, 1, seed=35),
    _case("resnet20_stage2_first_s2", 2, 32, 32, 16, 32, 3, 1, seed=36, stride=2),
    _case("resnet20_stage2", 2, 16, 16, 32, 32, 3, 1, seed=37),
    _case("resnet20_stage3_first_s2", 3, 16, 16, 32, 64, 3, 1, seed=38, stride=2),
    _case("resnet20_stage3", 4, 8, 8, 64, 64, 3, 1, seed=39),
    _case("resnet_56_128_3x3_s2", 2, 56, 56, 128, 128, 3, 1, seed=15, stride=2),
    _case("resnet_28_256_3x3_s2", 2, 28, 28, 256, 256, 3, 1, seed=16, stride=2),
    _case("resnet_14_512_3x3_s2", 2, 14, 14, 512, 512, 3, 1, seed=17, stride=2),
    _case("resnet_56_256to512_1x1_s2", 2, 56, 56, 256, 512, 1, 0, seed=18, stride=2),
    _case("resnet_28_512to1024_1x1_s2", 2, 28, 28, 512, 1024, 1, 0, seed=19, stride=2),
    _case("resnet_14_1024to2048_1x1_s2", 2, 14, 14, 1024, 2048, 1, 0, seed=20, stride=2),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: c.name)
def test_conv_forward_backward_parity(ctx, case):
    T = I.make_tensors(case)
    T["X"] = (T["X"].float() - 0.3).to(case.act_dtype)        # asymmetric range: Z != 0, pad must act as x^ = 0
    X64, W64, dY64, b64 = (I.as_f64(T[k]) for k in ("X", "W", "dY", "bias"))
    s_w = (O.init_minmax_w(W64, case.w_bits) * np.float32(0.9)).astype(np.float32)
    s_x, z_x = O.init_minmax_x(X64, case.x_bits)
    s_x = np.float32(s_x * np.float32(0.8))
    assert float(np.clip(np.rint(z_x), 0, 255)) > 0
    D = U.to_dev(T, s_w, s_x, z_x)
    geom = B.ConvGeom(case.B, case.H, case.Wd, case.Cin, case.R, case.S, case.stride, case.pad)
    is_bf16 = case.act_dtype == torch.bfloat16
    Yabs, Gx_abs, Gw_abs = U.conv_abs_bounds(case, T, s_w, s_x, z_x)

    Y = B.fq_linear_fwd(ctx, D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], D["bias"], case.w_bits, case.x_bits,
                        False, conv=geom)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ref = O.conv_forward(X64, W64, s_w, s_x, z_x, b64, case.w_bits, case.x_bits, case.stride, case.pad)
    got = U.np32(Y)
    U.assert_bf16_class(got, ref, case.name + " Y")
    U.assert_fp32_class(got, ref, Yabs + np.abs(b64), case.name + " Y", out_is_bf16=is_bf16)

    N = case.N
    sets = [np.zeros(0, np.int32), O.select_cwpl([W64], [max(1, N // 10)])[0], np.arange(N, dtype=np.int32)]
    outs = []
    for idx in sets:
        k = len(idx)
        idx_dev = torch.from_numpy(idx).cuda() if 0 < k < N else None
        out = B.fq_linear_bwd(ctx, D["dY"], D["X"], D["W"], D["s_w"], D["s_x"], D["z_x"], idx_dev, k,
                              case.w_bits, case.x_bits, False, want_db=True, conv=geom)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        g = {kk: (U.np32(v) if v is not None else None) for kk, v in out.items()}
        outs.append(g)
        args = (dY64, X64, W64, s_w, s_x, z_x, idx, case.w_bits, case.x_bits, case.stride, case.pad)
        ex = O.conv_backward_efqat(*args, operand_model="exact")
        bm = O.conv_backward_efqat(*args, operand_model="bf16")
        name = f"{case.name} k_sel={k}"
        clip_x = O.fake_quant_x(X64, s_x, z_x, case.x_bits)["flag"] != 0
        assert clip_x.any() and np.all(g["dX"][clip_x] == 0)
        U.assert_bf16_class(g["dX"], ex["dX"], name + " dX")
        U.assert_fp32_class(g["dX"], bm["dX"], Gx_abs, name + " dX", out_is_bf16=is_bf16)
        for key in ("dS_x", "dZ_x"):
            U.assert_fp32_class(g[key][0], bm[key], bm[key + "_abs"], name + " " + key, atol=1e-30)
        U.assert_fp32_class(g["db"], bm["db"], np.abs(dY64).reshape(-1, N).sum(axis=0), name + " db")
        dW = g["dW_sel"].reshape((k,) + W64.shape[1:])
        if k:
            U.assert_bf16_class(dW, ex["dW_sel"], name + " dW_sel")
            U.assert_fp32_class(dW, bm["dW_sel"], Gw_abs[idx], name + " dW_sel")
            U.assert_fp32_class(g["dS_w_sel"], bm["dS_w_sel"], bm["dS_w_sel_abs"], name + " dS_w", atol=1e-30)
    for o in outs[1:]:
        for key in ("dX", "dS_x", "dZ_x", "db"):
            assert np.array_equal(o[key], outs[0][key]), key
