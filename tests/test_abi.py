"""CPU-only checks of the C ABI: the library loads, exports every symbol the header
declares, and the host-side validation returns its error codes without touching a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2411_11038_b200 import binding as B
from paper_2411_11038_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.load()


def test_exports_every_declared_symbol(lib):
    inc = os.path.join(ROOT, "include")
    header = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    declared = set(re.findall(r"\b(efqat_[a-z0-9_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    seen = set()
    for code in list(range(-11, 1)) + [1, 2, 3]:
        s = B.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 15
    assert B.status_string(-99) == "unknown status"


def test_ratio_to_k(lib):
    assert B.ratio_to_k(0.05, 512) == 25
    assert B.ratio_to_k(0.1, 221184) == 22118
    assert B.ratio_to_k(0.0, 768) == 0 and B.ratio_to_k(1.0, 768) == 768
    assert B.ratio_to_k(0.25, 2304) == 576 and B.ratio_to_k(0.05, 3072) == 153


def test_validate_layer_codes(lib):
    ok = B.layer_desc(256, 512, 512, B.F32)
    spec = B.QSpec(8, 8, 1)
    assert B.validate_layer(ok, spec) == 0
    assert B.validate_layer(B.layer_desc(0, 512, 512, B.F32), spec) == -2
    assert B.validate_layer(B.layer_desc(256, 510, 512, B.F32), spec) == -3
    assert B.validate_layer(B.layer_desc(256, 512, 100, B.F32), spec) == -3
    assert B.validate_layer(B.layer_desc(256, 512, 512, 7), spec) == -4
    assert B.validate_layer(ok, B.QSpec(9, 8, 0)) == -5
    assert B.validate_layer(ok, B.QSpec(8, 1, 0)) == -5
    conv = B.ConvGeom(B=2, H=8, W=8, Cin=16, R=1, S=1)
    assert B.validate_layer(B.layer_desc(128, 32, 16, B.BF16, conv), spec) == 0
    assert B.validate_layer(B.layer_desc(127, 32, 16, B.BF16, conv), spec) == -2
    conv2 = B.ConvGeom(B=2, H=8, W=8, Cin=16, R=3, S=3, stride=2, pad=1)
    assert B.validate_layer(B.layer_desc(32, 32, 144, B.BF16, conv2), spec) == 0          # 8x8 -> 4x4
    assert B.validate_layer(B.layer_desc(128, 32, 144, B.BF16, conv2), spec) == -2        # M of stride 1
    conv3 = B.ConvGeom(B=2, H=8, W=8, Cin=16, R=3, S=3, stride=3, pad=1)
    assert B.validate_layer(B.layer_desc(18, 32, 144, B.BF16, conv3), spec) == -9         # strides 1 and 2 only
    conv4 = B.ConvGeom(B=1, H=16, W=16, Cin=8, R=9, S=9, stride=1, pad=4)
    assert B.validate_layer(B.layer_desc(256, 32, 648, B.BF16, conv4), spec) == -9        # filters up to 7 x 7


def test_workspace_queries(lib):
    d = B.layer_desc(4096, 768, 768, B.BF16)
    spec = B.QSpec(8, 8, 0)
    w0 = B.workspace_bytes(d, spec, 0)
    w38 = B.workspace_bytes(d, spec, 38)
    wN = B.workspace_bytes(d, spec, 768)
    assert 0 < w0 <= w38 <= wN
    assert w0 >= 4096 * 768 * 2 + 768 * 768 * 2
    with pytest.raises(B.EfqatError) as e:
        B.workspace_bytes(d, spec, 769)
    assert e.value.code == -8
    assert B.select_workspace_bytes(144, 221184) > 221184 * 16


def test_null_context_is_rejected_before_any_launch(lib):
    d = B.layer_desc(256, 512, 512, B.F32)
    spec = B.QSpec(8, 8, 1)
    rc = lib.efqat_fq_linear_fwd(None, C.byref(d), C.byref(spec), None, None, None, None, None, None, None,
                                 None, 0, None)
    assert rc == -1
    rc = lib.efqat_fq_linear_bwd(None, C.byref(d), C.byref(spec), None, None, None, None, None, None, None, 0,
                                 None, None, None, None, None, None, None, None, 0, None)
    assert rc == -1
    code = C.c_int(0)
    assert lib.efqat_device_status(None, C.byref(code)) == -1
    assert lib.efqat_destroy(None) == -1


def test_weight_cache_and_network_queries(lib):
    """Host-side behaviour of the cache / network entry points: sizes, and errors found before any launch."""
    spec = B.QSpec(8, 8, 0)
    big = B.layer_desc(4096, 768, 768, B.BF16)            # forward on 8-bit codes: 1 + 2 bytes per weight + row sums
    small = B.layer_desc(4096, 520, 256, B.BF16)          # forward on bf16 codes: 2 + 2 bytes per weight
    nb, ns = B.weight_cache_bytes(big, spec), B.weight_cache_bytes(small, spec)
    assert 3 * 768 * 768 + 4 * 768 <= nb <= 3 * 768 * 768 + 4 * 768 + 4096
    assert 4 * 520 * 256 <= ns <= 4 * 520 * 256 + 4096
    out = C.c_size_t(0)
    assert lib.efqat_weight_cache_bytes(C.byref(B.layer_desc(0, 8, 8, B.BF16)), C.byref(spec), C.byref(out)) == -2
    assert lib.efqat_weight_cache_bytes(C.byref(big), C.byref(spec), None) == -1
    assert lib.efqat_weight_cache_update(None, C.byref(big), C.byref(spec), None, None, None, 0, None, 0, None) == -1
    assert lib.efqat_fq_linear_fwd_cached(None, C.byref(big), C.byref(spec), None, None, None, None, None, None,
                                          None, 0, None, 0, None) == -1
    assert lib.efqat_fq_linear_bwd_cached(None, C.byref(big), C.byref(spec), None, None, None, None, None, None,
                                          None, 0, None, None, None, None, None, None, None, None, 0, None, 0,
                                          None) == -1
    for fn in (lib.efqat_network_fwd, lib.efqat_network_bwd, lib.efqat_network_cache_update):
        assert fn(None, 1, None, None) == -1
    adam = B.Adam(1e-6, 0.9, 0.999, 1e-8, 1, 0)
    assert lib.efqat_network_qparam_adam(None, C.byref(adam), 1, None, None, None) == -1
    # workspace of a layer that takes the one-pass backward: one partial product per CTA
    skinny = B.layer_desc(200704, 256, 64, B.BF16)
    assert B.workspace_bytes(skinny, spec, 256) >= 148 * 256 * 64 * 4


def test_workspace_of_the_input_layer_forms(lib):
    """Convolutions with few input channels keep a zero-framed copy of the activation codes and the
    banded weights of the strip-form grad-input in the workspace: the query must cover both."""
    spec = B.QSpec(4, 8, 0)
    conv = B.ConvGeom(B=4, H=224, W=224, Cin=8, R=7, S=7, stride=2, pad=3)
    d = B.layer_desc(4 * 112 * 112, 64, 392, B.BF16, conv)
    assert B.validate_layer(d, spec) == 0
    need = 4 * 230 * 230 * 8 * 2 + 64 * 7 * 7 * 64 * 2            # framed codes + banded weights [N, R * nP * 64]
    assert B.workspace_bytes(d, spec, 64) >= need
    # a wide layer of the same extent keeps the dense code layout
    conv2 = B.ConvGeom(B=4, H=56, W=56, Cin=64, R=3, S=3, stride=1, pad=1)
    d2 = B.layer_desc(4 * 56 * 56, 64, 576, B.BF16, conv2)
    assert B.workspace_bytes(d2, spec, 0) < 4 * 56 * 56 * 64 * 2 + 64 * 576 * 2 + (1 << 20)


def test_network_layer_lists():
    """The layer lists of the two convolutional networks the bench runs: counts, channels and work
    as the architectures fix them (ResNet-50: 4.1 G multiply-adds per 224 x 224 image with the input
    layer on 8 stored channels; ResNet-20: 41 M per 32 x 32 image)."""
    from paper_2411_11038_b200 import inputs as I
    r50, r20 = I.resnet50(2), I.resnet20(2)
    assert len(r50) == 54 and sum(c.conv for c in r50) == 53 and sum(c.N for c in r50) == 26560 + 1000
    assert len(r20) == 20 and sum(c.conv for c in r20) == 19 and sum(c.N for c in r20) == 16 + 6 * 16 + 6 * 32 + 6 * 64 + 16
    macs50 = sum(c.M * c.N * c.K for c in r50) / 2
    macs20 = sum(c.M * c.N * c.K for c in r20) / 2
    assert 4.0e9 < macs50 < 4.4e9 and 40e6 < macs20 < 43e6
    for c in r50 + r20:
        if c.conv:
            ho = (c.H + 2 * c.pad - c.R) // c.stride + 1
            assert c.M == c.B * ho * ho and c.K == c.R * c.S * c.Cin
    # consecutive layers of a stage agree in their map size: the 3x3 of a ResNet-50 block reads what its 1x1 wrote
    by = {c.name: c for c in r50}
    assert by["rn50_s2b1_b"].H == 56 and by["rn50_s2b1_b"].stride == 2 and by["rn50_s2b1_c"].H == 28
    assert by["rn50_s4b3_c"].H == 7 and by["rn50_s4b3_c"].N == 2048
