"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors and names shapes; it contains none of the
method's arithmetic, so both the CUDA binding's tests and the CPU oracle's tests
can feed on the same bytes.

The paper trains ResNet-20 / ResNet-50 / BERT-base on CIFAR-10 / ImageNet /
SQuAD (Section 4).  Those datasets and checkpoints are not used here: the
workloads below take the *shapes* of those networks' quantized layers and fill
them with seeded Gaussian data.

Draw order for a layer is fixed: X, W, dY, bias, all from one
`torch.Generator('cpu')`; X and dY are cast to the activation dtype afterwards.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import torch


@dataclass
class LayerCase:
    name: str
    M: int                 # tokens, or B*Ho*Wo
    K: int                 # fan-in, or R*S*Cin
    N: int                 # output channels
    act_dtype: torch.dtype = torch.bfloat16
    w_bits: int = 8
    x_bits: int = 8
    x_symmetric: bool = False
    w_std: Optional[float] = 0.02      # None -> Kaiming normal sqrt(2/K)
    x_abs: bool = False                # post-ReLU-like |N(0,1)| activations
    seed: int = 0
    # conv geometry (linear layers keep the defaults)
    conv: bool = False
    B: int = 1
    H: int = 1
    Wd: int = 1
    Cin: int = 0
    R: int = 1
    S: int = 1
    stride: int = 1
    pad: int = 0
    tensors: dict = field(default_factory=dict, repr=False)


def make_tensors(case: LayerCase, with_bias: bool = True):
    """Return dict(X, W, dY, bias) of CPU tensors for `case`.

    Linear: X [M,K], W [N,K] fp32, dY [M,N], bias [N] fp32.
    Conv:   X [B,H,W,Cin], W [N,R,S,Cin] fp32, dY [B,Ho,Wo,N]."""
    g = torch.Generator(device="cpu")
    g.manual_seed(case.seed)
    if case.conv:
        Ho = (case.H + 2 * case.pad - case.R) // case.stride + 1
        Wo = (case.Wd + 2 * case.pad - case.S) // case.stride + 1
        xs = (case.B, case.H, case.Wd, case.Cin)
        ws = (case.N, case.R, case.S, case.Cin)
        ys = (case.B, Ho, Wo, case.N)
        fan_in = case.R * case.S * case.Cin
    else:
        xs, ws, ys, fan_in = (case.M, case.K), (case.N, case.K), (case.M, case.N), case.K
    X = torch.randn(xs, generator=g, dtype=torch.float32)
    if case.x_abs:
        X = X.abs()
    std = case.w_std if case.w_std is not None else math.sqrt(2.0 / fan_in)
    W = torch.randn(ws, generator=g, dtype=torch.float32) * std
    dY = torch.randn(ys, generator=g, dtype=torch.float32)
    bias = torch.randn((case.N,), generator=g, dtype=torch.float32) * 0.1
    out = dict(X=X.to(case.act_dtype).contiguous(), W=W.contiguous(),
               dY=dY.to(case.act_dtype).contiguous())
    out["bias"] = bias if with_bias else None
    return out


def as_f64(t: torch.Tensor):
    """Exact widening of a CPU tensor to a float64 numpy array."""
    return t.detach().to(torch.float64).numpy()


# ---------------------------------------------------------------------------
# the five workload families
# ---------------------------------------------------------------------------
def config1() -> List[LayerCase]:
    """Single fake-quantized linear, fp32 I/O, symmetric activations, seed 0."""
    return [LayerCase("cfg1_linear", 256, 512, 512, act_dtype=torch.float32,
                      x_symmetric=True, seed=0)]


def config2() -> List[LayerCase]:
    """BERT-base-shaped encoder linears, M = 32 x 128 tokens, bf16 activations."""
    shapes = [("qkv", 768, 2304), ("attn_out", 768, 768),
              ("ffn_up", 768, 3072), ("ffn_down", 3072, 768)]
    return [LayerCase(f"cfg2_{n}", 4096, k, o, seed=2000 + i)
            for i, (n, k, o) in enumerate(shapes)]


def config3(batch: int = 64) -> List[LayerCase]:
    """ResNet-50-shaped convolutions, NHWC bf16, W4A8, |N(0,1)| activations."""
    out = []
    stages = [(56, 64, 256), (28, 128, 512), (14, 256, 1024), (7, 512, 2048)]
    i = 0
    for hw, cin, cout in stages:
        for r, pad in ((1, 0), (3, 1)):
            out.append(LayerCase(
                f"cfg3_{hw}x{hw}_{cin}to{cout}_{r}x{r}", batch * hw * hw, r * r * cin, cout,
                w_bits=4, x_bits=8, w_std=None, x_abs=True, seed=3000 + i,
                conv=True, B=batch, H=hw, Wd=hw, Cin=cin, R=r, S=r, stride=1, pad=pad))
            i += 1
    return out


def config3_strided(batch: int = 64) -> List[LayerCase]:
    """The stride-2 layers of ResNet-50: the 7x7 input layer (3 channels stored as 8), the 3x3
    stride-2 convolution opening stages 2-4 and the 1x1 stride-2 shortcut beside each."""
    specs = [("stem", 224, 8, 64, 7, 3), ("56_128_3x3", 56, 128, 128, 3, 1), ("28_256_3x3", 28, 256, 256, 3, 1),
             ("14_512_3x3", 14, 512, 512, 3, 1), ("56_256to512_1x1", 56, 256, 512, 1, 0),
             ("28_512to1024_1x1", 28, 512, 1024, 1, 0), ("14_1024to2048_1x1", 14, 1024, 2048, 1, 0)]
    out = []
    for i, (name, hw, cin, cout, r, pad) in enumerate(specs):
        ho = (hw + 2 * pad - r) // 2 + 1
        out.append(LayerCase(f"cfg3s_{name}_s2", batch * ho * ho, r * r * cin, cout, w_bits=4, x_bits=8, w_std=None,
                             x_abs=True, seed=3100 + i, conv=True, B=batch, H=hw, Wd=hw, Cin=cin, R=r, S=r,
                             stride=2, pad=pad))
    return out


def resnet50(batch: int = 64) -> List[LayerCase]:
    """Every convolution of ResNet-50 at 224 x 224 (bottleneck blocks 3-4-6-3, stride on the 3x3
    convolution, input stored with 8 channels) and the classifier: 54 quantized layers, W4A8,
    |N(0,1)| activations.  Section 4 "Setup" quantizes all of them, input, output and shortcut
    layers included."""
    out = []

    def conv(name, hw, cin, cout, r, stride):
        pad = r // 2
        ho = (hw + 2 * pad - r) // stride + 1
        out.append(LayerCase(f"rn50_{name}", batch * ho * ho, r * r * cin, cout, w_bits=4, x_bits=8, w_std=None,
                             x_abs=True, seed=3200 + len(out), conv=True, B=batch, H=hw, Wd=hw, Cin=cin, R=r, S=r,
                             stride=stride, pad=pad))
        return ho

    conv("stem", 224, 8, 64, 7, 2)
    hw, cin = 56, 64                                    # after the 3x3 stride-2 max-pool
    for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        for b in range(blocks):
            stride = 2 if (b == 0 and stage > 0) else 1
            tag = f"s{stage + 1}b{b + 1}"
            if b == 0:
                conv(tag + "_shortcut", hw, cin, 4 * width, 1, stride)
            conv(tag + "_a", hw, cin, width, 1, 1)
            ho = conv(tag + "_b", hw, width, width, 3, stride)
            conv(tag + "_c", ho, width, 4 * width, 1, 1)
            hw, cin = ho, 4 * width
    out.append(LayerCase("rn50_fc", batch, 2048, 1000, w_bits=4, x_bits=8, w_std=None, x_abs=True,
                         seed=3200 + len(out)))
    return out


def resnet20(batch: int = 128) -> List[LayerCase]:
    """The 20 quantized layers of the CIFAR-10 ResNet-20 at 32 x 32: a 3x3 input layer (3 channels
    stored as 8), three stages of three basic blocks (two 3x3 convolutions each) with 16, 32 and
    64 channels, the first convolution of stages 2 and 3 with stride 2, parameter-free shortcuts,
    and the classifier.  W4A8, |N(0,1)| activations."""
    out = []

    def conv(name, hw, cin, cout, stride):
        ho = (hw + 2 - 3) // stride + 1
        out.append(LayerCase(f"rn20_{name}", batch * ho * ho, 9 * cin, cout, w_bits=4, x_bits=8, w_std=None,
                             x_abs=True, seed=3300 + len(out), conv=True, B=batch, H=hw, Wd=hw, Cin=cin, R=3, S=3,
                             stride=stride, pad=1))
        return ho

    conv("stem", 32, 8, 16, 1)
    hw, cin = 32, 16
    for stage, width in enumerate((16, 32, 64)):
        for b in range(3):
            stride = 2 if (b == 0 and stage > 0) else 1
            ho = conv(f"s{stage + 1}b{b + 1}_a", hw, cin, width, stride)
            conv(f"s{stage + 1}b{b + 1}_b", ho, width, width, 1)
            hw, cin = ho, width
    out.append(LayerCase("rn20_fc", batch, 64, 16, w_bits=4, x_bits=8, w_std=None, x_abs=True, seed=3300 + len(out)))
    return out


def config4(layers: int = 24, M: int = 9216) -> List[LayerCase]:
    """BERT-large-shaped stack: per block Q,K,V,O 1024->1024, FFN 1024->4096->1024."""
    out = []
    for b in range(layers):
        for j, (k, n) in enumerate([(1024, 1024)] * 4 + [(1024, 4096), (4096, 1024)]):
            out.append(LayerCase(f"cfg4_b{b}_l{j}", M, k, n, w_bits=4, x_bits=8,
                                 w_std=None, seed=4000 + 6 * b + j))
    return out


def config5(w_bits: int = 8, x_bits: int = 8) -> List[LayerCase]:
    """GEMM-shape sweep at M = 16384 tokens."""
    return [LayerCase(f"cfg5_{k}x{n}_w{w_bits}a{x_bits}", 16384, k, n,
                      w_bits=w_bits, x_bits=x_bits, seed=5000 + i)
            for i, (k, n) in enumerate([(1024, 1024), (4096, 4096),
                                        (4096, 16384), (8192, 8192)])]


def shrink(case: LayerCase, M: int) -> LayerCase:
    """Same layer with fewer rows (linear cases only) -- used where the oracle
    must finish in seconds."""
    assert not case.conv
    c = LayerCase(**{k: v for k, v in case.__dict__.items() if k != "tensors"})
    c.M = M
    c.name = f"{case.name}_M{M}"
    return c
