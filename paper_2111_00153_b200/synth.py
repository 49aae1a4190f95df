"""Seeded synthetic inputs shaped like the paper's ResNet-18 and BERT workloads.

This module only draws random tensors and lists layer shapes.  It holds none of the
method's arithmetic (no quantizer, no row assignment, no contraction) so that the CPU
oracle and the CUDA library can both be fed from it without sharing any logic.

Generator: ``numpy.random.Generator(PCG64(seed))``, seed = 1000 * config + index.
"""
from __future__ import annotations

from dataclasses import dataclass
import numpy as np

RATIO_RMSMP1 = (60, 35, 5)   # PoT-4 : Fixed-4 : Fixed-8 used on the smaller FPGA (Table 6)
RATIO_RMSMP2 = (65, 30, 5)   # ... on the larger FPGA (Table 6)
RATIO_SWEEP = ((0, 100, 0), (100, 0, 0), (60, 35, 5), (50, 40, 10))


def rng(config: int, index: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(1000 * config + index))


def weights_normal(g: np.random.Generator, shape, sigma: float = 0.02) -> np.ndarray:
    """BERT-style initialisation: N(0, sigma^2), fp32."""
    return (g.standard_normal(shape, dtype=np.float32) * np.float32(sigma)).astype(np.float32)


def weights_kaiming(g: np.random.Generator, M: int, Cin: int, kh: int, kw: int) -> np.ndarray:
    """Kaiming-normal filters [M][Cin][kh][kw], sigma = sqrt(2 / fan_in), fp32.

    Each filter additionally gets its own gain drawn uniformly from [0.5, 1.5] so that
    the per-filter variances differ the way trained filters' do (a pure i.i.d. draw would
    make the variance ranking noise only)."""
    sigma = np.float32(np.sqrt(2.0 / (Cin * kh * kw)))
    w = g.standard_normal((M, Cin, kh, kw), dtype=np.float32) * sigma
    gain = g.uniform(0.5, 1.5, size=(M, 1, 1, 1)).astype(np.float32)
    return (w * gain).astype(np.float32)


def alpha_rows(W: np.ndarray) -> np.ndarray:
    """Per-row clip value handed to the quantizer: max |w| of the row (1 for an all-zero row)."""
    a = np.abs(W.reshape(W.shape[0], -1)).max(axis=1).astype(np.float32)
    a[a == 0] = np.float32(1.0)
    return a


def act_codes_uniform(g: np.random.Generator, shape) -> np.ndarray:
    """4-bit unsigned activation codes drawn uniformly from 0..15 (int8 storage)."""
    return g.integers(0, 16, size=shape, dtype=np.int8)


def act_halfnormal(g: np.random.Generator, shape) -> np.ndarray:
    """Post-ReLU-like activations |N(0,1)|, fp32; quantized U4 with alpha_a = 3."""
    return np.abs(g.standard_normal(shape, dtype=np.float32))


def act_normal(g: np.random.Generator, shape) -> np.ndarray:
    """N(0,1) activations, fp32; quantized S4 with alpha_a = 3."""
    return g.standard_normal(shape, dtype=np.float32)


ALPHA_ACT = 3.0  # three standard deviations of the generating distribution


@dataclass(frozen=True)
class ConvShape:
    name: str
    M: int        # output filters = weight rows
    Cin: int
    k: int        # square kernel
    stride: int
    pad: int
    H: int        # input height = width
    count: int = 1  # how many identical layers of this shape the network has

    @property
    def Ho(self) -> int:
        return (self.H + 2 * self.pad - self.k) // self.stride + 1

    @property
    def K(self) -> int:
        return self.Cin * self.k * self.k

    def macs(self, batch: int) -> int:
        return self.M * self.K * batch * self.Ho * self.Ho


def resnet18_convs() -> list[ConvShape]:
    """All 3x3 and 1x1 convolutions of ResNet-18 at 224x224 input (19 layers)."""
    L = []
    L.append(ConvShape("l1.conv3x3", 64, 64, 3, 1, 1, 56, 4))
    for i, (cin, cout, h) in enumerate(((64, 128, 56), (128, 256, 28), (256, 512, 14)), start=2):
        L.append(ConvShape(f"l{i}.conv3x3_s2", cout, cin, 3, 2, 1, h, 1))
        L.append(ConvShape(f"l{i}.conv3x3", cout, cout, 3, 1, 1, h // 2, 3))
        L.append(ConvShape(f"l{i}.down1x1_s2", cout, cin, 1, 2, 0, h, 1))
    return L


RESNET18_CONV1 = ConvShape("conv1_7x7", 64, 3, 7, 2, 3, 224, 1)   # not in the 3x3/1x1 stack
RESNET18_FC_MACS = 512 * 1000

CONFIG2_CONV = ConvShape("conv256_14", 256, 256, 3, 1, 1, 14, 1)   # batch 32

BERT_BASE_LINEARS = (("qkv", 2304, 768), ("attn_out", 768, 768), ("ffn1", 3072, 768),
                     ("ffn2", 768, 3072))       # (name, M, K), N = 4096 tokens
BERT_BASE_TOKENS = 4096
BERT_LARGE_LINEARS = (("h2h", 1024, 1024), ("ffn1", 4096, 1024), ("ffn2", 1024, 4096))
BERT_LARGE_TOKENS = (1, 8, 128)
