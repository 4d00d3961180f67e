"""Seeded synthetic inputs for the quantized-layer workloads.

This module only *generates data and shapes*: random tensors with the stated
distributions, layer-shape lists, and the per-tensor range that a workload
prescribes.  It holds none of the method's arithmetic (no quantizer, no packing,
no contraction) and imports neither the CUDA binding nor the CPU oracle, so both
can be driven from the same bytes.

Every tensor comes from ``numpy.random.default_rng([seed, config, layer, tensor])``
so that a tensor can be regenerated alone.  Activations are NHWC (or [rows, k]),
convolution weights are [Cout, R, S, Cin].
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

TENSOR_A, TENSOR_W = 0, 1


def rng_for(seed: int, config: int, layer: int, tensor: int) -> np.random.Generator:
    return np.random.default_rng([seed, config, layer, tensor])


def normal_f32(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return x


def per_tensor_scale(x: np.ndarray, bits: int) -> np.float32:
    """Workload rule for the grid step of a tensor: max|x| / (2^bits - 1), in binary32."""
    m = np.float32(np.max(np.abs(x))) if x.size else np.float32(0.0)
    if not np.isfinite(m) or m <= 0:
        m = np.float32(1.0)
    return np.float32(m / np.float32((1 << bits) - 1))


@dataclass
class FcCase:
    """One fully-connected layer: a [Mg, Kg] fp32, w fp32 either [Ng, Kg] or k-major [Kg, Ng]."""
    name: str
    a: np.ndarray
    w: np.ndarray
    k_major: bool
    ab: int
    wb: int
    relu: bool = False

    @property
    def Mg(self): return self.a.shape[0]
    @property
    def Kg(self): return self.a.shape[1]
    @property
    def Ng(self): return self.w.shape[1] if self.k_major else self.w.shape[0]


@dataclass
class ConvShape:
    name: str
    N: int
    H: int
    W: int
    C: int
    Cout: int
    R: int
    S: int
    stride: int
    pad: int
    ab: int
    wb: int
    pool_after: bool = False      # 2x2 max-pool follows (done by the harness, outside the library)
    branch: bool = False          # 1x1 projection evaluated on its block's input, not chained

    @property
    def Ho(self): return (self.H + 2 * self.pad - self.R) // self.stride + 1
    @property
    def Wo(self): return (self.W + 2 * self.pad - self.S) // self.stride + 1
    @property
    def Mg(self): return self.N * self.Ho * self.Wo
    @property
    def Kg(self): return self.R * self.S * self.C
    @property
    def int_macs(self): return self.Mg * self.Cout * self.Kg


@dataclass
class ConvCase:
    shape: ConvShape
    a: np.ndarray          # [N,H,W,C] fp32
    w: np.ndarray          # [Cout,R,S,C] fp32
    relu: bool = False


def fc_config1(seed: int = 0) -> FcCase:
    """2-bit x 2-bit FC: A[64,512] = min(ReLU(N(0,1)), 3), W[512,256] ~ N(0, 0.05) stored k-major."""
    a = normal_f32(rng_for(seed, 1, 0, TENSOR_A), (64, 512))
    a = np.minimum(np.maximum(a, np.float32(0)), np.float32(3.0))
    w = normal_f32(rng_for(seed, 1, 0, TENSOR_W), (512, 256), 0.05)
    return FcCase("fc_64x256x512_w2a2", a, w, True, 2, 2)


def conv_config2(seed: int = 0, batch: int = 32) -> ConvCase:
    """2-bit x 2-bit 3x3 conv, 256->256 channels, 14x14, stride 1 pad 1 (implicit GEMM 6272x256x2304)."""
    shp = ConvShape("conv3x3_256_14", batch, 14, 14, 256, 256, 3, 3, 1, 1, 2, 2)
    a = np.maximum(normal_f32(rng_for(seed, 2, 0, TENSOR_A), (batch, 14, 14, 256)), np.float32(0))
    w = normal_f32(rng_for(seed, 2, 0, TENSOR_W), (256, 3, 3, 256), 0.02)
    return ConvCase(shp, a, w)


GEMM_SWEEP_BITS = [(1, 1), (2, 2), (3, 3), (4, 4), (2, 4)]   # (wb, ab)


def gemm_config3(seed: int = 0, n: int = 4096, wb: int = 2, ab: int = 2, variant: int = 0) -> FcCase:
    """Square GEMM: A = min(|N(0,1)|, 4), W ~ N(0, 0.02) as [Ng, Kg]. `variant` draws another A."""
    a = np.abs(normal_f32(rng_for(seed, 3, variant, TENSOR_A), (n, n)))
    np.minimum(a, np.float32(4.0), out=a)
    w = normal_f32(rng_for(seed, 3, 0, TENSOR_W), (n, n), 0.02)
    return FcCase(f"gemm_{n}_w{wb}a{ab}", a, w, False, ab, wb)


def resnet18_shapes(batch: int = 256, ab: int = 3, wb: int = 3) -> list[ConvShape]:
    """Quantized convolutions of a ResNet-18-shaped stack at 224x224 input (after the fp32 stem:
    7x7/2 conv + 3x3/2 max-pool -> 56x56x64).  16 3x3 convs in sequence plus three 1x1/2
    projections, each evaluated on the input of its stage."""
    L: list[ConvShape] = []
    hw, c = 56, 64
    for stage, cout in enumerate([64, 128, 256, 512]):
        for i in range(4):
            stride = 2 if (stage > 0 and i == 0) else 1
            L.append(ConvShape(f"s{stage + 1}c{i + 1}_3x3_{c}_{cout}_{hw}", batch, hw, hw, c, cout, 3, 3,
                               stride, 1, ab, wb))
            if stride == 2:
                L.append(ConvShape(f"s{stage + 1}proj_1x1_{c}_{cout}_{hw}", batch, hw, hw, c, cout, 1, 1,
                                   2, 0, ab, wb, branch=True))
                hw //= 2
            c = cout
    return L


# Per-stage bit widths of the paper's mixed-precision ResNet-18 (Table 4): (activation bits M, weight bits K)
# for Conv2_x .. Conv5_x; the stem (Conv1) and the FC layer stay outside the library (their widths only enter
# the compression ratio).
RESNET18_MIXED = {
    1: {"stem_wb": 8, "stages": [(8, 8), (8, 7), (8, 7), (8, 6)], "fc_wb": 8, "compression": 5.0},
    2: {"stem_wb": 8, "stages": [(4, 5), (4, 3), (4, 2), (4, 2)], "fc_wb": 6, "compression": 14.1},
}


def resnet18_mixed_shapes(precision: int, batch: int = 256) -> list[ConvShape]:
    """The ResNet-18-shaped stack with the per-stage (activation, weight) widths of Table 4, Precision#1 or #2."""
    stages = RESNET18_MIXED[precision]["stages"]
    out = []
    for s in resnet18_shapes(batch):
        stage = int(s.name[1]) - 1                      # names start with s<stage>
        ab, wb = stages[stage]
        out.append(ConvShape(s.name + f"_a{ab}w{wb}", s.N, s.H, s.W, s.C, s.Cout, s.R, s.S, s.stride, s.pad, ab, wb,
                             branch=s.branch))
    return out


def resnet18_weight_bits(precision: int) -> tuple[int, int]:
    """(bits of all weights at the table's widths, bits at fp32) for the whole ResNet-18: 7x7 stem, the 19
    quantized convolutions, and the 512x1000 FC layer (biases and normalisation parameters not counted)."""
    cfg = RESNET18_MIXED[precision]
    stem, fc = 7 * 7 * 3 * 64, 512 * 1000
    q = stem * cfg["stem_wb"] + fc * cfg["fc_wb"]
    n = stem + fc
    for s in resnet18_mixed_shapes(precision, batch=1):
        params = s.Cout * s.R * s.S * s.C
        q += params * s.wb
        n += params
    return q, 32 * n


def vgg16_shapes(batch: int = 64, ab: int = 4, wb: int = 4) -> list[ConvShape]:
    """13 3x3 stride-1 pad-1 convolutions of a VGG-16-shaped stack at 224x224x3, 2x2 max-pool after each block."""
    cfg = [(64, 2), (128, 2), (256, 3), (512, 3), (512, 3)]
    L: list[ConvShape] = []
    hw, c = 224, 3
    for b, (cout, reps) in enumerate(cfg):
        for i in range(reps):
            L.append(ConvShape(f"b{b + 1}c{i + 1}_3x3_{c}_{cout}_{hw}", batch, hw, hw, c, cout, 3, 3, 1, 1,
                               ab, wb, pool_after=(i == reps - 1)))
            c = cout
        hw //= 2
    return L


def he_weights(seed: int, config: int, layer: int, shp: ConvShape) -> np.ndarray:
    fan_in = shp.R * shp.S * shp.C
    return normal_f32(rng_for(seed, config, layer, TENSOR_W), (shp.Cout, shp.R, shp.S, shp.C),
                      float(np.sqrt(2.0 / fan_in)))


def layer_input(seed: int, config: int, layer: int, shp: ConvShape, signed: bool = False) -> np.ndarray:
    """Stand-alone input for one layer of a stack: N(0,1) (signed, first layer of an image stack)
    or ReLU(N(0,1)) (what a layer after a ReLU sees)."""
    a = normal_f32(rng_for(seed, config, layer, TENSOR_A), (shp.N, shp.H, shp.W, shp.C))
    if not signed:
        np.maximum(a, np.float32(0), out=a)
    return a


def maxpool2x2_nhwc(x: np.ndarray) -> np.ndarray:
    """2x2 stride-2 max-pool done by the harness between blocks of a stack (not a library call)."""
    n, h, w, c = x.shape
    return x.reshape(n, h // 2, 2, w // 2, 2, c).max(axis=(2, 4))


def sample_pairs(seed: int, Mg: int, Ng: int, count: int, full_rows: int = 0):
    """Output coordinates to check at sizes the oracle cannot finish in full: `full_rows`
    complete rows spread over the matrix (first, last, and tile edges included) plus
    `count` uniformly random (row, col) pairs."""
    rng = np.random.default_rng([seed, 99, Mg, Ng])
    rows, cols = [], []
    if full_rows > 0:
        pick = {0, Mg - 1, min(Mg - 1, 127), min(Mg - 1, 128), Mg // 2}
        while len(pick) < min(full_rows, Mg):
            pick.add(int(rng.integers(0, Mg)))
        for r in sorted(pick):
            rows.append(np.full(Ng, r, dtype=np.int64))
            cols.append(np.arange(Ng, dtype=np.int64))
    if count > 0:
        rows.append(rng.integers(0, Mg, size=count, dtype=np.int64))
        cols.append(rng.integers(0, Ng, size=count, dtype=np.int64))
    return np.concatenate(rows), np.concatenate(cols)
