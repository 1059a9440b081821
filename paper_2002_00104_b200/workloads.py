"""Seeded synthetic inputs for the PWLQ hot path (no quantizer arithmetic lives here).

The paper evaluates on pretrained torchvision CNN weights and on activations
of those networks (Sec. 5), which are not available offline; it argues that
both are bell-shaped with long tails, close to Gaussian or Laplacian (Sec. 1,
Sec. 3.1).  The tensors below therefore have the *shapes* of those networks'
layers and Gaussian / Laplacian *values*, drawn from numpy's PCG64 generator
(``numpy.random.default_rng(seed)``) on the host, so that every consumer reads
the same bytes.

A workload is a set of rows ("channels", Sec. 5: weights are quantized per
output channel, activations per layer).  Rows are stored back to back in one
flat fp32 array; ``row_offsets[c]`` is the flat index of row ``c``'s first
value, ``row_offsets[C]`` the total length.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np


@dataclass
class Workload:
    name: str
    x: np.ndarray                    # flat float32
    row_offsets: np.ndarray          # int64 [C + 1]
    bits: int
    K: int
    tensors: List[Tuple[str, int, int, int]] = field(default_factory=list)
    # (layer name, rows, row length, first row index)

    @property
    def C(self) -> int:
        return int(self.row_offsets.size - 1)

    @property
    def total(self) -> int:
        return int(self.row_offsets[-1])

    @property
    def elem_cand(self) -> int:
        """Number of (value, candidate) evaluations of one search."""
        return self.total * self.K

    def uniform_n(self):
        """Row length if all rows are equally long, else None."""
        d = np.diff(self.row_offsets)
        return int(d[0]) if d.size and np.all(d == d[0]) else None


def ratio_grid(K: int) -> np.ndarray:
    """Candidate ratios p/m = (k+1)/K, k = 0..K-1, each one fp32 division."""
    k = np.arange(1, K + 1, dtype=np.float32)
    return (k / np.float32(K)).astype(np.float32)


def resnet50_layers() -> List[Tuple[str, int, int]]:
    """(name, out_channels, fan_in) of every conv and the fc of ResNet-50 v1.5."""
    layers = [("stem.conv7x7", 64, 3 * 7 * 7)]
    cin = 64
    for si, (blocks, w) in enumerate(zip((3, 4, 6, 3), (64, 128, 256, 512))):
        for bi in range(blocks):
            pre = f"s{si + 1}.b{bi}"
            layers.append((pre + ".conv1x1a", w, cin))
            layers.append((pre + ".conv3x3", w, w * 9))
            layers.append((pre + ".conv1x1b", 4 * w, w))
            if bi == 0:
                layers.append((pre + ".down1x1", 4 * w, cin))
            cin = 4 * w
    layers.append(("fc", 1000, 2048))
    return layers


def mobilenetv2_layers() -> List[Tuple[str, int, int]]:
    """(name, out_channels, fan_in) of every conv and the fc of MobileNetV2 (width 1.0)."""
    layers = [("stem.conv3x3", 32, 3 * 3 * 3)]
    cin = 32
    settings = ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1))
    bi = 0
    for t, c, reps, _stride in settings:
        for _ in range(reps):
            hid = cin * t
            pre = f"ir{bi}"
            if t != 1:
                layers.append((pre + ".expand1x1", hid, cin))
            layers.append((pre + ".dw3x3", hid, 9))
            layers.append((pre + ".project1x1", c, hid))
            cin = c
            bi += 1
    layers.append(("last.conv1x1", 1280, cin))
    layers.append(("fc", 1000, 1280))
    return layers


def _assemble(name, parts, layers, bits, K) -> Workload:
    offs = [0]
    tensors = []
    row = 0
    for (lname, C, n), _ in zip(layers, parts):
        tensors.append((lname, C, n, row))
        for _c in range(C):
            offs.append(offs[-1] + n)
        row += C
    x = np.concatenate([p.reshape(-1) for p in parts]).astype(np.float32, copy=False)
    return Workload(name, np.ascontiguousarray(x), np.asarray(offs, dtype=np.int64), bits, K,
                    tensors)


def single_conv(seed: int = 0) -> Workload:
    """One 64x64x3x3 conv weight, Laplace(0, 0.02); per-tensor 4-bit, K = 100."""
    rng = np.random.default_rng(seed)
    x = rng.laplace(0.0, 0.02, size=64 * 64 * 3 * 3).astype(np.float32)
    return Workload("single_conv_64x64x3x3", x, np.array([0, x.size], dtype=np.int64), 4, 100,
                    [("conv", 1, x.size, 0)])


def resnet50(seed: int = 1000) -> Workload:
    """All ResNet-50 v1.5 conv + fc weights, N(0, sqrt(2/fan_in)); per-channel 4-bit, K = 256."""
    layers = resnet50_layers()
    parts = []
    for li, (_n, C, fan_in) in enumerate(layers):
        rng = np.random.default_rng(seed + li)
        parts.append(rng.normal(0.0, np.sqrt(2.0 / fan_in), size=(C, fan_in)).astype(np.float32))
    return _assemble("resnet50_v1.5_weights", parts, layers, 4, 256)


def mobilenetv2(seed: int = 2000) -> Workload:
    """MobileNetV2 weights, Laplace with per-channel scale 10^U(-3,-1); per-channel 3-bit, K = 256."""
    layers = mobilenetv2_layers()
    parts = []
    for li, (_n, C, fan_in) in enumerate(layers):
        rng = np.random.default_rng(seed + li)
        scale = np.power(10.0, rng.uniform(-3.0, -1.0, size=(C, 1)))
        parts.append((rng.laplace(0.0, 1.0, size=(C, fan_in)) * scale).astype(np.float32))
    return _assemble("mobilenetv2_weights", parts, layers, 3, 256)


def relu_activation(seed: int = 4000, shape=(32, 256, 56, 56)) -> Workload:
    """ReLU(N(0,1)) activation with 1 % |Cauchy(0,1)| outliers; per-tensor 4-bit, K = 1024."""
    rng = np.random.default_rng(seed)
    total = int(np.prod(shape))
    x = np.maximum(rng.standard_normal(total, dtype=np.float32), np.float32(0.0))
    n_out = total // 100
    pos = rng.choice(total, size=n_out, replace=False)
    x[pos] = np.abs(rng.standard_cauchy(n_out)).astype(np.float32)
    return Workload("relu_activation_" + "x".join(map(str, shape)), x,
                    np.array([0, total], dtype=np.int64), 4, 1024, [("act", 1, total, 0)])


def laplace_matrix(seed: int = 5000, rows: int = 4096, cols: int = 4096, bits: int = 4,
                   K: int = 256) -> Workload:
    """rows x cols Laplace(0, 0.01) weight, one channel per row."""
    rng = np.random.default_rng(seed)
    x = rng.laplace(0.0, 0.01, size=(rows, cols)).astype(np.float32)
    offs = np.arange(rows + 1, dtype=np.int64) * cols
    return Workload(f"laplace_{rows}x{cols}", x.reshape(-1), offs, bits, K,
                    [("w", rows, cols, 0)])


def small_mixed(seed: int = 7, bits: int = 4, K: int = 64) -> Workload:
    """A small ragged case: a few rows of each awkward length (tile tails, unaligned rows)."""
    lengths = [1, 9, 9, 9, 27, 64, 147, 147, 256, 576, 1000, 2304, 4607, 9001]
    rng = np.random.default_rng(seed)
    parts, layers = [], []
    for i, n in enumerate(lengths):
        if i % 2 == 0:
            v = rng.normal(0.0, 0.05, size=(1, n))
        else:
            v = rng.laplace(0.0, 0.02, size=(1, n))
        parts.append(v.astype(np.float32))
        layers.append((f"row{i}", 1, n))
    return _assemble("small_mixed", parts, layers, bits, K)
