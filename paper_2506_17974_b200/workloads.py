"""Seeded synthetic gradient sets shaped like the workloads LQ-SGD is evaluated on.

This module only *describes and draws inputs*: layer shape lists and random
gradient tensors.  It holds none of the compression arithmetic and is the one
module both the CUDA path's tests/benchmarks and the CPU oracle's tests feed
from, so that both sides always see bit-identical fp32 arrays.

Shapes follow the matricisation the paper's byte counts imply (Tables I-III):
a conv weight [C_out, C_in, k, k] becomes an n x m matrix with n = C_out rows
and m = C_in*k*k columns (Section IV notation, G in R^{n x m}); every 1-D tensor
(bias, batch-norm scale/shift) bypasses the low-rank path.

A layer is a tuple (rows, cols).  cols == 1 marks a 1-D tensor of length rows.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Sequence, Tuple

import torch

Shape = Tuple[int, int]


def _resnet18_convs(in_channels: int) -> List[Shape]:
    """Weight matrices of a CIFAR-style ResNet-18, in network order (fc excluded)."""
    s: List[Shape] = [(64, in_channels * 9)]            # stem 3x3 conv
    s += [(64, 64 * 9)] * 4                             # stage 1: 2 blocks x 2 convs
    s += [(128, 64 * 9)] + [(128, 128 * 9)] * 3 + [(128, 64)]        # stage 2 + 1x1 shortcut
    s += [(256, 128 * 9)] + [(256, 256 * 9)] * 3 + [(256, 128)]      # stage 3
    s += [(512, 256 * 9)] + [(512, 512 * 9)] * 3 + [(512, 256)]      # stage 4
    return s


def _resnet18_vectors(num_classes: int) -> List[Shape]:
    """1-D tensors of the same network: one (scale, shift) pair per batch-norm, fc bias."""
    bn_channels = [64] * 5 + [128] * 5 + [256] * 5 + [512] * 5   # one BN after every conv
    v: List[Shape] = []
    for c in bn_channels:
        v += [(c, 1), (c, 1)]
    v.append((num_classes, 1))
    return v


def resnet18_layers(num_classes: int = 10, in_channels: int = 3) -> List[Shape]:
    """All trainable tensors of ResNet-18: 21 matrices followed by the 1-D tensors."""
    return _resnet18_convs(in_channels) + [(num_classes, 512)] + _resnet18_vectors(num_classes)


def mnist_cnn_layers() -> List[Shape]:
    """MNIST-style CNN: conv1 32x25, conv2 64x800, fc1 512x3136, fc2 10x512 + biases."""
    return [(32, 25), (64, 800), (512, 3136), (10, 512), (32, 1), (64, 1), (512, 1), (10, 1)]


def is_matrix(shape: Shape) -> bool:
    return shape[0] > 1 and shape[1] > 1


def matrix_elements(layers: Sequence[Shape]) -> int:
    return sum(n * m for n, m in layers if is_matrix((n, m)))


def vector_elements(layers: Sequence[Shape]) -> int:
    return sum(n * m for n, m in layers if not is_matrix((n, m)))


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration."""
    name: str
    layers: Tuple[Shape, ...]
    rank: int
    bits: int
    workers: int
    steps: int
    dist: str          # "normal" | "student_t3"
    scale: str         # "const:<sigma>" | "fan_in"  (sigma = 1/sqrt(cols))
    alpha: float = 127.0
    seed: int = 0

    @property
    def gradient_bytes_per_worker(self) -> int:
        return 4 * sum(n * m for n, m in self.layers)


def config1() -> Workload:
    return Workload("single_256x576", ((256, 576),), rank=2, bits=4, workers=1, steps=10,
                    dist="normal", scale="const:0.01")


def config2() -> Workload:
    return Workload("mnist_cnn", tuple(mnist_cnn_layers()), rank=4, bits=4, workers=4, steps=50,
                    dist="normal", scale="fan_in")


def config3(workers: int = 8, rank: int = 2, bits: int = 4, num_classes: int = 10) -> Workload:
    return Workload("resnet18_cifar", tuple(resnet18_layers(num_classes)), rank=rank, bits=bits,
                    workers=workers, steps=100, dist="student_t3", scale="fan_in")


def config4(rows: int, cols: int) -> Workload:
    return Workload(f"large_{rows}x{cols}", ((rows, cols),), rank=8, bits=4, workers=1, steps=20,
                    dist="normal", scale="const:0.01")


CONFIG4_SIZES = ((1024, 4096), (4096, 4096), (4096, 16384), (8192, 25088))


def config5(rank: int, bits: int) -> Workload:
    w = config3(workers=16, rank=rank, bits=bits, num_classes=100)
    return dataclasses.replace(w, name=f"resnet18_cifar100_r{rank}_b{bits}")


def _stream_seed(seed: int, step: int, worker: int, layer: int) -> int:
    """Distinct 63-bit seed per (seed, step, worker, layer): a splitmix64-style integer mix."""
    x = (seed * 0x9E3779B97F4A7C15 + step * 0xBF58476D1CE4E5B9
         + worker * 0x94D049BB133111EB + layer * 0xD6E8FEB86659FD93 + 0x2545F4914F6CDD1D)
    x &= (1 << 64) - 1
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & ((1 << 64) - 1)
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & ((1 << 64) - 1)
    x ^= x >> 31
    return x & ((1 << 63) - 1)


def draw_tensor(shape: Shape, dist: str, sigma: float, seed: int, device="cpu") -> torch.Tensor:
    """One fp32 tensor of `shape`; normal, or Student-t with 3 degrees of freedom, times sigma."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    n, m = shape
    if dist == "normal":
        x = torch.randn((n, m), generator=gen, device=device, dtype=torch.float32)
    elif dist == "student_t3":
        z = torch.randn((4, n, m), generator=gen, device=device, dtype=torch.float32)
        x = z[0] / torch.sqrt((z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / 3.0)
    else:
        raise ValueError(f"unknown distribution {dist!r}")
    return (x * sigma).contiguous()


def layer_sigma(wl: Workload, shape: Shape) -> float:
    if not is_matrix(shape):
        return 0.01
    if wl.scale == "fan_in":
        return 1.0 / math.sqrt(shape[1])
    if wl.scale.startswith("const:"):
        return float(wl.scale.split(":", 1)[1])
    raise ValueError(wl.scale)


def draw_gradients(wl: Workload, step: int, device="cpu") -> List[List[torch.Tensor]]:
    """grads[worker][layer]: the step's fp32 gradient of every layer for every worker."""
    out = []
    for w in range(wl.workers):
        per_layer = []
        for li, shape in enumerate(wl.layers):
            dist = wl.dist if is_matrix(shape) else "normal"
            per_layer.append(draw_tensor(shape, dist, layer_sigma(wl, shape),
                                         _stream_seed(wl.seed, step, w, li), device))
        out.append(per_layer)
    return out
