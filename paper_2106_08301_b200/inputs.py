"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU checker.

This module holds no arithmetic of the method: it only draws random tensors of
the shapes and distributions of the five synthetic workloads and names them.
Weights are fp32; activations are drawn in fp32 and rounded once to bf16, and
those bf16 values are what every consumer sees.

The workloads stand in for the paper's CNN layers (Section 4.2: VGG-16,
ResNet-50, MobileNet-V2 convolutions and fully connected layers), whose trained
weights and datasets are not shipped with this library: 3x3 and 1x1 ResNet-style
convolutions, a small linear layer, and two large linear layers.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Tuple

import torch

SEED_BASE = 21060830


def seed_for(config: int, case: int = 0) -> int:
    return SEED_BASE + 1000 * int(config) + int(case)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def normal_weights(rows: int, cols: int, std: float, seed: int) -> torch.Tensor:
    """fp32 [rows, cols] ~ N(0, std^2), CPU, contiguous."""
    w = torch.randn(rows, cols, generator=_gen(seed), dtype=torch.float32)
    return (w * float(std)).contiguous()


def normal_activations_bf16(shape: Tuple[int, ...], seed: int) -> torch.Tensor:
    """bf16 tensor ~ N(0,1) rounded once to bf16, CPU, contiguous."""
    x = torch.randn(*shape, generator=_gen(seed), dtype=torch.float32)
    return x.to(torch.bfloat16).contiguous()


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic workload.

    rows x cols is the weight viewed as W[N][K] (K = reduction axis; for a
    convolution K = cin*kh*kw in [cout, cin, kh, kw] order).  `unified_permille`
    counts unified AND pruned blocks together, `pruned_permille` the pruned ones.
    """
    name: str
    config: int
    rows: int
    cols: int
    block: int
    unified_permille: int
    pruned_permille: int
    weight_std: float
    m: int = 0                       # GEMM rows of the activation matrix (0: conv)
    conv: Optional[Tuple[int, int, int, int, int, int, int, int]] = None
    # conv = (batch, cin, h, w, kh, kw, stride, pad)

    @property
    def n_blocks(self) -> int:
        return self.rows * self.cols // self.block

    def weights(self, case: int = 0) -> torch.Tensor:
        if self.name.startswith("proj_p"):
            case += 900 + int(self.name[len("proj_p"):].split("_b")[0])      # one tensor per size
        return normal_weights(self.rows, self.cols, self.weight_std,
                              seed_for(self.config, case))

    def activations(self, case: int = 0, m: Optional[int] = None) -> torch.Tensor:
        s = seed_for(self.config, 500 + case)
        if self.conv is not None:
            n, c, h, w = self.conv[:4]
            return normal_activations_bf16((n, c, h, w), s)
        return normal_activations_bf16((int(m if m is not None else self.m), self.cols), s)


WORKLOADS = {
    # 256x256 linear, batch 64, b=4, 50% unified of which half pruned
    "c1_linear": Workload("c1_linear", 1, 256, 256, 4, 500, 250, 0.02, m=64),
    # 3x3 conv 128->128, 28x28, batch 32, Kaiming-normal std = sqrt(2/1152)
    "c2_conv3x3": Workload("c2_conv3x3", 2, 128, 1152, 4, 600, 300, math.sqrt(2.0 / 1152.0),
                           conv=(32, 128, 28, 28, 3, 3, 1, 1)),
    # 1x1 conv as GEMM, M = 64*56*56
    "c3_conv1x1": Workload("c3_conv1x1", 3, 1024, 256, 8, 750, 500, 0.02, m=200704),
    # transformer FFN up-projection 4096 -> 16384, 8192 tokens
    "c4_ffn": Workload("c4_ffn", 4, 16384, 4096, 16, 800, 600, 0.02, m=8192),
}


def sweep_workload(block: int, pruned_permille: int) -> Workload:
    """4096x4096 sweep point: unified fraction = pruned + 10% (capped at 100%)."""
    u = min(1000, pruned_permille + 100)
    return Workload(f"c5_sweep_b{block}_p{pruned_permille}", 5, 4096, 4096, block, u,
                    pruned_permille, 0.02, m=8192)


def projection_sweep_workload(log2_params: int, block: int) -> Workload:
    """Projection-only point of the size sweep: 2**log2_params weights, 50 % unified of which half
    pruned; no activations (m = 0)."""
    rows, cols = projection_sweep_shape(log2_params)
    return Workload(f"proj_p{log2_params}_b{block}", 5, rows, cols, block, 500, 250, 0.02, m=0)


def projection_sweep_shape(log2_params: int) -> Tuple[int, int]:
    """Square-ish [rows, cols] with rows*cols = 2**log2_params and cols a multiple of 64."""
    cols = 1 << ((log2_params + 1) // 2)
    rows = (1 << log2_params) // cols
    return rows, cols
