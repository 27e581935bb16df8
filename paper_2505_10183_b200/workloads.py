"""Seeded synthetic workloads: tensor-shape lists, rank/group layouts and gradient values.

This module holds none of the method's arithmetic.  It only says *what the inputs
look like*: gradient tensor shapes of the CNNs the paper's kind of training job uses
(Section IV-B trains MobileNetV2; ResNet-18/50 are the usual companions), how the
simulated ranks split into vendor groups (Section III-A), the per-rank step times or
batch shares (Section III-C), and i.i.d. N(0, sigma=1e-3) gradient values from fixed
seeds.  Both the CUDA path and the CPU oracle are fed from here.

The shape lists are generated from the published architecture tables (He et al. 2016
for ResNet, Sandler et al. 2018 for MobileNetV2) in the parameter order the common
implementations use: convolution weight, then batch-norm weight and bias.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from math import prod
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

Shape = Tuple[int, ...]

SEED_BASE = 0x4B540000
SIGMA = 1.0e-3
MIB = 1 << 20


# ----------------------------------------------------------------------------- shape lists
def _bn(c: int) -> List[Shape]:
    return [(c,), (c,)]


def resnet18_shapes(num_classes: int = 10) -> List[Shape]:
    s: List[Shape] = [(64, 3, 7, 7)] + _bn(64)
    inp = 64
    for width, stride in ((64, 1), (128, 2), (256, 2), (512, 2)):
        for block in range(2):
            st = stride if block == 0 else 1
            s += [(width, inp, 3, 3)] + _bn(width) + [(width, width, 3, 3)] + _bn(width)
            if st != 1 or inp != width:
                s += [(width, inp, 1, 1)] + _bn(width)
            inp = width
    s += [(num_classes, 512), (num_classes,)]
    return s


def resnet50_shapes(num_classes: int = 1000) -> List[Shape]:
    s: List[Shape] = [(64, 3, 7, 7)] + _bn(64)
    inp = 64
    for width, blocks, stride in ((64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)):
        out = width * 4
        for block in range(blocks):
            st = stride if block == 0 else 1
            s += [(width, inp, 1, 1)] + _bn(width)
            s += [(width, width, 3, 3)] + _bn(width)
            s += [(out, width, 1, 1)] + _bn(out)
            if st != 1 or inp != out:
                s += [(out, inp, 1, 1)] + _bn(out)
            inp = out
    s += [(num_classes, 2048), (num_classes,)]
    return s


def mobilenet_v2_shapes(num_classes: int = 1000) -> List[Shape]:
    s: List[Shape] = [(32, 3, 3, 3)] + _bn(32)
    inp = 32
    for t, c, n, _stride in ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                             (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)):
        for _ in range(n):
            hidden = inp * t
            if t != 1:
                s += [(hidden, inp, 1, 1)] + _bn(hidden)      # expansion
            s += [(hidden, 1, 3, 3)] + _bn(hidden)            # depthwise
            s += [(c, hidden, 1, 1)] + _bn(c)                 # linear projection
            inp = c
    s += [(1280, inp, 1, 1)] + _bn(1280)
    s += [(num_classes, 1280), (num_classes,)]
    return s


TINY_SHAPES: List[Shape] = [(16, 3, 3, 3), (16,), (32, 16, 3, 3), (32,), (10, 512), (10,)]


def numels(shapes: Sequence[Shape]) -> List[int]:
    return [int(prod(sh)) for sh in shapes]


# ----------------------------------------------------------------------------- workloads
@dataclass
class Workload:
    """One synchronisation problem: who the ranks are and what they hold."""
    name: str
    config_id: int
    shapes: List[Shape]
    dtype: str                       # "f32" or "bf16": gradient element type
    group_of: List[int]              # rank -> group
    shares: Optional[List[int]]      # batch shares, or None when they come from step_times
    step_times: Optional[List[float]] = None
    global_batch: int = 256
    bucket_cap_bytes: int = 25 * MIB
    staged: bool = False             # partials cross pinned host memory
    numel: List[int] = field(init=False)

    def __post_init__(self):
        self.numel = numels(self.shapes)

    @property
    def K(self) -> int:
        return len(self.group_of)

    @property
    def G(self) -> int:
        return max(self.group_of) + 1

    @property
    def T(self) -> int:
        return len(self.shapes)

    @property
    def N(self) -> int:
        return sum(self.numel)

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "f32" else 2


def tiny() -> Workload:
    return Workload("tiny", 0, list(TINY_SHAPES), "f32", [0, 0, 1, 1], [64, 64, 32, 32])


def resnet18() -> Workload:
    return Workload("resnet18", 1, resnet18_shapes(10), "f32", [0, 0, 1, 1], None,
                    step_times=[1.0, 1.0, 1.6, 1.6], global_batch=256, staged=True)


def resnet50() -> Workload:
    return Workload("resnet50", 2, resnet50_shapes(1000), "bf16", [0] * 4 + [1] * 4,
                    [48] * 4 + [32] * 4)


def mobilenet_v2() -> Workload:
    return Workload("mobilenet_v2", 3, mobilenet_v2_shapes(1000), "f32", [0] * 4 + [1] * 2 + [2] * 2,
                    None, step_times=[1.0] * 4 + [1.4] * 2 + [2.1] * 2, global_batch=256)


def sweep_shares(K: int, total: int = 512) -> List[int]:
    """Integer shares for a sweep point: draw u_r uniformly in [16, 128], then scale
    to the requested total by floor + largest fractional part (ties: lower rank)."""
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 4000 + K))
    u = rng.integers(16, 129, size=K).astype(np.int64)
    s = int(u.sum())
    base = (u * total) // s
    rem = (u * total) % s
    order = sorted(range(K), key=lambda i: (-int(rem[i]), i))
    for i in order[: total - int(base.sum())]:
        base[i] += 1
    assert int(base.sum()) == total and int(base.min()) >= 1
    return [int(v) for v in base]


def sweep_point(K: int, bytes_per_rank: int, dtype: str) -> Workload:
    """Flat buffer per rank, ranks 0..K/2-1 in group 0 and the rest in group 1."""
    es = 4 if dtype == "f32" else 2
    n = bytes_per_rank // es
    return Workload("sweep_K%d_%dB_%s" % (K, bytes_per_rank, dtype), 4, [(n,)], dtype,
                    [0] * (K // 2) + [1] * (K - K // 2), sweep_shares(K),
                    bucket_cap_bytes=1 << 62)


def by_name(name: str) -> Workload:
    return {"tiny": tiny, "resnet18": resnet18, "resnet50": resnet50,
            "mobilenet_v2": mobilenet_v2}[name]()


# ----------------------------------------------------------------------------- values
def _seed(config_id: int, rank: int) -> int:
    return SEED_BASE + 1000 * config_id + rank


def rank_gradients(wl: Workload, rank: int, device: str = "cpu") -> torch.Tensor:
    """All N gradient values of one rank as one 1-D tensor, tensor after tensor in
    list order: i.i.d. N(0, SIGMA) in fp32, narrowed with torch's cast when the
    workload's dtype is bf16.  The generator lives on ``device``: CPU values are
    reproducible everywhere; device values only feed runs whose expected values are
    computed from a copy of the very same bytes."""
    gen = torch.Generator(device=device)
    gen.manual_seed(_seed(wl.config_id, rank))
    x = torch.randn(wl.N, generator=gen, device=device, dtype=torch.float32) * SIGMA
    if wl.dtype == "bf16":
        x = x.to(torch.bfloat16)
    return x


def split_tensors(flat: torch.Tensor, numel: Sequence[int]) -> List[torch.Tensor]:
    """Cut a rank's value vector into its per-parameter tensors.  Every tensor is a
    fresh allocation (as real per-parameter gradients are), not a view."""
    out, pos = [], 0
    for n in numel:
        out.append(flat[pos:pos + n].clone())
        pos += n
    return out


def as_numpy(t: torch.Tensor) -> np.ndarray:
    """Host copy of a tensor's bytes: float32 array, or uint16 bit patterns for bf16."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
