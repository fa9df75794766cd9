"""Seeded synthetic inputs for the five benchmark configurations.

This module holds no arithmetic of the method: it only draws tensors with the
shapes, dtypes and value distributions of the workloads (a transformer FFN
activation, a large LLM FFN activation with outliers, a CNN feature map, a
size sweep).  Both the CUDA path and the CPU oracle consume the tensors it
returns, so the two are always compared on identical inputs.

Draw order for one case (one ``torch.Generator`` seeded with ``seed``):
``x`` body (standard normal, fp32), then -- only when the case has outliers --
the Bernoulli mask (uniform < p) and the outlier values, then ``grad_out``.
Values are scaled in fp32 and cast once to the case dtype.
"""
from __future__ import annotations

import dataclasses
from typing import Iterator, Sequence, Tuple

import torch

ACTIVATIONS = ("gelu", "silu", "sigmoid", "tanh", "elu", "softplus", "leaky_relu")   # the sweep of config 5
EXTRA_ACTIVATIONS = ("relu", "selu")                                                 # rows of Table 1 beyond it


@dataclasses.dataclass(frozen=True)
class Case:
    name: str
    acts: Tuple[str, ...]
    bits: Tuple[int, ...]
    dtype: str                    # "f32" | "bf16" | "f16"
    shape: Tuple[int, ...]
    x_std: float
    g_std: float
    seed: int
    outlier_p: float = 0.0
    outlier_std: float = 0.0

    @property
    def n(self) -> int:
        n = 1
        for d in self.shape:
            n *= d
        return n

    @property
    def torch_dtype(self) -> torch.dtype:
        return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[self.dtype]


C1 = Case("c1_gelu3_f32_1m", ("gelu",), (3,), "f32", (1048576,), 1.0, 1.0, 0)
C2 = Case("c2_silu_bf16_roberta_ffn", ("silu",), (1, 2, 4), "bf16", (32, 128, 3072), 1.5, 1e-2, 1)
C3 = Case("c3_gelu_bf16_llm_ffn", ("gelu",), (1, 2, 3, 4), "bf16", (8, 2048, 16384), 1.0, 1.0, 2,
          outlier_p=0.01, outlier_std=10.0)
C4 = Case("c4_cnn_f32_nchw", ("sigmoid", "tanh", "elu"), (2,), "f32", (64, 256, 56, 56), 1.0, 1.0, 3)

SWEEP_SIZES = (2 ** 16, 2 ** 20, 2 ** 24, 2 ** 28, 2 ** 24 + 7)


def sweep_cases(sizes: Sequence[int] = SWEEP_SIZES) -> Iterator[Case]:
    """Config 5: every activation x bits 1..4 x size, in bf16 and fp32, seed 4."""
    for n in sizes:
        for dtype in ("bf16", "f32"):
            yield Case(f"c5_sweep_{dtype}_{n}", ACTIVATIONS, (1, 2, 3, 4), dtype, (n,), 2.0, 1.0, 4)


CONFIGS = {"c1": C1, "c2": C2, "c3": C3, "c4": C4}


def draw(case: Case, device: str | torch.device = "cpu", n: int | None = None):
    """Returns (x, grad_out) for ``case`` as flat tensors of the case dtype.

    ``n`` overrides the element count (used to draw a bounded sample with the
    same distribution)."""
    device = torch.device(device)
    n = case.n if n is None else int(n)
    gen = torch.Generator(device=device)
    gen.manual_seed(case.seed)
    x = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
    x.mul_(case.x_std)
    if case.outlier_p > 0.0:
        mask = torch.rand(n, generator=gen, device=device, dtype=torch.float32) < case.outlier_p
        out = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
        out.mul_(case.outlier_std)
        x = torch.where(mask, out, x)
        del mask, out
    g = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
    g.mul_(case.g_std)
    return x.to(case.torch_dtype), g.to(case.torch_dtype)


def to_numpy_bits(t: torch.Tensor):
    """Host view for the oracle: float32 array, or uint16 bfloat16 bit patterns."""
    import numpy as np

    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    if t.dtype in (torch.float32, torch.float16):
        return t.numpy()
    if t.dtype in (torch.int32, torch.uint8):
        return t.numpy()
    raise TypeError(t.dtype)


def shard_range(n: int, rank: int, world: int, align: int = 128) -> Tuple[int, int]:
    """Contiguous element range [lo, hi) of ``rank`` when a flat tensor of ``n``
    elements is split over ``world`` independent workers.  Every interior cut
    is a multiple of ``align`` elements, so each shard's packed words are whole
    (and 16-byte aligned for every bit width) and the concatenation of the
    shards' outputs is the single-worker bit stream."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    units = (n + align - 1) // align
    lo_u = (units * rank) // world
    hi_u = (units * (rank + 1)) // world
    return min(lo_u * align, n), min(hi_u * align, n)
