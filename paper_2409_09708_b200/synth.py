"""Seeded synthetic inputs and workload tables.

This module holds none of the method's arithmetic: it only draws random
tensors and lists layer shapes.  It serves both the CUDA library's callers and
the CPU oracle's callers, so that both sides see the same bytes; it imports
neither of them.

The tensors stand in for ImageNet-1k activations and trained DeiT / Swin
weights (Sec. 4 of the paper), which are not available: activations are
N(0, 1), weights and biases N(0, 0.02), drawn in fp32 and rounded to the
16-bit storage type.  Layer shapes are the real ones of DeiT-B and Swin-B; a
"layer" is one of the four linear modules of a transformer block (qkv, proj,
fc1, fc2 -- Sec. 3, L = 4B).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

X_STD = 1.0
W_STD = 0.02
B_STD = 0.02


@dataclass(frozen=True)
class Layer:
    """One linear module under sparsity level N:M, with the seeds of its tensors."""
    name: str
    rows: int      # token rows R
    in_: int       # input (reduction) dimension K
    out: int       # output features O
    N: int
    M: int
    seed_x: int
    seed_w: int
    seed_b: int

    @property
    def dense_equiv_flops(self) -> float:
        return 2.0 * self.rows * self.in_ * self.out

    @property
    def kept_flops(self) -> float:
        return self.dense_equiv_flops * self.N / self.M


def torch_dtype(name: str) -> torch.dtype:
    return {"f16": torch.float16, "bf16": torch.bfloat16}[name]


def randn(shape, seed: int, std: float, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """N(0, std) tensor: fp32 draw from a generator seeded with ``seed``, one rounding to dtype.

    CPU and CUDA generators give different streams for the same seed; callers
    draw on one device and copy the bytes to the other side.
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    t = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if std != 1.0:
        t.mul_(std)
    return t.to(dtype)


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw uint16 bit patterns of a 16-bit float tensor, as a host numpy array."""
    assert t.dtype in (torch.float16, torch.bfloat16)
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(dtype)


def layer_tensors(layer: Layer, dtype: torch.dtype, device="cpu", with_x=True):
    """(X or None, W, bias) of a layer, drawn on ``device``."""
    X = randn((layer.rows, layer.in_), layer.seed_x, X_STD, dtype, device) if with_x else None
    W = randn((layer.out, layer.in_), layer.seed_w, W_STD, dtype, device)
    b = randn((layer.out,), layer.seed_b, B_STD, dtype, device)
    return X, W, b


def _seeds(config: int, index: int):
    base = 1000 * config + 10 * index
    return base, base + 1, base + 2


def _block(dim: int, mlp: int):
    return [("qkv", dim, 3 * dim), ("proj", dim, dim), ("fc1", dim, mlp), ("fc2", mlp, dim)]


def single_layer() -> list[Layer]:
    """One 768x768 layer at 4:8 on 197 tokens, fp16, seed 0."""
    return [Layer("proj", 197, 768, 768, 4, 8, 0, 1, 2)]


def deit_b_block(batch: int = 64) -> list[Layer]:
    """The four linears of one DeiT-B block: qkv 4:8, proj 2:8, fc1 2:8, fc2 1:8."""
    levels = [(4, 8), (2, 8), (2, 8), (1, 8)]
    layers = []
    for i, ((name, k, o), (n, m)) in enumerate(zip(_block(768, 3072), levels)):
        layers.append(Layer(name, batch * 197, k, o, n, m, *_seeds(2, i)))
    return layers


def deit_b_stack(batch: int = 256) -> list[Layer]:
    """All 48 linears of DeiT-B, level per layer drawn uniformly from {1:8, 2:8, 4:8, 8:8}."""
    choices = [(1, 8), (2, 8), (4, 8), (8, 8)]
    draw = np.random.default_rng(3).integers(0, len(choices), 48)
    layers = []
    for blk in range(12):
        for j, (name, k, o) in enumerate(_block(768, 3072)):
            i = 4 * blk + j
            n, m = choices[int(draw[i])]
            layers.append(Layer("blk%d.%s" % (blk, name), batch * 197, k, o, n, m, *_seeds(3, i)))
    return layers


SWIN_B_DIMS = (128, 256, 512, 1024)
SWIN_B_DEPTHS = (2, 2, 18, 2)
SWIN_B_TOKENS = (3136, 784, 196, 49)


def swin_b_stack(batch: int = 128) -> list[Layer]:
    """All 96 linears of Swin-B, level per layer drawn from {1:4, 2:4, 1:8, 2:8, 4:8}."""
    choices = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8)]
    draw = np.random.default_rng(4).integers(0, len(choices), 96)
    layers = []
    i = 0
    for stage, (dim, depth, tokens) in enumerate(zip(SWIN_B_DIMS, SWIN_B_DEPTHS, SWIN_B_TOKENS)):
        for blk in range(depth):
            for name, k, o in _block(dim, 4 * dim):
                n, m = choices[int(draw[i])]
                layers.append(Layer("s%d.b%d.%s" % (stage, blk, name), batch * tokens, k, o, n, m,
                                    *_seeds(4, i)))
                i += 1
    return layers


SWEEP_ROWS = (4096, 16384, 65536)
SWEEP_SHAPES = ((768, 768), (768, 3072), (3072, 768), (1024, 4096), (4096, 1024))
SWEEP_LEVELS = ((1, 4), (2, 4), (1, 8), (2, 8), (4, 8), (1, 16), (2, 16), (4, 16), (8, 16))


def sweep() -> list[Layer]:
    """Shape / sparsity sweep: rows x (K, O) x level (each run in fp16 and bf16 by the caller)."""
    layers = []
    i = 0
    for rows in SWEEP_ROWS:
        for k, o in SWEEP_SHAPES:
            for n, m in SWEEP_LEVELS:
                layers.append(Layer("r%d.k%d.o%d.%d:%d" % (rows, k, o, n, m), rows, k, o, n, m,
                                    50000 + 10 * i, 50001 + 10 * i, 50002 + 10 * i))
                i += 1
    return layers


WORKLOADS = {
    "single_layer": (single_layer, "f16"),
    "deit_b_block_b64": (deit_b_block, "f16"),
    "deit_b_stack_b256": (deit_b_stack, "bf16"),
    "swin_b_stack_b128": (swin_b_stack, "bf16"),
}


def workload(name: str):
    """(layers, dtype name) of a named workload."""
    fn, dt = WORKLOADS[name]
    return fn(), dt


def sample_rows(rows: int, count: int, seed: int, tile: int = 128) -> np.ndarray:
    """Sorted row indices for spot checks: the first and last row of the first, a middle
    and the last row tile are always included, the rest are drawn uniformly."""
    forced = {0, min(tile - 1, rows - 1), rows - 1, (rows - 1) // tile * tile}
    mid = (rows // tile // 2) * tile
    forced |= {mid, min(mid + tile - 1, rows - 1)}
    rng = np.random.default_rng(seed)
    extra = rng.choice(rows, size=min(rows, max(count - len(forced), 0)), replace=False)
    picked = sorted(forced | set(int(v) for v in extra))
    return np.asarray(picked, dtype=np.int64)
