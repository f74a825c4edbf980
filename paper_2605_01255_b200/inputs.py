"""Seeded synthetic inputs and workload shapes.  Holds none of the method's arithmetic.

Both the CUDA tests/bench and the CPU oracle tests draw their X, W, G from here so that they see
identical values.  All generators are numpy (host) and deterministic in (seed, shape).

Recipes (they stand in for the activations, gradients and weights of the paper's LLaMA/Qwen
fine-tuning runs, which need datasets and checkpoints that are not available):
  * "gaussian": X, G ~ N(0, 1), W ~ N(0, 0.02^2).
  * "heavy_lowrank": X = D Z diag(sigma) Q^T with Z iid N(0,1), sigma_i = 1/i, Q a product of four
    seeded Householder reflections (orthogonal, so the spectrum i^-1 is kept exactly), D a diagonal
    of |Student-t(nu=3)| draws, one per token row; rescaled to unit RMS.
Values are rounded to the I/O dtype (bf16 by round-to-nearest-even) before anyone uses them.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np


# --------------------------------------------------------------------------- dtype helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """binary32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    b = b + (np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))
    return (b >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> binary32 values."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """The values of x after storage in `dtype` ("f32" or "bf16"), as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f32":
        return x
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(x))
    raise ValueError(dtype)


# --------------------------------------------------------------------------- generators
def _gen(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(int(seed)))


def gaussian(shape: Tuple[int, ...], seed: int, std: float = 1.0, dtype: str = "f32") -> np.ndarray:
    x = _gen(seed).standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return round_to_dtype(x, dtype)


def orthonormal_rows(r: int, d: int, seed: int, dtype: str = "f32") -> np.ndarray:
    """r orthonormal rows of length d (the Q factor of a seeded Gaussian matrix), rounded to `dtype`:
    a stand-in for the basis V^T that a subspace method hands to the explicit-factor calls."""
    q, _ = np.linalg.qr(_gen(seed).standard_normal((d, r)))
    return round_to_dtype(np.ascontiguousarray(q.T).astype(np.float32), dtype)


def heavy_lowrank(m: int, d: int, seed: int, dtype: str = "bf16") -> np.ndarray:
    g = _gen(seed)
    x = g.standard_normal((m, d), dtype=np.float32)
    x *= (1.0 / np.arange(1, d + 1, dtype=np.float32))[None, :]
    for _ in range(4):  # x <- x (I - 2 v v^T), v unit
        v = g.standard_normal(d).astype(np.float32)
        v /= np.linalg.norm(v)
        x -= 2.0 * (x @ v)[:, None] * v[None, :]
    x *= np.abs(g.standard_t(3.0, size=m)).astype(np.float32)[:, None]
    x /= np.sqrt(np.mean(x.astype(np.float64) ** 2)).astype(np.float32)
    return round_to_dtype(x, dtype)


# --------------------------------------------------------------------------- workloads
@dataclass(frozen=True)
class Linear:
    name: str
    d_in: int
    d_out: int
    slot: int  # which distinct layer input it reads (q, k, v share slot 0; gate, up share slot 2)


@dataclass(frozen=True)
class Workload:
    name: str
    tokens: int
    linears: Tuple[Linear, ...]
    r: int
    dtype: str
    recipe: str = "gaussian"
    layers: int = 1


def _decoder(hidden: int, inter: int) -> Tuple[Linear, ...]:
    return (Linear("q", hidden, hidden, 0), Linear("k", hidden, hidden, 0), Linear("v", hidden, hidden, 0),
            Linear("o", hidden, hidden, 1), Linear("gate", hidden, inter, 2), Linear("up", hidden, inter, 2),
            Linear("down", inter, hidden, 3))


def workload(name: str, r: int | None = None) -> Workload:
    """The five configurations; `r` overrides the rank where a configuration sweeps it."""
    if name == "single_fp32":
        return Workload(name, 512, (Linear("linear", 256, 256, 0),), r or 16, "f32")
    if name == "qwen0.5b_mlp":
        return Workload(name, 4096, (Linear("gate", 896, 4864, 0), Linear("up", 896, 4864, 0),
                                     Linear("down", 4864, 896, 1)), r or 64, "bf16")
    if name == "llama1b_layer":
        return Workload(name, 16384, _decoder(2048, 8192), r or 128, "bf16")
    if name == "llama3b_layer":
        return Workload(name, 16384, _decoder(3072, 8192), r or 128, "bf16")
    if name == "llama3b_gqa_layer":  # the real LLaMA-3.2-3B widths: grouped-query k and v project to 1024
        lins = list(_decoder(3072, 8192))
        lins[1], lins[2] = Linear("k", 3072, 1024, 0), Linear("v", 3072, 1024, 0)
        return Workload(name, 16384, tuple(lins), r or 128, "bf16")
    if name == "llama3b_fused_layer":  # the same layer with the weights of linears on one input stacked: one launch each
        return Workload(name, 16384, (Linear("qkv", 3072, 3 * 3072, 0), Linear("o", 3072, 3072, 1),
                                      Linear("gate_up", 3072, 2 * 8192, 2), Linear("down", 8192, 3072, 3)), r or 128, "bf16")
    if name == "llama3b_stack28":
        return Workload(name, 16384, _decoder(3072, 8192), r or 128, "bf16", "heavy_lowrank", 28)
    raise KeyError(name)


WORKLOADS: List[str] = ["single_fp32", "qwen0.5b_mlp", "llama1b_layer", "llama3b_layer", "llama3b_stack28", "llama3b_gqa_layer",
                        "llama3b_fused_layer"]

# data seeds: X of slot s in layer l, G and W of linear k in layer l
def seed_x(layer: int, slot: int) -> int:
    return 1_000 + 16 * layer + slot


def seed_g(layer: int, k: int) -> int:
    return 2_000 + 16 * layer + k


def seed_w(layer: int, k: int) -> int:
    return 3_000 + 16 * layer + k


SKETCH_STEP_STRIDE = 1 << 20   # seeds of consecutive training steps are this far apart (16 * layers stays far below it)


def sketch_seed(base: int, layer: int, slot: int, step: int = 0) -> int:
    """One sketch per distinct layer input: linears that share an input share S and XS.  `step` gives every
    training step its own sketches (the compression randomness must be fresh per step for the gradient estimate to
    be unbiased over the run); callers that keep optimizer moments in the factor space keep step = 0 instead."""
    return int(base) + 16 * layer + slot + SKETCH_STEP_STRIDE * int(step)


def make_x(wl: Workload, layer: int, lin: Linear, tokens: int | None = None) -> np.ndarray:
    m = tokens or wl.tokens
    if wl.recipe == "heavy_lowrank":
        return heavy_lowrank(m, lin.d_in, seed_x(layer, lin.slot), wl.dtype)
    return gaussian((m, lin.d_in), seed_x(layer, lin.slot), 1.0, wl.dtype)


def make_g(wl: Workload, layer: int, k: int, tokens: int | None = None) -> np.ndarray:
    return gaussian((tokens or wl.tokens, wl.linears[k].d_out), seed_g(layer, k), 1.0, wl.dtype)


def make_w(wl: Workload, layer: int, k: int) -> np.ndarray:
    lin = wl.linears[k]
    return gaussian((lin.d_out, lin.d_in), seed_w(layer, k), 0.02, wl.dtype)
