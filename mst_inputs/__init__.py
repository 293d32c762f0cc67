"""Seeded synthetic inputs for the masked fully-connected layer workloads.

This module only *draws* data: activations, weights, upstream gradients and
binary masks with the shapes of GPT-2 fully-connected layers.  It holds none
of the method's arithmetic (no products, no selection, no hashing used by the
topology update), so both the CPU checker and the CUDA library can be fed
from it without sharing any computation.

All arrays are numpy, generated on the host from ``numpy.random.PCG64``
streams keyed by an explicit seed; nothing here touches a GPU.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

BASE_SEED = 0x4D5354  # "MST"


# --------------------------------------------------------------------------
# bf16 helpers (storage format only: round-to-nearest-even, widen)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    rnd = ((u >> 16) & 1) + 0x7FFF
    return ((u + rnd) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 patterns (uint16) to float32 exactly."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed) & 0xFFFFFFFFFFFFFFFF, *[int(s) for s in stream]]))


def normal(shape: Tuple[int, ...], std: float, seed: int, *stream: int) -> np.ndarray:
    """float32 samples of N(0, std^2)."""
    g = _rng(seed, *stream)
    return (g.standard_normal(size=shape, dtype=np.float32) * np.float32(std)).astype(np.float32)


# --------------------------------------------------------------------------
# masks
# --------------------------------------------------------------------------
def uniform_mask(out_features: int, in_features: int, nnz: int, seed: int, *stream: int) -> np.ndarray:
    """Exactly ``nnz`` active entries: the head of a seeded permutation of all entries."""
    n = out_features * in_features
    if not 0 <= nnz <= n:
        raise ValueError("nnz out of range")
    g = _rng(seed, *stream, 0x6D61736B)
    m = np.zeros(n, dtype=np.uint8)
    if nnz == n:
        m[:] = 1
    elif nnz > 0:
        m[g.permutation(n)[:nnz]] = 1
    return m.reshape(out_features, in_features)


def zipf_row_counts(out_features: int, in_features: int, nnz: int, alpha: float, seed: int, *stream: int) -> np.ndarray:
    """Row populations proportional to rank^-alpha over a seeded row order.

    Each row is capped at ``in_features``; the excess of capped rows is
    re-spread over the remaining rows in proportion to their weights
    (water-filling), and the fractional counts are rounded by largest
    remainder so that the total is exactly ``nnz``.
    """
    n = out_features * in_features
    if not 0 <= nnz <= n:
        raise ValueError("nnz out of range")
    g = _rng(seed, *stream, 0x7A697066)
    order = g.permutation(out_features)            # order[rank] = row
    w = np.arange(1, out_features + 1, dtype=np.float64) ** (-float(alpha))
    share = np.zeros(out_features, dtype=np.float64)
    free = np.ones(out_features, dtype=bool)
    remaining = float(nnz)
    for _ in range(out_features + 1):
        if not free.any() or remaining <= 0:
            break
        s = w[free].sum()
        prop = np.zeros(out_features)
        prop[free] = w[free] / s * remaining
        over = free & (prop >= in_features)
        if not over.any():
            share[free] = prop[free]
            break
        share[over] = in_features
        remaining -= in_features * int(over.sum())
        free &= ~over
    base = np.minimum(np.floor(share).astype(np.int64), in_features)
    short = int(nnz - base.sum())
    if short > 0:
        frac = share - base
        frac[base >= in_features] = -1.0
        idx = np.argsort(-frac, kind="stable")[:short]
        base[idx] += 1
    counts = np.zeros(out_features, dtype=np.int64)
    counts[order] = base
    assert counts.sum() == nnz and counts.max(initial=0) <= in_features
    return counts


def zipf_mask(out_features: int, in_features: int, nnz: int, alpha: float, seed: int, *stream: int) -> np.ndarray:
    """Mask whose row populations follow :func:`zipf_row_counts`; columns uniform without replacement."""
    counts = zipf_row_counts(out_features, in_features, nnz, alpha, seed, *stream)
    g = _rng(seed, *stream, 0x636F6C73)
    m = np.zeros((out_features, in_features), dtype=np.uint8)
    for o in range(out_features):
        c = int(counts[o])
        if c == in_features:
            m[o, :] = 1
        elif c > 0:
            m[o, g.permutation(in_features)[:c]] = 1
    return m


# --------------------------------------------------------------------------
# layer problems
# --------------------------------------------------------------------------
@dataclass
class LayerProblem:
    """One masked linear layer with its activations and upstream gradient.

    ``X``, ``W``, ``dY`` are float32 arrays holding the *stored-precision*
    values: for ``dtype == 'bf16'`` every value is exactly representable in
    bfloat16 and ``*_bits`` hold the uint16 patterns.
    """
    name: str
    layer_id: int
    out_features: int
    in_features: int
    tokens: int
    dtype: str                      # 'f32' | 'bf16'
    mask: np.ndarray                # uint8 [O, I]
    W: np.ndarray                   # float32 [O, I] (dense; values off-mask are ignored by the layer)
    X: np.ndarray                   # float32 [T, I]
    dY: np.ndarray                  # float32 [T, O]
    W_bits: np.ndarray = field(default=None, repr=False)
    X_bits: np.ndarray = field(default=None, repr=False)
    dY_bits: np.ndarray = field(default=None, repr=False)

    @property
    def nnz(self) -> int:
        return int(self.mask.sum(dtype=np.int64))


def make_layer(name: str, layer_id: int, out_features: int, in_features: int, tokens: int, dtype: str,
               mask: np.ndarray, seed: int, w_std: float = 0.02, x_std: float = 1.0,
               dy_std: float = 1e-2) -> LayerProblem:
    X = normal((tokens, in_features), x_std, seed, layer_id, 1)
    W = normal((out_features, in_features), w_std, seed, layer_id, 2)
    dY = normal((tokens, out_features), dy_std, seed, layer_id, 3)
    p = LayerProblem(name, layer_id, out_features, in_features, tokens, dtype, mask, W, X, dY)
    if dtype == "bf16":
        p.W_bits, p.X_bits, p.dY_bits = f32_to_bf16_bits(W), f32_to_bf16_bits(X), f32_to_bf16_bits(dY)
        p.W, p.X, p.dY = bf16_bits_to_f32(p.W_bits), bf16_bits_to_f32(p.X_bits), bf16_bits_to_f32(p.dY_bits)
    elif dtype != "f32":
        raise ValueError("dtype must be 'f32' or 'bf16'")
    return p


def block_shapes(d_model: int) -> List[Tuple[str, int, int]]:
    """(name, out_features, in_features) of the four FC weights of a GPT-2 block."""
    return [("qkv", 3 * d_model, d_model), ("attn_proj", d_model, d_model),
            ("fc1", 4 * d_model, d_model), ("fc2", d_model, 4 * d_model)]


GPT2_WIDTH = {"small": 768, "medium": 1024, "large": 1280}
GPT2_BLOCKS = {"small": 12, "medium": 24, "large": 36}


def exact_nnz(out_features: int, in_features: int, density: float) -> int:
    """round(density * numel), halves rounded up (never hit by the listed configs)."""
    return int(np.floor(density * out_features * in_features + 0.5))


def uniform_layer(name: str, layer_id: int, out_features: int, in_features: int, tokens: int, dtype: str,
                  density: float, seed: int) -> LayerProblem:
    nnz = exact_nnz(out_features, in_features, density)
    m = uniform_mask(out_features, in_features, nnz, seed, layer_id)
    return make_layer(name, layer_id, out_features, in_features, tokens, dtype, m, seed)


def zipf_layer(name: str, layer_id: int, out_features: int, in_features: int, tokens: int, dtype: str,
               density: float, seed: int, alpha: float = 1.1) -> LayerProblem:
    nnz = exact_nnz(out_features, in_features, density)
    m = zipf_mask(out_features, in_features, nnz, alpha, seed, layer_id)
    return make_layer(name, layer_id, out_features, in_features, tokens, dtype, m, seed)


# The five workloads -------------------------------------------------------
def config1(tokens: int = 256) -> List[LayerProblem]:
    """Single fp32 layer 768 -> 3072 at density 0.25, 256 tokens."""
    return [uniform_layer("fc1", 0, 3072, 768, tokens, "f32", 0.25, BASE_SEED + 1)]


def config2(tokens: int = 8192, density: float = 0.25) -> List[LayerProblem]:
    """The four FC weights of one GPT-2-small block, bf16, uniform masks."""
    return [uniform_layer(n, i, o, k, tokens, "bf16", density, BASE_SEED + 2)
            for i, (n, o, k) in enumerate(block_shapes(768))]


def config3_density(layer_id: int, seed: int = BASE_SEED + 3) -> float:
    """Per-layer density in [0.03, 0.10] from a seeded uniform draw."""
    u = _rng(seed, layer_id, 0x64656E73).random()
    return 0.03 + 0.07 * float(u)


def config3(tokens: int = 8192, blocks: int = 12, first_block: int = 0) -> List[LayerProblem]:
    """Ultra-sparse phase, GPT-2-small shapes, Zipf(1.1) row populations."""
    out = []
    for b in range(first_block, first_block + blocks):
        for j, (n, o, k) in enumerate(block_shapes(768)):
            lid = 4 * b + j
            out.append(zipf_layer(f"b{b}.{n}", lid, o, k, tokens, "bf16", config3_density(lid), BASE_SEED + 3))
    return out


def config4(tokens: int = 16384, blocks: int = 24, first_block: int = 0, density: float = 0.1) -> List[LayerProblem]:
    """GPT-2-medium FC layers, bf16, uniform masks at density 0.1."""
    out = []
    for b in range(first_block, first_block + blocks):
        for j, (n, o, k) in enumerate(block_shapes(1024)):
            out.append(uniform_layer(f"b{b}.{n}", 4 * b + j, o, k, tokens, "bf16", density, BASE_SEED + 4))
    return out


CONFIG5_DENSITIES = (1.0, 0.5, 0.25, 0.1, 0.05, 0.02)


def config5(density: float, tokens: int = 16384) -> List[LayerProblem]:
    """One GPT-2-large block's four FC shapes at one point of the density sweep."""
    return [uniform_layer(n, i, o, k, tokens, "bf16", density, BASE_SEED + 5)
            for i, (n, o, k) in enumerate(block_shapes(1280))]


# --------------------------------------------------------------------------
# attention inputs
# --------------------------------------------------------------------------
@dataclass
class AttentionProblem:
    """Fused qkv activations of a GPT-2 attention layer: ``qkv`` is [batch * seq, 3 * heads * head_dim] (the output
    of the qkv projection: queries, keys, values side by side, heads contiguous inside each), stored-precision bf16
    values as float32 plus their bit patterns."""
    batch: int
    seq: int
    heads: int
    head_dim: int
    qkv: np.ndarray
    qkv_bits: np.ndarray

    def split(self):
        """(Q, K, V) as float32 [batch, heads, seq, head_dim] views of the stored values."""
        c = self.heads * self.head_dim
        x = self.qkv.reshape(self.batch, self.seq, 3, self.heads, self.head_dim)
        return tuple(np.ascontiguousarray(x[:, :, k].transpose(0, 2, 1, 3)) for k in range(3))


def attention_problem(batch: int, seq: int, heads: int = 12, head_dim: int = 64, seed: int = BASE_SEED + 7,
                      std: float = 1.0) -> AttentionProblem:
    """N(0, std^2) queries, keys and values (unit variance gives scaled scores of unit variance), rounded to bf16."""
    x = normal((batch * seq, 3 * heads * head_dim), std, seed, 0x617474)
    bits = f32_to_bf16_bits(x)
    return AttentionProblem(batch, seq, heads, head_dim, bf16_bits_to_f32(bits), bits)
