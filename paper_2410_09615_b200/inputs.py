"""Seeded synthetic inputs for the compressed linear layer.

Host-side numpy only.  This module holds the *recipe* for the workloads (shapes,
value distributions, seeds) and the bfloat16 bit conversions needed to state
them; it contains none of the arithmetic of packing or of the layer forward, and
it is the only module shared by the GPU tests, the CPU oracle tests and the
benchmark.

Recipe (one layer):
  W  ~ N(0, 0.02^2) fp32 [d_out, d_in]        zero-centred bell-shaped weights
  s  = max|W| / 7 (fp32)                       AbsMax scale, one per tensor
  codes = clamp(rint(W / s), -8, 7) int8       symmetric uniform 4-bit grid
  mask  = the two largest |W| of every aligned group of four along d_in
          (ties: lower index wins)             NVIDIA 2:4 pattern
  L ~ N(0, 0.02^2) [d_out, r],  R ~ N(0, 0.02^2) [r, d_in],  X ~ N(0, 1) [b, d_in],
  each rounded to bfloat16 (round to nearest even) and carried as uint16 bits.
Streams: numpy PCG64 seeded with [seed, 1] (weights), [seed, 2] (adapters),
[seed, 3] (activations), [seed, 4] (row samples).
"""
from __future__ import annotations

from dataclasses import dataclass
import numpy as np


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); return the uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    out = rounded.astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = 0x7FC0
    return out


def bf16_bits_to_f64(h: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    h = np.ascontiguousarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def default_rank(d_in: int, d_out: int) -> int:
    """Rank = 10 % of the smaller dimension, rounded up to a multiple of 16."""
    return round_up(int(np.ceil(0.1 * min(d_in, d_out) - 1e-9)), 16)


def rank_for_ratio(ratio: float, d_in: int, d_out: int) -> int:
    if ratio <= 0:
        return 0
    return round_up(int(np.ceil(ratio * min(d_in, d_out) - 1e-9)), 16)


@dataclass
class Layer:
    """One compressed linear layer plus one activation batch (all host arrays)."""
    d_in: int
    d_out: int
    r: int
    b: int
    seed: int
    s: float                 # fp32 scale (python float holding an fp32 value)
    codes: np.ndarray        # int8  [d_out, d_in]
    mask: np.ndarray         # uint8 [d_out, d_in]
    L: np.ndarray | None     # uint16 (bf16 bits) [d_out, r]
    R: np.ndarray | None     # uint16 (bf16 bits) [r, d_in]
    X: np.ndarray            # uint16 (bf16 bits) [b, d_in]


def top2_mask(W: np.ndarray) -> np.ndarray:
    """2:4 magnitude mask along the last axis; ties resolved to the lower index.
    An element is kept when fewer than two others of its group beat it, where
    "beats" means larger magnitude, or equal magnitude at a lower index."""
    d_out, d_in = W.shape
    a = np.abs(W).reshape(d_out, d_in // 4, 4)
    mask = np.empty(a.shape, dtype=np.uint8)
    for i in range(4):
        beaten = np.zeros(a.shape[:2], dtype=np.uint8)
        for j in range(4):
            if j < i:
                beaten += a[..., j] >= a[..., i]
            elif j > i:
                beaten += a[..., j] > a[..., i]
        mask[..., i] = beaten < 2
    return mask.reshape(d_out, d_in)


def make_weights(d_out: int, d_in: int, seed: int):
    """(s, codes, mask) of one layer; row blocks are generated one after another
    from a single stream so that large layers do not need several full-size
    temporaries."""
    rng = np.random.default_rng([int(seed), 1])
    W = np.empty((d_out, d_in), np.float32)
    step = max(1, (1 << 24) // d_in)
    for r0 in range(0, d_out, step):
        blk = W[r0:r0 + step]
        rng.standard_normal(blk.shape, dtype=np.float32, out=blk)
    W *= np.float32(0.02)
    s = np.float32(np.max(np.abs(W))) / np.float32(7.0)
    codes = np.empty((d_out, d_in), np.int8)
    mask = np.empty((d_out, d_in), np.uint8)
    for r0 in range(0, d_out, step):
        blk = W[r0:r0 + step]
        codes[r0:r0 + step] = np.clip(np.rint(blk / s), -8, 7).astype(np.int8)
        mask[r0:r0 + step] = top2_mask(blk)
    return float(s), codes, mask


def make_adapters(d_out: int, d_in: int, r: int, seed: int):
    if r <= 0:
        return None, None
    rng = np.random.default_rng([int(seed), 2])
    L = f32_to_bf16_bits(rng.standard_normal((d_out, r), dtype=np.float32) * np.float32(0.02))
    R = f32_to_bf16_bits(rng.standard_normal((r, d_in), dtype=np.float32) * np.float32(0.02))
    return L, R


def make_activations(b: int, d_in: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng([int(seed), 3])
    return f32_to_bf16_bits(rng.standard_normal((b, d_in), dtype=np.float32))


def make_layer(d_in: int, d_out: int, r: int, b: int, seed: int, weights=None) -> Layer:
    """All host arrays of one case.  ``weights`` = a cached (s, codes, mask) triple
    to reuse across cases that share a weight; otherwise generated from ``seed``."""
    s, codes, mask = weights if weights is not None else make_weights(d_out, d_in, seed)
    L, R = make_adapters(d_out, d_in, r, seed)
    X = make_activations(b, d_in, seed)
    return Layer(d_in, d_out, r, b, seed, s, codes, mask, L, R, X)


# ---------------------------------------------------------------------------
# Workload table: (d_in, d_out) of the LLaMA-2 linear layers, by model size.
# "count" is how many linears of that shape one transformer block has
# (q, k, v, o / gate, up / down; the 70B model uses grouped-query k, v).
# ---------------------------------------------------------------------------
LLAMA2_SHAPES = {
    "7b": [("attn_qkvo", 4096, 4096, 4), ("mlp_gate_up", 4096, 11008, 2), ("mlp_down", 11008, 4096, 1)],
    "13b": [("attn_qkvo", 5120, 5120, 4), ("mlp_gate_up", 5120, 13824, 2), ("mlp_down", 13824, 5120, 1)],
    "70b": [("attn_qo", 8192, 8192, 2), ("attn_kv", 8192, 1024, 2),
            ("mlp_gate_up", 8192, 28672, 2), ("mlp_down", 28672, 8192, 1)],
}

# Workload configurations: index -> (model key or None, batch sizes, rank ratios)
CONFIGS = {
    0: dict(name="single_512", shapes=[("single", 512, 512, 1)], batches=[8], ranks="fixed64"),
    1: dict(name="llama2_7b_decode", shapes=LLAMA2_SHAPES["7b"], batches=[1, 16], ranks=[0.1]),
    2: dict(name="llama2_7b_prefill", shapes=LLAMA2_SHAPES["7b"], batches=[2048], ranks=[0.1]),
    3: dict(name="llama2_13b", shapes=LLAMA2_SHAPES["13b"], batches=[1, 16, 2048], ranks=[0.1]),
    4: dict(name="llama2_70b", shapes=LLAMA2_SHAPES["70b"], batches=[1, 16, 4096],
            ranks=[0.0, 0.05, 0.1, 0.2]),
}


def config_cases(cfg: int):
    """Yield (layer_name, d_in, d_out, r, b, seed, weight_seed) for every case of a
    configuration.  Cases that differ only in batch size or rank share the
    layer's weight (``weight_seed``); adapters and activations use ``seed``."""
    c = CONFIGS[cfg]
    for li, (name, d_in, d_out, _count) in enumerate(c["shapes"]):
        wseed = 1000 * cfg + 10 * li
        for bi, b in enumerate(c["batches"]):
            if c["ranks"] == "fixed64":
                yield name, d_in, d_out, 64, b, 0, 0
                continue
            for ri, ratio in enumerate(c["ranks"]):
                r = rank_for_ratio(ratio, d_in, d_out)
                yield name, d_in, d_out, r, b, wseed + bi + 100 * ri, wseed


def sample_rows(b: int, tile: int = 128, seed: int = 0, dense_edges: bool = True) -> np.ndarray:
    """Token rows on which a large-batch output is compared one by one: the
    first and the last ``tile`` rows (all of them, or their first / middle / last
    row when ``dense_edges`` is False) plus one seeded row in every other tile."""
    if b <= 2 * tile and dense_edges:
        return np.arange(b, dtype=np.int32)
    rng = np.random.default_rng([int(seed), 4])
    if dense_edges:
        rows = list(range(tile)) + list(range(b - tile, b))
    else:
        e = min(tile, b)
        rows = [0, e // 2, e - 1, b - e, b - 1 - e // 2, b - 1]
    for t in range(1, (b - 1) // tile):
        lo, hi = t * tile, min((t + 1) * tile, b - tile)
        if hi > lo:
            rows.append(int(rng.integers(lo, hi)))
    rows = [x for x in rows if 0 <= x < b]
    return np.array(sorted(set(rows)), dtype=np.int32)
