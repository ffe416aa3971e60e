"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path's tests and bench.

This module only *makes inputs*: random bf16 tensors of the shapes and value
distributions of BERT-family linear layers, random kept-column subsets, and the
workload tables.  It contains none of the method's arithmetic (no norms, no
penalties, no threshold decisions, no products) so that both sides of a parity
test can draw bit-identical inputs from it without sharing any of the code
under test.

bf16 tensors are carried as ``numpy.uint16`` bit patterns (numpy has no bf16
dtype); ``bf16_bits_to_f32`` gives the exact float value of each pattern.

Stand-in note: the paper fine-tunes and prunes BERT_BASE / RoBERTa_BASE /
DistilBERT on GLUE (Section 4.2).  Neither the checkpoints nor the datasets
are used here; only the layer shapes (hidden 768, FFN 3072, 12 or 6 layers, 6
weight matrices per layer), the compression rates of Tables 1 and 2 and the
default seed 42 (Section 5.4) are taken from it.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np

DEFAULT_SEED = 42  # the paper's default seed (Section 5.4)


# --------------------------------------------------------------------------
# random streams and bf16 encoding
# --------------------------------------------------------------------------
def stream(seed: int, *tags: int) -> np.random.Generator:
    """Independent counter-based (Philox) stream keyed by (seed, tags...)."""
    ss = np.random.SeedSequence([int(seed) & 0xFFFFFFFF, *[int(t) & 0xFFFFFFFF for t in tags]])
    return np.random.Generator(np.random.Philox(ss))


def tag_of(name: str) -> int:
    """Stable 32-bit tag of a tensor name (FNV-1a), so streams do not depend on call order."""
    h = 0x811C9DC5
    for ch in name.encode():
        h = ((h ^ ch) * 0x01000193) & 0xFFFFFFFF
    return h


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float values to bf16 (round-to-nearest-even) and return the bit patterns."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact float32 value of each bf16 bit pattern."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


_TINY_BITS = np.uint16(0x3000)  # 2**-31 as bf16: replaces an exact zero draw


def _nonzero(bits: np.ndarray) -> np.ndarray:
    """Make sure no generated weight is exactly +-0 (a zero must mean 'pruned')."""
    out = bits.copy()
    out[(out & 0x7FFF) == 0] = _TINY_BITS
    return out


def normal_bf16(seed: int, name: str, shape: Sequence[int], std: float) -> np.ndarray:
    g = stream(seed, tag_of(name))
    x = g.standard_normal(size=tuple(shape), dtype=np.float64) * std
    return _nonzero(f32_to_bf16_bits(x.astype(np.float32)))


def student_t_bf16(seed: int, name: str, shape: Sequence[int], nu: float, std: float) -> np.ndarray:
    """Heavy-tailed weights: Student-t(nu) rescaled to the given standard deviation (nu > 2)."""
    g = stream(seed, tag_of(name))
    x = g.standard_t(nu, size=tuple(shape)) * (std / np.sqrt(nu / (nu - 2.0)))
    return _nonzero(f32_to_bf16_bits(x.astype(np.float32)))


# --------------------------------------------------------------------------
# kept sets drawn by seed, and the pruned weight they imply
# --------------------------------------------------------------------------
def random_keep_sets(seed: int, name: str, n_blocks: int, n_groups: int, keep: int) -> np.ndarray:
    """bool [n_blocks, n_groups]: in every block a uniformly random subset of exactly `keep` groups."""
    g = stream(seed, tag_of(name), 0x6B656570)
    scores = g.random(size=(n_blocks, n_groups))
    order = np.argsort(scores, axis=1, kind="stable")
    keep_mask = np.zeros((n_blocks, n_groups), dtype=bool)
    np.put_along_axis(keep_mask, order[:, :keep], True, axis=1)
    return keep_mask


def zero_groups(w_bits: np.ndarray, keep: np.ndarray, block: int, orient: str) -> np.ndarray:
    """Copy of W (bf16 bits, [rows, cols]) with every group not in `keep` set to +0.

    orient "C": keep is [rows/block, cols], a group is `block` consecutive rows of one column.
    orient "R": keep is [rows, cols/block], a group is `block` consecutive columns of one row.
    """
    rows, cols = w_bits.shape
    if orient == "C":
        full = np.repeat(keep, block, axis=0)
    elif orient == "R":
        full = np.repeat(keep, block, axis=1)
    else:
        raise ValueError(orient)
    assert full.shape == (rows, cols)
    return np.where(full, w_bits, np.uint16(0)).astype(np.uint16)


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class LinearSpec:
    name: str
    n_out: int
    k_in: int
    gelu: bool
    rate: float        # target compression rate c (total / kept weights)
    block: int         # d: rows per row-block (orientation C)
    src: str = "x"     # which earlier tensor feeds it ("x" = the layer input)


@dataclass(frozen=True)
class Workload:
    name: str
    tokens: int
    linears: Tuple[LinearSpec, ...]
    weight_dist: str = "normal"   # "normal" or "student_t3"
    prune: str = "seeded_sets"    # "seeded_sets" (kept sets by seed, pack with t_b = 0) or "percentile"


def kept_per_block(k_in: int, rate: float) -> int:
    return int(round(k_in / rate))


def single_layer_small(block: int = 16) -> Workload:
    """One 768x768 linear at 128 tokens, 2.0x compression (batch 1, sequence 128)."""
    return Workload("single_linear_768_T128_c2", 128,
                    (LinearSpec("dense", 768, 768, False, 2.0, block),))


def bert_base_layer(tokens: int = 4096, rate: float = 3.0, block: int = 16,
                    hidden: int = 768, ffn: int = 3072, prefix: str = "L0") -> Workload:
    """The four linears of one encoder layer: fused QKV, attention output, FFN up (+GELU), FFN down.

    Attention itself, residuals and LayerNorm are not part of the path; the attention-output
    linear reads the V third of the QKV output, FFN-up reads the attention-output result and
    FFN-down reads FFN-up's (see `chain_source`).
    """
    return Workload(f"bert_layer_h{hidden}_T{tokens}_c{rate:g}_d{block}", tokens, (
        LinearSpec(f"{prefix}.qkv", 3 * hidden, hidden, False, rate, block, "x"),
        LinearSpec(f"{prefix}.attn_out", hidden, hidden, False, rate, block, "qkv_v"),
        LinearSpec(f"{prefix}.ffn_up", ffn, hidden, True, rate, block, "attn_out"),
        LinearSpec(f"{prefix}.ffn_down", hidden, ffn, False, rate, block, "ffn_up"),
    ))


def bert_base_stack_rates(seed: int, n_layers: int = 12, total_rate: float = 5.0,
                          hidden: int = 768, ffn: int = 3072) -> List[List[float]]:
    """Per-matrix rates c_i ~ U(3,7) for the 6 matrices (Q,K,V,O,up,down) of each layer, then all
    scaled by one factor so that sum(weights)/sum(weights/c_i) equals `total_rate`."""
    g = stream(seed, tag_of("stack_rates"))
    c = g.uniform(3.0, 7.0, size=(n_layers, 6))
    sizes = np.array([hidden * hidden] * 4 + [hidden * ffn] * 2, dtype=np.float64)
    total = sizes.sum() * n_layers
    kept = (sizes[None, :] / c).sum()
    c = c * (total_rate / (total / kept))
    return c.tolist()


def distil_stack(tokens: int = 8192, n_layers: int = 6, rate: float = 1.79, block: int = 32,
                 hidden: int = 768, ffn: int = 3072) -> Workload:
    """DistilBERT-shaped stack with heavy-tailed weights pruned by a per-matrix percentile threshold."""
    lin: List[LinearSpec] = []
    for l in range(n_layers):
        p = f"L{l}"
        lin += [
            LinearSpec(f"{p}.qkv", 3 * hidden, hidden, False, rate, block, "x" if l == 0 else f"L{l-1}.ffn_down"),
            LinearSpec(f"{p}.attn_out", hidden, hidden, False, rate, block, "qkv_v"),
            LinearSpec(f"{p}.ffn_up", ffn, hidden, True, rate, block, "attn_out"),
            LinearSpec(f"{p}.ffn_down", hidden, ffn, False, rate, block, "ffn_up"),
        ]
    return Workload(f"distil_stack_T{tokens}_c{rate:g}_d{block}", tokens, tuple(lin),
                    weight_dist="student_t3", prune="percentile")


def make_weight(seed: int, spec: LinearSpec, dist: str = "normal") -> np.ndarray:
    """Unpruned bf16 weight [n_out, k_in] (the nn.Linear orientation), std 0.02."""
    if dist == "normal":
        return normal_bf16(seed, spec.name + ".W", (spec.n_out, spec.k_in), 0.02)
    if dist == "student_t3":
        return student_t_bf16(seed, spec.name + ".W", (spec.n_out, spec.k_in), 3.0, 0.02)
    raise ValueError(dist)


def make_bias(seed: int, spec: LinearSpec) -> np.ndarray:
    return normal_bf16(seed, spec.name + ".b", (spec.n_out,), 0.02)


def make_activations(seed: int, name: str, tokens: int, k_in: int) -> np.ndarray:
    return normal_bf16(seed, name + ".X", (tokens, k_in), 1.0)


def make_pruned_weight(seed: int, spec: LinearSpec, dist: str = "normal",
                       orient: str = "C") -> Tuple[np.ndarray, np.ndarray]:
    """(W with the non-kept groups zeroed, keep sets) for the 'kept sets drawn by seed' recipe."""
    w = make_weight(seed, spec, dist)
    if orient == "C":
        n_blocks, n_groups = spec.n_out // spec.block, spec.k_in
    else:
        n_blocks, n_groups = spec.k_in // spec.block, spec.n_out
    keep = random_keep_sets(seed, spec.name + ".keep", n_blocks, n_groups,
                            kept_per_block(n_groups, spec.rate))
    if orient == "R":
        keep = np.ascontiguousarray(keep.T)      # [rows, cols/block]
    return zero_groups(w, keep, spec.block, orient), keep
