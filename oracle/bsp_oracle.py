"""CPU oracle for block-structured pruning and the linear layer it speeds up.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the CUDA
library is checked against.  It is written from the paper (Li, Kong et al.,
"Efficient Transformer-based Large Scale Language Representations using
Hardware-friendly Block Structured Pruning", EMNLP-Findings 2020) and shares no
code with the CUDA path; the library never imports or calls it.  Only tests,
the smoke check and the benchmark's CPU-baseline leg use it.

Everything is numpy in float64 on the exact values of the bf16 inputs, except
the *keep decision*, which the method takes on a float32 quantity that is
defined exactly below (`decision_sumsq32`) so that a float32 device and this
oracle decide identically.

Conventions
-----------
W is one linear layer's weight, [rows = N_out, cols = K_in], given as bf16 bit
patterns (uint16).  Two group geometries:

* orientation "C" (Eq. 3, column pruning inside a block): W is cut into
  rows/d row-blocks of d consecutive rows; a group is one column of one
  row-block, W[beta*d:(beta+1)*d, j].  Per-group arrays have shape
  [rows/d, cols].
* orientation "R" (Algorithm 1 as printed, and Eq. 2, row pruning inside a
  block): W is cut into cols/h vertical strips of h consecutive columns; a
  group is one row of one strip, W[i, alpha*h:(alpha+1)*h].  Per-group arrays
  have shape [rows, cols/h].

Every function names the passage of the paper it follows.  Parity pins for
each function live in tests/test_oracle_*.py; none is unpinned.
"""
from __future__ import annotations

import math
from fractions import Fraction
from typing import Optional, Tuple

import numpy as np

try:  # a library erf (vectorised); pinned against math.erf in the tests
    from scipy.special import erf as _erf_vec
except Exception:  # pragma: no cover - scipy is part of the image
    _erf_vec = np.vectorize(math.erf, otypes=[np.float64])


# ---------------------------------------------------------------------------
# input decoding
# ---------------------------------------------------------------------------
def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of each bf16 bit pattern, as float64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _grouped(a: np.ndarray, block: int, orient: str) -> np.ndarray:
    """View of a [rows, cols] array with the group's elements on the last axis.

    "C": [rows/d, cols, d]   "R": [rows, cols/h, h]
    """
    rows, cols = a.shape
    if orient == "C":
        if block < 1 or rows % block:
            raise ValueError("block height must divide the number of rows")
        return a.reshape(rows // block, block, cols).transpose(0, 2, 1)
    if orient == "R":
        if block < 1 or cols % block:
            raise ValueError("block width must divide the number of columns")
        return a.reshape(rows, cols // block, block)
    raise ValueError(f"orientation must be 'C' or 'R', got {orient!r}")


# ---------------------------------------------------------------------------
# group norms, gamma, penalty  (Section 3.2)
# ---------------------------------------------------------------------------
def group_sumsq_values(w: np.ndarray, block: int, orient: str) -> np.ndarray:
    """S_g for a matrix given as float64 values (used for bf16 inputs and by the gradient pins)."""
    g = _grouped(np.asarray(w, dtype=np.float64), block, orient)
    return (g * g).sum(axis=-1)


def group_sumsq(w_bits: np.ndarray, block: int, orient: str) -> np.ndarray:
    """S_g = sum of squares of the group's weights (the quantity under the root in Eq. 2 / Eq. 3)."""
    return group_sumsq_values(bf16_to_f64(w_bits), block, orient)


def group_norms(w_bits: np.ndarray, block: int, orient: str) -> np.ndarray:
    """l2 norm of every group: the square root in Eq. 2 / Eq. 3, the `l2_norms(i,j)` of Algorithm 1."""
    return np.sqrt(group_sumsq(w_bits, block, orient))


def gamma_update(norms: np.ndarray, eps: float) -> np.ndarray:
    """Penalty weights gamma = 1 / (||W_g||_2 + eps)  (the update rule stated under Eq. 2 and Eq. 3)."""
    return 1.0 / (norms + eps)


def penalty_l2(norms: np.ndarray, gamma: Optional[np.ndarray]) -> float:
    """sum_g gamma_g * ||W_g||_2 : the regulariser of Eq. 2 / Eq. 3 without the factor lambda.

    gamma=None means gamma == 1, which is the plain group-Lasso term printed before Eq. 2.
    """
    if gamma is None:
        return float(norms.sum())
    return float((gamma * norms).sum())


def alpha_update_sq(sumsq: np.ndarray, eps: float) -> np.ndarray:
    """Squared-norm variant of the reweighting: alpha = 1 / (||W_g||^2 + eps).

    The paper uses the norm itself (`gamma_update`); this variant exists because a caller may ask
    for the penalty on squared norms.  It is the same update with S_g in place of ||W_g||.
    """
    return 1.0 / (sumsq + eps)


def penalty_l2sq(sumsq: np.ndarray, alpha: Optional[np.ndarray]) -> float:
    """sum_g alpha_g * ||W_g||^2  (squared-norm variant; alpha=None means alpha == 1)."""
    if alpha is None:
        return float(sumsq.sum())
    return float((alpha * sumsq).sum())


def penalty_grad_values(w: np.ndarray, block: int, orient: str, gamma: np.ndarray, squared: bool = False) -> np.ndarray:
    """Gradient with respect to W of the regulariser with the penalty weights held fixed, as
    Algorithm 2 holds gamma between milestones while Adam minimises `mixed_loss`.

    Eq. 2 / Eq. 3 form:  d/dW_e [ gamma_g ||W_g||_2 ] = gamma_g * W_e / ||W_g||_2   (0 for an all-zero group,
    the minimum-norm subgradient).  Squared-norm variant:  d/dW_e [ alpha_g ||W_g||^2 ] = 2 alpha_g W_e.
    w: float64 values [rows, cols]; gamma: per-group array; result [rows, cols], without the factor lambda.
    """
    w = np.asarray(w, dtype=np.float64)
    full_gamma = _expand(np.asarray(gamma, dtype=np.float64), block, orient)
    if squared:
        return 2.0 * full_gamma * w
    n = _expand(np.sqrt(group_sumsq_values(w, block, orient)), block, orient)
    with np.errstate(divide="ignore", invalid="ignore"):
        g = np.where(n > 0, full_gamma * w / n, 0.0)
    return g


def penalty_grad(w_bits: np.ndarray, block: int, orient: str, gamma: np.ndarray, squared: bool = False) -> np.ndarray:
    """`penalty_grad_values` on bf16 weights."""
    return penalty_grad_values(bf16_to_f64(w_bits), block, orient, gamma, squared)


# ---------------------------------------------------------------------------
# the keep decision  (Algorithm 1: prune iff l2 norm <= t_b)
# ---------------------------------------------------------------------------
def decision_sumsq32(w_bits: np.ndarray, block: int, orient: str) -> np.ndarray:
    """The float32 quantity on which the keep decision is taken.

    Defined exactly: start from +0 and add the squares of the group's elements one at a time in
    increasing index order (row index for "C", column index for "R"), each addition rounded to
    float32.  The square of a bf16 value has at most 16 significant bits, so it is exact in
    float32 and the only roundings are those of the additions; the value therefore does not
    depend on whether a device fuses the multiply and the add.
    """
    u = np.ascontiguousarray(w_bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    g = _grouped(u.view(np.float32), block, orient)
    acc = np.zeros(g.shape[:-1], dtype=np.float32)
    for e in range(g.shape[-1]):
        x = g[..., e]
        acc = (acc + x * x).astype(np.float32)
    return acc


def threshold_sq32(t_b: float) -> np.float32:
    """t_b squared in float32: the value the float32 sum of squares is compared with."""
    t = np.float32(t_b)
    return np.float32(t * t)


def keep_flags(w_bits: np.ndarray, block: int, orient: str, t_b: float) -> np.ndarray:
    """keep_g = not (l2 norm <= t_b), the negation of Algorithm 1's test, per group.

    Taken as S32_g > t_b^2 in float32 (see `decision_sumsq32`); a negative t_b prunes nothing,
    since no norm is <= a negative number.  t_b = 0 keeps exactly the groups holding a non-zero
    weight, which is the group-level form of Algorithm 2's Mask = (W != 0).
    """
    s32 = decision_sumsq32(w_bits, block, orient)
    if t_b < 0:
        return np.ones(s32.shape, dtype=bool)
    return s32 > threshold_sq32(t_b)


def _expand(keep: np.ndarray, block: int, orient: str) -> np.ndarray:
    return np.repeat(keep, block, axis=0 if orient == "C" else 1)


def prune(w_bits: np.ndarray, block: int, orient: str, t_b: float) -> np.ndarray:
    """Algorithm 1 (vectorised): W_p = W with every group whose norm is <= t_b set to zero."""
    keep = _expand(keep_flags(w_bits, block, orient, t_b), block, orient)
    return np.where(keep, w_bits, np.uint16(0)).astype(np.uint16)


def prune_groupwise(w_bits: np.ndarray, block: int, orient: str, t_b: float) -> np.ndarray:
    """Algorithm 1's decision rule applied group by group, for small matrices (a slow cross-check of `prune`).

    Every group is visited on its own, in no particular order: its elements are taken as an explicit
    slice of W, the float32 decision quantity is summed element by element, and the test
    "norm <= t_b" (as S32 <= t_b^2, like `keep_flags`) fills one entry of a keep table.  The table is
    then applied to a copy of W in a single masking step.
    """
    m, n = w_bits.shape
    if (m if orient == "C" else n) % block:
        raise ValueError("block must divide the pruned dimension")
    vals = bf16_to_f64(w_bits).astype(np.float32)
    t2 = threshold_sq32(t_b)
    table = np.ones((m, n), dtype=bool)
    groups = [(slice(b * block, (b + 1) * block), slice(j, j + 1)) for b in range(m // block) for j in range(n)] \
        if orient == "C" else \
        [(slice(i, i + 1), slice(a * block, (a + 1) * block)) for a in range(n // block) for i in range(m)]
    for rows, cols in reversed(groups):
        acc = np.float32(0.0)
        for x in vals[rows, cols].ravel():          # increasing row index (C) / column index (R)
            acc = np.float32(acc + x * x)
        if t_b >= 0 and acc <= t2:
            table[rows, cols] = False
    return np.where(table, w_bits, np.uint16(0)).astype(np.uint16)


def mask_of(w_pruned_bits: np.ndarray) -> np.ndarray:
    """Algorithm 2's mask loop: Mask_ij = 0 if W_ij == 0 else 1 (both signs of zero count as zero)."""
    return (np.ascontiguousarray(w_pruned_bits, dtype=np.uint16) & np.uint16(0x7FFF)) != 0


def group_any(mask: np.ndarray, block: int, orient: str) -> np.ndarray:
    """Group-level mask: a group is kept iff any of its elements has Mask = 1."""
    return _grouped(mask, block, orient).any(axis=-1)


# ---------------------------------------------------------------------------
# choosing t_b from a percentile, or a keep count per block  (Section 3.1 allows a given
# threshold or a percentile)
# ---------------------------------------------------------------------------
def percentile_threshold(w_bits: np.ndarray, block: int, orient: str, rate: float) -> float:
    """Per-matrix threshold for a target compression rate c = total/kept.

    With G groups, r = floor(G * (1 - 1/c)) groups are to go: t_b is derived from the r-th
    smallest float32 sum of squares S (1-based); r = 0 returns -1 (prune nothing).  t_b is the
    float32 square root of S, bumped up by single ulps until its float32 square is >= S, so that
    Algorithm 1's `<=` test removes that group and every group tied with it.
    """
    s32 = decision_sumsq32(w_bits, block, orient).ravel()
    r = int(math.floor(s32.size * (1.0 - 1.0 / rate)))
    if r <= 0:
        return -1.0
    s_r = np.float32(np.partition(s32, r - 1)[r - 1])
    t = np.float32(np.sqrt(s_r))
    while np.float32(t * t) < s_r:
        t = np.nextafter(t, np.float32(np.inf))
    return float(t)


def keep_topk_per_block(w_bits: np.ndarray, block: int, orient: str, keep_count: int) -> np.ndarray:
    """Keep exactly `keep_count` groups in every block: the largest by float32 sum of squares.

    Ties: the larger S first, then the lower group index within the block.  A "block" is a
    row-block for "C" (its groups are its columns) and a vertical strip for "R" (its groups are
    its rows).
    """
    s32 = decision_sumsq32(w_bits, block, orient)
    per_block = s32 if orient == "C" else s32.T            # [blocks, groups in block]
    keep = np.zeros(per_block.shape, dtype=bool)
    for b in range(per_block.shape[0]):
        idx = sorted(range(per_block.shape[1]), key=lambda g: (-float(per_block[b, g]), g))
        keep[b, idx[:keep_count]] = True
    return keep if orient == "C" else np.ascontiguousarray(keep.T)


# ---------------------------------------------------------------------------
# Algorithm 2, retraining loop: "Update W using Adam", then W = W * Mask
# ---------------------------------------------------------------------------
def adam_step_masked(w: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, step: int, lr: float,
                     beta1: float, beta2: float, eps: float, weight_decay: float,
                     mask: Optional[np.ndarray]) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One iteration of Algorithm 2's retraining loop on one weight matrix, in float64.

    The algorithm says only "update W ... using Adam" and then "W = W * Mask".  Adam is taken as
    published (Kingma & Ba, 2015, Algorithm 1, with bias correction), `step` counting from 1:
        m <- beta1 m + (1 - beta1) g          v <- beta2 v + (1 - beta2) g^2
        mhat = m / (1 - beta1^step)           vhat = v / (1 - beta2^step)
        W <- W - lr * mhat / (sqrt(vhat) + eps)
    A weight decay, which the paper does not mention, is the decoupled one (W <- W - lr * wd * W, taken
    on the old W) and is 0 unless asked for.  The moments are updated for every weight, pruned or not,
    as the algorithm's order of operations implies; then the mask is applied to W only.
    mask None = the reweighted-training loop's plain update (no mask yet).
    Returns (W, m, v).
    """
    w = np.asarray(w, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    m_new = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v_new = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    mhat = m_new / (1.0 - beta1 ** step)
    vhat = v_new / (1.0 - beta2 ** step)
    w_new = w - lr * mhat / (np.sqrt(vhat) + eps) - lr * weight_decay * w
    if mask is not None:
        w_new = w_new * np.asarray(mask, dtype=np.float64)
    return w_new, m_new, v_new


def repack_values(w_bits: np.ndarray, blk_ptr: np.ndarray, idx: np.ndarray, block: int) -> np.ndarray:
    """Packed tiles of an UPDATED W under a fixed set of kept columns (orientation C): Algorithm 2 fixes the
    mask before retraining, so the storage of Section 3.1 keeps its indices and only its values change.
    Tile of row-block b: rows [b*block, (b+1)*block) restricted to idx[blk_ptr[b]:blk_ptr[b+1]], row-major."""
    rows = w_bits.shape[0]
    out = []
    for b in range(rows // block):
        cols = idx[blk_ptr[b]:blk_ptr[b + 1]]
        out.append(np.ascontiguousarray(w_bits[b * block:(b + 1) * block][:, cols]).reshape(-1))
    return np.concatenate(out) if out else np.zeros(0, dtype=np.uint16)


# ---------------------------------------------------------------------------
# compressed storage  (Section 3.1: only non-zero rows/columns at block level are indexed)
# ---------------------------------------------------------------------------
def pack(w_bits: np.ndarray, keep: np.ndarray, block: int, orient: str
         ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Canonical packed form of W restricted to the kept groups.

    "C": blk_ptr[b] = number of kept groups in row-blocks before b (int32, rows/d + 1 entries);
         idx[blk_ptr[b]:blk_ptr[b+1]] = kept column indices of row-block b, ascending;
         vals = for each row-block in order a dense [d, kc_b] row-major tile of the kept columns'
         bit patterns, starting at element d * blk_ptr[b].
    "R": the same with strips of h columns as blocks: idx holds kept row indices of each strip,
         and the tile of strip a is [kc_a, h] row-major at element h * blk_ptr[a].
    """
    rows, cols = w_bits.shape
    per_block = keep if orient == "C" else np.ascontiguousarray(keep.T)
    n_blocks = per_block.shape[0]
    blk_ptr = np.zeros(n_blocks + 1, dtype=np.int32)
    idx_parts, val_parts = [], []
    for b in range(n_blocks):
        kept = np.flatnonzero(per_block[b]).astype(np.int32)
        blk_ptr[b + 1] = blk_ptr[b] + kept.size
        idx_parts.append(kept)
        if orient == "C":
            tile = w_bits[b * block:(b + 1) * block, :][:, kept]       # [d, kc]
        else:
            tile = w_bits[:, b * block:(b + 1) * block][kept, :]       # [kc, h]
        val_parts.append(np.ascontiguousarray(tile).ravel())
    idx = np.concatenate(idx_parts) if idx_parts else np.zeros(0, np.int32)
    vals = np.concatenate(val_parts) if val_parts else np.zeros(0, np.uint16)
    return blk_ptr, idx.astype(np.int32), vals.astype(np.uint16)


def unpack(blk_ptr: np.ndarray, idx: np.ndarray, vals: np.ndarray, rows: int, cols: int,
           block: int, orient: str) -> np.ndarray:
    """Inverse of `pack`: the dense [rows, cols] matrix with zeros in the pruned groups."""
    out = np.zeros((rows, cols), dtype=np.uint16)
    for b in range(len(blk_ptr) - 1):
        lo, hi = int(blk_ptr[b]), int(blk_ptr[b + 1])
        kept = idx[lo:hi]
        tile = vals[block * lo: block * hi]
        if orient == "C":
            out[b * block:(b + 1) * block, kept] = tile.reshape(block, hi - lo)
        else:
            out[kept, b * block:(b + 1) * block] = tile.reshape(hi - lo, block)
    return out


def compression_rate(rows: int, cols: int, kept_weights: int) -> Fraction:
    """Compression rate = total weights / kept weights, as an exact fraction.

    (Section 4.4 equates a rate of 1.428x with 30% sparsity, i.e. rate = 1 / (1 - sparsity).)
    """
    return Fraction(rows * cols, kept_weights)


def storage_words_coo(nnz: int) -> int:
    """COO storage: three vectors (row, col, data), one entry each per non-zero (Section 4.4)."""
    return 3 * nnz


def storage_words_block_structured(nnz: int, n_groups: int) -> int:
    """Block-structured storage as Section 4.4's worked example counts it: the kept values plus
    one word per group of the matrix."""
    return nnz + n_groups


# ---------------------------------------------------------------------------
# the linear layer  Y = act(X W^T + b)  over the pruned weight
# ---------------------------------------------------------------------------
def gelu(x: np.ndarray) -> np.ndarray:
    """Exact (erf) GELU, x * Phi(x) = 0.5 x (1 + erf(x / sqrt 2)), the activation of BERT's FFN."""
    return 0.5 * x * (1.0 + _erf_vec(x / math.sqrt(2.0)))


def linear_masked_dense(x_bits: np.ndarray, w_bits: np.ndarray, mask: np.ndarray,
                        bias_bits: Optional[np.ndarray], act: int) -> np.ndarray:
    """Y[t, n] = act( sum_k X[t,k] * (W[n,k] * Mask[n,k]) + b[n] ) in float64 over all K terms.

    This is the plain definition of what a pruned layer computes: the dense product with the
    mask applied (Algorithm 2: W = W * Mask).  act: 0 identity, 1 GELU.
    """
    x = bf16_to_f64(x_bits)
    w = bf16_to_f64(w_bits) * mask
    y = x @ w.T
    if bias_bits is not None:
        y = y + bf16_to_f64(bias_bits)[None, :]
    return gelu(y) if act == 1 else y


def linear_from_packed(x_bits: np.ndarray, blk_ptr: np.ndarray, idx: np.ndarray, vals: np.ndarray,
                       n_out: int, block: int, bias_bits: Optional[np.ndarray], act: int
                       ) -> np.ndarray:
    """Second, independent evaluation straight from the packed form (orientation "C").

    Row-block b only reads the columns of X listed in its index list.  Used to check the
    invariant packed product == masked dense product; not the parity reference itself.
    """
    x = bf16_to_f64(x_bits)
    y = np.zeros((x.shape[0], n_out), dtype=np.float64)
    for b in range(n_out // block):
        lo, hi = int(blk_ptr[b]), int(blk_ptr[b + 1])
        if hi > lo:
            tile = bf16_to_f64(vals[block * lo: block * hi]).reshape(block, hi - lo)
            y[:, b * block:(b + 1) * block] = x[:, idx[lo:hi]] @ tile.T
    if bias_bits is not None:
        y = y + bf16_to_f64(bias_bits)[None, :]
    return gelu(y) if act == 1 else y


def linear_backward_input(dy_bits: np.ndarray, w_bits: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """dX[t, k] = sum_n dY[t, n] * (W[n, k] * Mask[n, k]): the gradient of the masked layer of Algorithm 2's
    retraining loop (W = W * Mask) with respect to its input, float64."""
    return bf16_to_f64(dy_bits) @ (bf16_to_f64(w_bits) * mask)


def linear_backward_weight(dy_bits: np.ndarray, x_bits: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """dW[n, k] = Mask[n, k] * sum_t dY[t, n] * X[t, k]: the gradient with respect to the weight of the masked
    layer of Algorithm 2's retraining loop; pruned positions get no gradient (W = W * Mask).  float64."""
    return (bf16_to_f64(dy_bits).T @ bf16_to_f64(x_bits)) * mask


def row_scales(x_bits: np.ndarray, w_bits: np.ndarray, mask: np.ndarray,
               bias_bits: Optional[np.ndarray]) -> np.ndarray:
    """||X[t,:]||_2 * ||(W*Mask)[n,:]||_2 + |b[n]|: the magnitude an output's error is judged against."""
    xn = np.sqrt((bf16_to_f64(x_bits) ** 2).sum(axis=1))
    wn = np.sqrt(((bf16_to_f64(w_bits) * mask) ** 2).sum(axis=1))
    s = xn[:, None] * wn[None, :]
    if bias_bits is not None:
        s = s + np.abs(bf16_to_f64(bias_bits))[None, :]
    return s
