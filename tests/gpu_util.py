"""Helpers for the GPU parity tests: numpy bit patterns <-> CUDA tensors, and the error metrics."""
import numpy as np
import torch

import paper_2009_08065_b200 as bsp

DEV = "cuda"


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> int16 CUDA tensor holding the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint16)


def packed_to_host(pk: bsp.PackedMatrix):
    blk_ptr = pk.blk_ptr.cpu().numpy()
    n = int(blk_ptr[-1])
    return blk_ptr, pk.idx.cpu().numpy()[:n], bits_of(pk.vals)[: n * pk.block], pk.keep.cpu().numpy().astype(bool), int(pk.kept_weights.item())


def upload_packed(blk_ptr, idx, vals, rows, cols, block, orient=0) -> bsp.PackedMatrix:
    """A PackedMatrix whose device buffers hold an oracle-made packed form."""
    pk = bsp.PackedMatrix.allocate(rows, cols, block, orient, DEV)
    pk.blk_ptr.copy_(torch.from_numpy(blk_ptr))
    pk.idx[: idx.size].copy_(torch.from_numpy(idx))
    pk.vals[: vals.size].copy_(torch.from_numpy(vals.view(np.int16)))
    return pk


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# Tolerances of the linear layer (bf16 inputs, float32 accumulation, bf16 output):
#   max over outputs of |Y - Y_ref| / (||x_t|| * ||w_n|| + |b_n|) <= 2e-2
#   sum |Y - Y_ref| / sum |Y_ref| <= 5e-3
MAX_SCALED_ERR = 2e-2
MEAN_REL_ERR = 5e-3


def linear_errors(y_bits: np.ndarray, y_ref: np.ndarray, scales: np.ndarray):
    y = bf16_bits_to_f64(y_bits)
    diff = np.abs(y - y_ref)
    max_scaled = float((diff / np.maximum(scales, 1e-30)).max()) if diff.size else 0.0
    mean_rel = float(diff.sum() / max(np.abs(y_ref).sum(), 1e-30))
    return max_scaled, mean_rel


def assert_linear_close(y_bits, y_ref, scales, what=""):
    assert np.isfinite(bf16_bits_to_f64(y_bits)).all(), what
    max_scaled, mean_rel = linear_errors(y_bits, y_ref, scales)
    assert max_scaled <= MAX_SCALED_ERR, f"{what}: max scaled error {max_scaled}"
    assert mean_rel <= MEAN_REL_ERR, f"{what}: mean relative error {mean_rel}"
    return max_scaled, mean_rel
