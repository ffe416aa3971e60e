"""ctypes binding of libbsp.so.  Same names as the C entry points; arguments are torch CUDA
tensors (or None) whose device pointers are handed to the library unchanged.

bf16 tensors may be passed either as torch.bfloat16 or as raw bit patterns (torch.uint16 /
torch.int16); the library only sees the pointer.  There is no CPU fallback: if the shared
library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

ORIENT_C, ORIENT_R = 0, 1
PEN_L2, PEN_L2SQ = 0, 1
ACT_NONE, ACT_GELU = 0, 1

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))


def library_path() -> str:
    return os.path.join(_PKG_DIR, "libbsp.so")


class BspError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {bsp_status_string(status)} (status {status}, cuda error {lib.bsp_last_cuda_error()})")


def _load() -> ctypes.CDLL:
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python paper_2009_08065_b200/build.py` "
            "(needs nvcc); this package has no fallback path")
    return ctypes.CDLL(path)


lib = _load()

_vp, _i, _f, _d = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_double
_sz, _szp = ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)

class _LayerJob(ctypes.Structure):
    """Mirror of `bsp_layer_job` in bsp.h."""
    _fields_ = [
        ("W", _vp), ("rows", _i), ("cols", _i), ("ldw", _i),
        ("threshold", _f), ("threshold_dev", _vp),
        ("norms", _vp), ("gamma_in", _vp), ("gamma_out", _vp), ("penalty", _vp),
        ("keep", _vp), ("blk_ptr", _vp), ("idx", _vp), ("vals", _vp), ("kept_weights", _vp),
        ("plan", _vp), ("plan_bytes", _sz),
        ("ws", _vp), ("ws_bytes", _sz),
    ]


class _ChainOp(ctypes.Structure):
    """Mirror of `bsp_chain_op` in bsp.h."""
    _fields_ = [
        ("plan", _vp), ("n_out", _i), ("k_in", _i), ("block", _i),
        ("bias", _vp), ("act", _i),
        ("Y", _vp), ("ldy", _i),
        ("src", _i), ("src_col", _i),
    ]


class _LinearCall(ctypes.Structure):
    """Mirror of `bsp_linear_call` in bsp.h."""
    _fields_ = [
        ("plan", _vp), ("gplan", _vp), ("kept_weights", ctypes.c_longlong),
        ("n_out", _i), ("k_in", _i), ("block", _i),
        ("X", _vp), ("ldx", _i), ("XT", _vp), ("ldxt", _i), ("tokens", _i),
        ("bias", _vp), ("act", _i),
        ("Y", _vp), ("ldy", _i), ("YT", _vp), ("ldyt", _i),
        ("plan_stable", _i),
    ]


_SIGNATURES = {
    "bsp_status_string": (ctypes.c_char_p, [_i]),
    "bsp_last_cuda_error": (_i, []),
    "bsp_group_norms": (_i, [_vp, _i, _i, _i, _i, _i, _f, _i, _vp, _vp, _vp, _vp, _vp]),
    "bsp_penalty_grad": (_i, [_vp, _i, _i, _i, _i, _i, _i, _vp, _f, _vp, _i, _i, _vp]),
    "bsp_pack_bound": (_i, [_i, _i, _i, _i, _szp, _szp, _szp]),
    "bsp_pack_scratch_bytes": (_i, [_i, _i, _i, _i, _szp]),
    "bsp_prune_pack": (_i, [_vp, _i, _i, _i, _i, _i, _f, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bsp_prune_pack_static": (_i, [_vp, _i, _i, _i, _i, _i, _f, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bsp_percentile_threshold": (_i, [_vp, _i, _i, _i, _i, _i, _d, _vp, _vp, _sz, _vp]),
    "bsp_apply_mask": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _vp]),
    "bsp_linear_gather_plan_bytes": (_i, [_i, _i, _i, _szp]),
    "bsp_linear_gather_plan": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "bsp_transpose": (_i, [_vp, _i, _i, _i, _vp, _i, _vp]),
    "bsp_linear_gathered": (_i, [_vp, _i, _i, _i, _vp, _i, _i, _vp, _i, _vp, _i, _vp]),
    "bsp_linear_gathered_ex": (_i, [_vp, _i, _i, _i, _vp, _i, _i, _vp, _i, _vp, _i, _i, _vp]),
    "bsp_masked_adam_step": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _i, _i, _f, _f, _f, _f, _f, _i, _vp, _i, _vp]),
    "bsp_dense_mask": (_i, [_vp, _i, _i, _i, _vp, _i, _vp]),
    "bsp_repack_values": (_i, [_vp, _i, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "bsp_prepare_batched": (_i, [ctypes.POINTER(_LayerJob), _i, _i, _f, _i, _vp]),
    "bsp_percentile_threshold_batched": (_i, [ctypes.POINTER(_LayerJob), _i, _i, ctypes.POINTER(_d), _vp]),
    "bsp_linear_plan_bytes": (_i, [_i, _i, _i, _szp]),
    "bsp_linear_plan": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "bsp_linear_plan_r": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "bsp_linear_plan_t": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "bsp_linear_backward_weight": (_i, [_vp, _i, _vp, _i, _i, _i, _i, _i, _vp, _vp, _i, _vp]),
    "bsp_linear_planned": (_i, [_vp, _i, _i, _i, _vp, _i, _i, _vp, _i, _vp, _i, _vp]),
    "bsp_linear_planned_ex": (_i, [_vp, _i, _i, _i, _vp, _i, _i, _vp, _i, _vp, _i, _i, _vp]),
    "bsp_linear": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _i, _i, _vp, _i, _vp, _i, _vp, _sz, _vp]),
    "bsp_linear_chain_ws_bytes": (_i, [_i, _i, _szp]),
    "bsp_linear_chain": (_i, [ctypes.POINTER(_ChainOp), _i, _vp, _i, _i, _vp, _sz, _vp]),
    "bsp_linear_route": (_i, [ctypes.POINTER(_LinearCall), ctypes.POINTER(_i)]),
    "bsp_linear_run": (_i, [ctypes.POINTER(_LinearCall), _i, ctypes.POINTER(_i), _vp]),
    "bsp_linear_tune": (_i, [ctypes.POINTER(_LinearCall), _i, ctypes.POINTER(_i), ctypes.POINTER(_f), ctypes.POINTER(_f), _vp]),
    "bsp_linear_status": (_i, [_vp]),
    "bsp_set_wait_limit_ms": (_i, [_i]),
    "bsp_wait_selftest": (_i, [ctypes.POINTER(_i), ctypes.POINTER(ctypes.c_longlong), _vp]),
    "bsp_linear_cuda_core": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _i, _i, _vp, _i, _vp, _i, _vp]),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(lib, _name)
    _fn.restype, _fn.argtypes = _res, _args

EXPORTED_SYMBOLS = tuple(_SIGNATURES)


def bsp_status_string(status: int) -> str:
    return lib.bsp_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


def _check(status: int, where: str) -> None:
    if status != 0:
        raise BspError(status, where)


def _ld(t: torch.Tensor) -> int:
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 2-D tensor with unit inner stride")
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _per_group_shape(rows: int, cols: int, block: int, orient: int) -> Tuple[int, int]:
    return (rows // block, cols) if orient == ORIENT_C else (rows, cols // block)


# ------------------------------------------------------------------------------------------
def bsp_group_norms(W: torch.Tensor, block: int, orient: int = ORIENT_C, eps: float = 1e-3, pen: int = PEN_L2,
                    norms: Optional[torch.Tensor] = None, gamma_in: Optional[torch.Tensor] = None,
                    gamma_out: Optional[torch.Tensor] = None, penalty: Optional[torch.Tensor] = None,
                    stream=None) -> None:
    """norms / gamma_out: float32 per-group tensors; penalty: one-element float64 tensor (all optional outputs)."""
    rows, cols = W.shape
    _check(lib.bsp_group_norms(_ptr(W), rows, cols, _ld(W), block, orient, eps, pen, _ptr(norms), _ptr(gamma_in),
                               _ptr(gamma_out), _ptr(penalty), _stream(stream)), "bsp_group_norms")


def bsp_penalty_grad(W: torch.Tensor, block: int, orient: int, pen: int, gamma: torch.Tensor, scale: float,
                     grad: torch.Tensor, accumulate: bool = False, stream=None) -> None:
    """grad: float32 [rows, cols]; gamma: float32 per-group tensor."""
    rows, cols = W.shape
    _check(lib.bsp_penalty_grad(_ptr(W), rows, cols, _ld(W), block, orient, pen, _ptr(gamma), scale, _ptr(grad),
                                _ld(grad), int(accumulate), _stream(stream)), "bsp_penalty_grad")


def bsp_pack_bound(rows: int, cols: int, block: int, orient: int = ORIENT_C) -> Tuple[int, int, int]:
    """(index entries, value elements, workspace bytes) in the worst case for this shape."""
    a, b, c = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib.bsp_pack_bound(rows, cols, block, orient, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "bsp_pack_bound")
    return a.value, b.value, c.value


def bsp_pack_scratch_bytes(rows: int, cols: int, block: int, orient: int = ORIENT_C) -> int:
    """Bytes of workspace that bsp_prune_pack itself uses (counts and flags)."""
    n = ctypes.c_size_t()
    _check(lib.bsp_pack_scratch_bytes(rows, cols, block, orient, ctypes.byref(n)), "bsp_pack_scratch_bytes")
    return n.value


@dataclass
class PackedMatrix:
    """Device buffers of the canonical packed form (sized for the worst case; blk_ptr[-1] entries are valid)."""
    rows: int
    cols: int
    block: int
    orient: int
    blk_ptr: torch.Tensor       # int32 [n_blocks + 1]
    idx: torch.Tensor           # int32
    vals: torch.Tensor          # bf16 bit patterns (uint16 storage viewed as int16)
    keep: torch.Tensor          # uint8 per-group flags
    kept_weights: torch.Tensor  # int64 [1]
    ws: torch.Tensor            # scratch

    @staticmethod
    def allocate(rows: int, cols: int, block: int, orient: int = ORIENT_C, device="cuda") -> "PackedMatrix":
        n_idx, n_val, ws_bytes = bsp_pack_bound(rows, cols, block, orient)
        n_blocks = rows // block if orient == ORIENT_C else cols // block
        return PackedMatrix(
            rows, cols, block, orient,
            torch.empty(n_blocks + 1, dtype=torch.int32, device=device),
            torch.empty(n_idx, dtype=torch.int32, device=device),
            torch.empty(n_val, dtype=torch.int16, device=device),
            torch.empty(_per_group_shape(rows, cols, block, orient), dtype=torch.uint8, device=device),
            torch.empty(1, dtype=torch.int64, device=device),
            torch.empty(ws_bytes, dtype=torch.uint8, device=device),
        )


def bsp_prune_pack(W: torch.Tensor, out: PackedMatrix, threshold: float = 0.0,
                   threshold_dev: Optional[torch.Tensor] = None, keep_per_block: int = -1, stream=None) -> None:
    rows, cols = W.shape
    _check(lib.bsp_prune_pack(_ptr(W), rows, cols, _ld(W), out.block, out.orient, threshold, _ptr(threshold_dev),
                              keep_per_block, _ptr(out.keep), _ptr(out.blk_ptr), _ptr(out.idx), _ptr(out.vals),
                              _ptr(out.kept_weights), _ptr(out.ws), out.ws.numel(), _stream(stream)),
           "bsp_prune_pack")


def bsp_prune_pack_static(W: torch.Tensor, out: PackedMatrix, threshold: float = 0.0,
                          threshold_dev: Optional[torch.Tensor] = None, keep_per_block: int = -1, stream=None) -> None:
    """bsp_prune_pack without a caller workspace: the scratch is a fixed array inside the library (out.ws is unused)."""
    rows, cols = W.shape
    _check(lib.bsp_prune_pack_static(_ptr(W), rows, cols, _ld(W), out.block, out.orient, threshold,
                                     _ptr(threshold_dev), keep_per_block, _ptr(out.keep), _ptr(out.blk_ptr),
                                     _ptr(out.idx), _ptr(out.vals), _ptr(out.kept_weights), _stream(stream)),
           "bsp_prune_pack_static")


def bsp_percentile_threshold(W: torch.Tensor, block: int, orient: int, rate: float, threshold_out: torch.Tensor,
                             ws: torch.Tensor, stream=None) -> None:
    rows, cols = W.shape
    _check(lib.bsp_percentile_threshold(_ptr(W), rows, cols, _ld(W), block, orient, rate, _ptr(threshold_out),
                                        _ptr(ws), ws.numel(), _stream(stream)), "bsp_percentile_threshold")


def bsp_apply_mask(W: torch.Tensor, block: int, orient: int, keep: torch.Tensor, stream=None) -> None:
    rows, cols = W.shape
    _check(lib.bsp_apply_mask(_ptr(W), rows, cols, _ld(W), block, orient, _ptr(keep), _stream(stream)),
           "bsp_apply_mask")


@dataclass
class LayerJob:
    """One matrix of a bsp_prepare_batched call (tensors as in the single-matrix calls; None = skip)."""
    W: torch.Tensor
    out: PackedMatrix
    threshold: float = 0.0
    threshold_dev: Optional[torch.Tensor] = None
    norms: Optional[torch.Tensor] = None
    gamma_in: Optional[torch.Tensor] = None
    gamma_out: Optional[torch.Tensor] = None
    penalty: Optional[torch.Tensor] = None
    plan: Optional[torch.Tensor] = None


def make_job_array(jobs):
    """The host descriptor array for bsp_prepare_batched; build it once and reuse it for repeated calls."""
    arr = (_LayerJob * len(jobs))()
    for a, j in zip(arr, jobs):
        rows, cols = j.W.shape
        a.W, a.rows, a.cols, a.ldw = _ptr(j.W), rows, cols, _ld(j.W)
        a.threshold, a.threshold_dev = j.threshold, _ptr(j.threshold_dev)
        a.norms, a.gamma_in, a.gamma_out, a.penalty = _ptr(j.norms), _ptr(j.gamma_in), _ptr(j.gamma_out), _ptr(j.penalty)
        a.keep, a.blk_ptr, a.idx, a.vals = _ptr(j.out.keep), _ptr(j.out.blk_ptr), _ptr(j.out.idx), _ptr(j.out.vals)
        a.kept_weights = _ptr(j.out.kept_weights)
        a.plan = _ptr(j.plan)
        a.plan_bytes = 0 if j.plan is None else j.plan.numel() * j.plan.element_size()
        a.ws, a.ws_bytes = _ptr(j.out.ws), j.out.ws.numel()
    return arr


def bsp_prepare_batched(jobs, block: int, eps: float = 1e-3, pen: int = PEN_L2, stream=None) -> None:
    """jobs: a list of LayerJob, or an array made by make_job_array."""
    arr = jobs if isinstance(jobs, ctypes.Array) else make_job_array(jobs)
    _check(lib.bsp_prepare_batched(arr, len(arr), block, eps, pen, _stream(stream)), "bsp_prepare_batched")


def bsp_percentile_threshold_batched(jobs, block: int, rates, stream=None) -> None:
    """Per-matrix percentile thresholds for a job array (each job's threshold_dev tensor receives its threshold)."""
    arr = jobs if isinstance(jobs, ctypes.Array) else make_job_array(jobs)
    r = (_d * len(arr))(*[float(v) for v in rates])
    _check(lib.bsp_percentile_threshold_batched(arr, len(arr), block, r, _stream(stream)), "bsp_percentile_threshold_batched")


def bsp_linear_plan_bytes(n_out: int, k_in: int, block: int) -> int:
    b = ctypes.c_size_t()
    _check(lib.bsp_linear_plan_bytes(n_out, k_in, block, ctypes.byref(b)), "bsp_linear_plan_bytes")
    return b.value


def bsp_linear_plan(packed: PackedMatrix, plan: torch.Tensor, stream=None) -> None:
    """Execution layout of a packed matrix of either orientation."""
    if packed.orient == ORIENT_R:
        _check(lib.bsp_linear_plan_r(_ptr(packed.blk_ptr), _ptr(packed.idx), _ptr(packed.vals), packed.rows, packed.cols,
                                     packed.block, _ptr(plan), plan.numel() * plan.element_size(), _stream(stream)),
               "bsp_linear_plan_r")
        return
    _check(lib.bsp_linear_plan(_ptr(packed.blk_ptr), _ptr(packed.idx), _ptr(packed.vals), packed.rows, packed.cols,
                               packed.block, _ptr(plan), plan.numel() * plan.element_size(), _stream(stream)),
           "bsp_linear_plan")


def bsp_linear_plan_t(packed: PackedMatrix, plan_t: torch.Tensor, stream=None) -> None:
    """Transposed execution layout (orientation C): the operand of dX = dY (W * Mask)."""
    _check(lib.bsp_linear_plan_t(_ptr(packed.blk_ptr), _ptr(packed.idx), _ptr(packed.vals), packed.rows, packed.cols,
                                 packed.block, _ptr(plan_t), plan_t.numel() * plan_t.element_size(), _stream(stream)),
           "bsp_linear_plan_t")


def bsp_linear_backward_weight(dY: torch.Tensor, X: torch.Tensor, block: int, keep: Optional[torch.Tensor],
                               dW: torch.Tensor, stream=None) -> None:
    """dW = (dY^T X) * Mask; dY [tokens, n_out], X [tokens, k_in], dW [n_out, k_in], all bf16."""
    _check(lib.bsp_linear_backward_weight(_ptr(dY), _ld(dY), _ptr(X), _ld(X), dY.shape[0], dY.shape[1], X.shape[1], block,
                                          _ptr(keep), _ptr(dW), _ld(dW), _stream(stream)), "bsp_linear_backward_weight")


def bsp_linear_planned(plan: torch.Tensor, n_out: int, k_in: int, block: int, X: torch.Tensor,
                       bias: Optional[torch.Tensor], act: int, Y: torch.Tensor, stream=None) -> None:
    _check(lib.bsp_linear_planned(_ptr(plan), n_out, k_in, block, _ptr(X), X.shape[0], _ld(X), _ptr(bias), act,
                                  _ptr(Y), _ld(Y), _stream(stream)), "bsp_linear_planned")


LINEAR_AUTO, LINEAR_ONE_CTA, LINEAR_CTA_PAIR = 0, 1, 2
LINEAR_PLAN_STABLE = 0x100     # OR into `algo`: the plan is older than the previous kernel in the stream
LINEAR_OUT_TRANSPOSED = 0x200  # OR into `algo`: Y is written as [n_out, tokens]


def bsp_linear_planned_ex(plan: torch.Tensor, n_out: int, k_in: int, block: int, X: torch.Tensor,
                          bias: Optional[torch.Tensor], act: int, Y: torch.Tensor, algo: int = LINEAR_AUTO,
                          stream=None) -> None:
    _check(lib.bsp_linear_planned_ex(_ptr(plan), n_out, k_in, block, _ptr(X), X.shape[0], _ld(X), _ptr(bias), act,
                                     _ptr(Y), _ld(Y), algo, _stream(stream)), "bsp_linear_planned_ex")


def bsp_linear(packed: PackedMatrix, X: torch.Tensor, bias: Optional[torch.Tensor], act: int, Y: torch.Tensor,
               ws: Optional[torch.Tensor], stream=None) -> None:
    _check(lib.bsp_linear(_ptr(packed.blk_ptr), _ptr(packed.idx), _ptr(packed.vals), packed.rows, packed.cols,
                          packed.block, _ptr(X), X.shape[0], _ld(X), _ptr(bias), act, _ptr(Y), _ld(Y), _ptr(ws),
                          0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)), "bsp_linear")


def bsp_masked_adam_step(W: torch.Tensor, grad: torch.Tensor, m: torch.Tensor, v: torch.Tensor,
                         keep: Optional[torch.Tensor], block: int, orient: int, lr: float, beta1: float, beta2: float,
                         eps: float, weight_decay: float, step: int, W_bf16: Optional[torch.Tensor] = None,
                         stream=None) -> None:
    """W, m, v, grad: float32 [rows, cols]; keep: per-group uint8 flags or None; W_bf16: optional bf16 output."""
    rows, cols = W.shape
    _check(lib.bsp_masked_adam_step(_ptr(W), _ptr(grad), _ptr(m), _ptr(v), rows, cols, _ld(W), _ld(grad), _ptr(keep),
                                    block, orient, lr, beta1, beta2, eps, weight_decay, step, _ptr(W_bf16),
                                    0 if W_bf16 is None else _ld(W_bf16), _stream(stream)), "bsp_masked_adam_step")


def bsp_dense_mask(W: torch.Tensor, mask: torch.Tensor, stream=None) -> None:
    """mask (uint8, same shape as W) = 1 where the bf16 weight is non-zero."""
    _check(lib.bsp_dense_mask(_ptr(W), W.shape[0], W.shape[1], _ld(W), _ptr(mask), _ld(mask), _stream(stream)),
           "bsp_dense_mask")


def bsp_repack_values(W: torch.Tensor, packed: PackedMatrix, stream=None) -> None:
    """Refreshes packed.vals from an updated bf16 W; blk_ptr and idx stay as they are."""
    _check(lib.bsp_repack_values(_ptr(W), W.shape[0], W.shape[1], _ld(W), packed.block, _ptr(packed.blk_ptr),
                                 _ptr(packed.idx), _ptr(packed.vals), _stream(stream)), "bsp_repack_values")


def bsp_linear_gather_plan_bytes(n_out: int, k_in: int, block: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib.bsp_linear_gather_plan_bytes(n_out, k_in, block, ctypes.byref(n)), "bsp_linear_gather_plan_bytes")
    return n.value


def bsp_linear_gather_plan(packed: PackedMatrix, gplan: torch.Tensor, stream=None) -> None:
    _check(lib.bsp_linear_gather_plan(_ptr(packed.blk_ptr), _ptr(packed.idx), _ptr(packed.vals), packed.rows,
                                      packed.cols, packed.block, _ptr(gplan), gplan.numel() * gplan.element_size(),
                                      _stream(stream)), "bsp_linear_gather_plan")


def bsp_transpose(X: torch.Tensor, XT: torch.Tensor, stream=None) -> None:
    _check(lib.bsp_transpose(_ptr(X), X.shape[0], X.shape[1], _ld(X), _ptr(XT), _ld(XT), _stream(stream)),
           "bsp_transpose")


def bsp_linear_gathered(gplan: torch.Tensor, n_out: int, k_in: int, block: int, XT: torch.Tensor,
                        bias: Optional[torch.Tensor], act: int, Y: torch.Tensor, stream=None) -> None:
    """XT is [k_in, tokens] (the transposed activations); Y is [tokens, n_out]."""
    _check(lib.bsp_linear_gathered(_ptr(gplan), n_out, k_in, block, _ptr(XT), XT.shape[1], _ld(XT), _ptr(bias), act,
                                   _ptr(Y), _ld(Y), _stream(stream)), "bsp_linear_gathered")


def bsp_linear_gathered_ex(gplan: torch.Tensor, n_out: int, k_in: int, block: int, XT: torch.Tensor,
                           bias: Optional[torch.Tensor], act: int, Y: torch.Tensor, out_transposed: bool = False,
                           stream=None) -> None:
    """As bsp_linear_gathered; with out_transposed the output tensor is [n_out, tokens]."""
    _check(lib.bsp_linear_gathered_ex(_ptr(gplan), n_out, k_in, block, _ptr(XT), XT.shape[1], _ld(XT), _ptr(bias), act,
                                      _ptr(Y), _ld(Y), int(out_transposed), _stream(stream)), "bsp_linear_gathered_ex")


@dataclass
class ChainOp:
    """One linear of a bsp_linear_chain call: reads X (src = -1) or the Y of an earlier op, from column src_col."""
    plan: torch.Tensor
    n_out: int
    k_in: int
    block: int
    bias: Optional[torch.Tensor]
    act: int
    Y: torch.Tensor
    src: int = -1
    src_col: int = 0


def make_chain_array(ops):
    """The host descriptor array for bsp_linear_chain; build it once and reuse it for repeated calls."""
    arr = (_ChainOp * len(ops))()
    for a, o in zip(arr, ops):
        a.plan, a.n_out, a.k_in, a.block = _ptr(o.plan), o.n_out, o.k_in, o.block
        a.bias, a.act = _ptr(o.bias), o.act
        a.Y, a.ldy = _ptr(o.Y), _ld(o.Y)
        a.src, a.src_col = o.src, o.src_col
    return arr


def bsp_linear_chain_ws_bytes(n_ops: int, tokens: int) -> int:
    b = ctypes.c_size_t()
    _check(lib.bsp_linear_chain_ws_bytes(n_ops, tokens, ctypes.byref(b)), "bsp_linear_chain_ws_bytes")
    return b.value


def bsp_linear_chain(ops, X: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    """ops: a list of ChainOp, or an array made by make_chain_array."""
    arr = ops if isinstance(ops, ctypes.Array) else make_chain_array(ops)
    _check(lib.bsp_linear_chain(arr, len(arr), _ptr(X), X.shape[0], _ld(X), _ptr(ws), ws.numel() * ws.element_size(),
                                _stream(stream)), "bsp_linear_chain")


def bsp_linear_cuda_core(packed: PackedMatrix, X: torch.Tensor, bias: Optional[torch.Tensor], act: int,
                         Y: torch.Tensor, stream=None) -> None:
    _check(lib.bsp_linear_cuda_core(_ptr(packed.blk_ptr), _ptr(packed.idx), _ptr(packed.vals), packed.rows,
                                    packed.cols, packed.block, _ptr(X), X.shape[0], _ld(X), _ptr(bias), act, _ptr(Y),
                                    _ld(Y), _stream(stream)), "bsp_linear_cuda_core")


def bsp_linear_status(stream=None) -> None:
    """Synchronises the stream; raises BspError(BSP_ERR_TIMEOUT) if a tensor-core launch gave up on a wait."""
    _check(lib.bsp_linear_status(_stream(stream)), "bsp_linear_status")


def bsp_set_wait_limit_ms(ms: int) -> None:
    """Limit of one device-side wait for kernels launched afterwards on the current device (default 2000 ms)."""
    _check(lib.bsp_set_wait_limit_ms(int(ms)), "bsp_set_wait_limit_ms")


def bsp_wait_selftest(stream=None) -> Tuple[int, int]:
    """Lets one CTA's bounded waits run out on purpose-made idle barriers; returns (waits that ran out, ns the
    mbarrier wait lasted).  bsp_linear_status reports BSP_ERR_TIMEOUT once afterwards."""
    n, ns = ctypes.c_int(0), ctypes.c_longlong(0)
    _check(lib.bsp_wait_selftest(ctypes.byref(n), ctypes.byref(ns), _stream(stream)), "bsp_wait_selftest")
    return n.value, ns.value


ROUTE_AUTO, ROUTE_ZERO_EXPANDED, ROUTE_GATHERED = 0, 1, 2


def make_linear_call(n_out: int, k_in: int, block: int, tokens: int, plan: Optional[torch.Tensor] = None,
                     gplan: Optional[torch.Tensor] = None, kept_weights: int = -1, X: Optional[torch.Tensor] = None,
                     XT: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None, act: int = ACT_NONE,
                     Y: Optional[torch.Tensor] = None, YT: Optional[torch.Tensor] = None, plan_stable: bool = False):
    """The descriptor of bsp_linear_route / bsp_linear_run / bsp_linear_tune (tensors as in the per-route calls)."""
    c = _LinearCall()
    c.plan, c.gplan, c.kept_weights = _ptr(plan), _ptr(gplan), int(kept_weights)
    c.n_out, c.k_in, c.block, c.tokens = n_out, k_in, block, tokens
    c.X, c.ldx = _ptr(X), 0 if X is None else _ld(X)
    c.XT, c.ldxt = _ptr(XT), 0 if XT is None else _ld(XT)
    c.bias, c.act = _ptr(bias), act
    c.Y, c.ldy = _ptr(Y), 0 if Y is None else _ld(Y)
    c.YT, c.ldyt = _ptr(YT), 0 if YT is None else _ld(YT)
    c.plan_stable = int(plan_stable)
    return c


def bsp_linear_route(call) -> int:
    r = _i(0)
    _check(lib.bsp_linear_route(ctypes.byref(call), ctypes.byref(r)), "bsp_linear_route")
    return r.value


def bsp_linear_run(call, route: int = ROUTE_AUTO, stream=None) -> int:
    """Runs the layer; returns the route taken (ROUTE_ZERO_EXPANDED or ROUTE_GATHERED)."""
    r = _i(0)
    _check(lib.bsp_linear_run(ctypes.byref(call), route, ctypes.byref(r), _stream(stream)), "bsp_linear_run")
    return r.value


def bsp_linear_tune(call, reps: int = 3, stream=None) -> Tuple[int, float, float]:
    """(faster route, ms of the zero-expanded route, ms of the gathering route); -1 for a route that is not possible."""
    r, a, b = _i(0), _f(0.0), _f(0.0)
    _check(lib.bsp_linear_tune(ctypes.byref(call), reps, ctypes.byref(r), ctypes.byref(a), ctypes.byref(b), _stream(stream)),
           "bsp_linear_tune")
    return r.value, a.value, b.value
