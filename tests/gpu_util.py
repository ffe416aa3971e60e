"""Helpers for the GPU parity tests: numpy bit patterns <-> CUDA tensors, and the error metrics."""
import numpy as np
import torch

import paper_2009_08065_b200 as bsp

DEV = "cuda"

GUARD_BYTES = 256
GUARD_PATTERN = 0xA5


class GuardedAllocations:
    """Stand-in for a memory checker: while active, every CUDA tensor made through torch's factory functions
    (torch.empty / zeros / ones / full / *_like, called by a test or by the binding's allocate helpers) is a view
    into a larger byte buffer with GUARD_BYTES of a known pattern before and after it.  `check()` asserts that
    no kernel wrote outside the tensors it was given.  The payload stays 256-byte aligned."""

    FACTORIES = ("empty", "zeros", "ones", "full")

    def __init__(self):
        self.live = []          # (raw byte buffer, payload bytes, description)
        self._saved = {}

    def _is_cuda(self, device):
        return device is not None and torch.device(device).type == "cuda"

    def _guarded(self, shape, dtype, device, what):
        dtype = dtype or torch.get_default_dtype()
        if isinstance(shape, int):
            shape = (shape,)
        shape = tuple(int(v) for v in shape)
        itemsize = torch.empty((), dtype=dtype).element_size()
        n = itemsize
        for v in shape:
            n *= v
        padded = (n + 255) // 256 * 256
        raw = self._saved["empty"](GUARD_BYTES + padded + GUARD_BYTES, dtype=torch.uint8, device=device)
        raw[:GUARD_BYTES] = GUARD_PATTERN
        raw[GUARD_BYTES + n:] = GUARD_PATTERN
        self.live.append((raw, n, f"{what}{shape} {dtype}"))
        return raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)

    def __enter__(self):
        alloc = self

        def wrap(name, orig):
            def factory(*size, **kw):
                if not alloc._is_cuda(kw.get("device")) or kw.get("pin_memory") or kw.get("out") is not None:
                    return orig(*size, **kw)
                args = list(size)
                fill = args.pop() if name == "full" else None
                shape = args[0] if len(args) == 1 and not isinstance(args[0], int) else tuple(args)
                t = alloc._guarded(shape, kw.get("dtype"), kw["device"], name)
                if name == "zeros":
                    t.zero_()
                elif name == "ones":
                    t.fill_(1)
                elif name == "full":
                    t.fill_(fill)
                return t
            return factory

        def wrap_like(name, orig):
            def like(t, **kw):
                device = kw.get("device", t.device)
                if not alloc._is_cuda(device) or kw.get("pin_memory"):
                    return orig(t, **kw)
                out = alloc._guarded(tuple(t.shape), kw.get("dtype", t.dtype), device, name)
                if name == "zeros_like":
                    out.zero_()
                return out
            return like

        for name in self.FACTORIES:
            self._saved[name] = getattr(torch, name)
        for name in ("empty_like", "zeros_like"):
            self._saved[name] = getattr(torch, name)
        for name in self.FACTORIES:
            setattr(torch, name, wrap(name, self._saved[name]))
        for name in ("empty_like", "zeros_like"):
            setattr(torch, name, wrap_like(name, self._saved[name]))
        return self

    def __exit__(self, *exc):
        for name, fn in self._saved.items():
            setattr(torch, name, fn)

    def check(self):
        if torch.cuda.is_available():
            torch.cuda.synchronize()
        for raw, n, what in self.live:
            head = raw[:GUARD_BYTES]
            tail = raw[GUARD_BYTES + n:]
            assert bool((head == GUARD_PATTERN).all()), f"bytes before {what} were overwritten"
            assert bool((tail == GUARD_PATTERN).all()), f"bytes after {what} were overwritten"
        return len(self.live)


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
