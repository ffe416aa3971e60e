"""bsp_prune_pack_static: the pack entry point for callers that cannot hand over a workspace
(a host whose framework owns all device memory, or a thread that must not call cudaMalloc).

Its scratch is a fixed array inside the library, so the call allocates nothing.  The GPU test
drives it through the C ABI twice in a row, on different matrices so that the second call runs
on scratch still holding the first call's contents, and requires bit-identical results to
bsp_prune_pack with a caller workspace.  This file sorts after the other test files on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2009_08065_b200 as bsp
import synth_inputs as si


def test_static_scratch_limit_is_enforced_on_the_host():
    """A shape whose scratch need exceeds the fixed array is refused before any CUDA call."""
    p = ctypes.c_void_p(0x1000)
    rows, cols, block = 8192, 8192, 8                    # 8.4 million groups: beyond the array
    assert bsp.bsp_pack_scratch_bytes(rows, cols, block) > (4 << 20)
    st = bsp.lib.bsp_prune_pack_static(p, rows, cols, cols, block, 0, 0.0, None, -1, None, p, p, p, None, None)
    assert st == -6
    # the limit counts what the pack touches (counts and flags), not the percentile call's float32 region
    assert bsp.bsp_pack_scratch_bytes(8192, 8192, 32) <= (4 << 20) < bsp.bsp_pack_bound(8192, 8192, 32)[2]
    assert bsp.lib.bsp_prune_pack_static(p, 10, 8, 8, 3, 0, 0.0, None, -1, None, p, p, p, None, None) == -2


@pytest.mark.gpu
def test_static_variant_matches_workspace_variant_twice_in_a_row():
    dev = "cuda"
    cases = [
        # (rows, cols, block, orient, threshold quantile, keep_per_block)
        (3072, 768, 16, bsp.ORIENT_C, 0.6, -1),
        (768, 768, 12, bsp.ORIENT_R, 0.3, -1),           # smaller: leaves stale bytes of the first call behind
        (768, 3072, 32, bsp.ORIENT_C, None, 1000),
    ]
    for n, (rows, cols, block, orient, quant, topk) in enumerate(cases):
        w_bits = si.student_t_bf16(77 + n, f"static{n}", (rows, cols), 3.0, 0.02)
        W = torch.from_numpy(w_bits.view(np.int16)).to(dev)
        thr = 0.0
        if quant is not None:
            norms = torch.empty((rows // block, cols) if orient == bsp.ORIENT_C else (rows, cols // block),
                                dtype=torch.float32, device=dev)
            bsp.bsp_group_norms(W, block, orient, 1e-3, bsp.PEN_L2, norms)
            thr = float(torch.quantile(norms.flatten()[:100000], quant).item())
        ref = bsp.PackedMatrix.allocate(rows, cols, block, orient, dev)
        out = bsp.PackedMatrix.allocate(rows, cols, block, orient, dev)
        for t in (ref.idx, ref.vals, out.idx, out.vals):
            t.zero_()                                     # entries past blk_ptr[-1] are not written by either call
        bsp.bsp_prune_pack(W, ref, thr, None, topk)
        bsp.bsp_prune_pack_static(W, out, thr, None, topk)
        torch.cuda.synchronize()
        assert 0 < int(ref.kept_weights.item()) < rows * cols
        assert torch.equal(out.keep, ref.keep)
        assert torch.equal(out.blk_ptr, ref.blk_ptr)
        assert torch.equal(out.idx, ref.idx)
        assert torch.equal(out.vals, ref.vals)
        assert torch.equal(out.kept_weights, ref.kept_weights)
