"""GPU parity of Algorithm 2's retraining step (bsp_masked_adam_step: Adam update, then W = W * Mask) and of the
value re-pack under fixed kept sets (bsp_repack_values), against the oracle.

Tolerances.  Moments: a sum of two rounded float32 terms: 3e-7 of the terms' magnitudes for m (the terms can
cancel), relative 1e-6 for v (both terms positive).  Weights: W' = fma(-lr, u, W) is rounded once
(half an ulp of W, 6e-8 |W|) and u = mhat / (sqrt(vhat) + eps) + wd W carries about five float32 roundings
(3e-7 relative, |u| of order 1), so |W' - W'_ref| <= 2e-7 |W'_ref| + 5e-6 lr.  The bf16 copy is the nearest-even
rounding of the float32 result the GPU itself produced, checked bit for bit; masked weights are exactly +0;
re-packed values are bit-exact.  The oracle gets the hyper-parameters rounded to float32, the
type in which the C ABI takes them.
"""
import numpy as np
import pytest
import torch

import paper_2009_08065_b200 as bsp
import synth_inputs as si
from oracle import bsp_oracle as O
from gpu_util import DEV, assert_linear_close, bits_of, packed_to_host, to_dev

pytestmark = pytest.mark.gpu


def f32_to_bf16_rne(a: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


@pytest.mark.parametrize("orient,block,shape,masked", [(0, 16, (768, 768), True), (0, 12, (96, 80), True),
                                                       (1, 5, (96, 80), True), (0, 16, (64, 72), False)])
def test_masked_adam_step_three_iterations(orient, block, shape, masked):
    rows, cols = shape
    o = "CR"[orient]
    spec = si.LinearSpec(f"adam{rows}x{cols}{o}", rows, cols, False, 2.0, block)
    wp, keep = si.make_pruned_weight(51, spec, orient=o)
    w0 = si.bf16_bits_to_f32(wp).astype(np.float32)
    mask = O.mask_of(wp) if masked else None
    # hyper-parameters as the C ABI receives them (float32), so that both sides start from the same numbers
    lr, b1, b2, eps, wd = (float(np.float32(h)) for h in (3e-5, 0.9, 0.999, 1e-8, 0.01))
    W = torch.from_numpy(w0.copy()).to(DEV)
    M = torch.zeros_like(W)
    V = torch.zeros_like(W)
    Wb = torch.full((rows, cols), 0x7FC0, dtype=torch.int16, device=DEV)
    keep_d = torch.from_numpy(keep.astype(np.uint8)).to(DEV) if masked else None
    for step in range(1, 4):
        g = (si.bf16_bits_to_f32(si.normal_bf16(60 + step, spec.name + ".g", (rows, cols), 1e-2)) *
             (1.0 + 0.5 * step)).astype(np.float32)
        w_prev, m_prev, v_prev = W.cpu().numpy(), M.cpu().numpy(), V.cpu().numpy()
        bsp.bsp_masked_adam_step(W, torch.from_numpy(g).to(DEV), M, V, keep_d, block, orient, lr, b1, b2, eps, wd,
                                 step, Wb)
        torch.cuda.synchronize()
        # the oracle takes the step from the state the GPU started it from
        w_ref, m_ref, v_ref = O.adam_step_masked(w_prev, g, m_prev, v_prev, step, lr, b1, b2, eps, wd, mask)
        w_gpu = W.cpu().numpy()
        # a moment is a sum of two rounded terms (of either sign for m): error relative to the terms
        m_terms = np.abs(b1 * m_prev.astype(np.float64)) + np.abs((1 - b1) * g.astype(np.float64))
        assert (np.abs(M.cpu().numpy() - m_ref) <= 3e-7 * m_terms).all()
        assert np.allclose(V.cpu().numpy(), v_ref, rtol=1e-6, atol=1e-30)
        assert (np.abs(w_gpu - w_ref) <= 2e-7 * np.abs(w_ref) + 5e-6 * lr).all()
        assert np.abs(w_gpu - w_prev).max() > 0.2 * lr                     # the step did move the weights
        if masked:
            assert not w_gpu.view(np.uint32)[~mask].any()                  # exactly +0
            assert (M.cpu().numpy()[~mask] != 0).any()                     # moments of pruned weights still move
        assert np.array_equal(bits_of(Wb), f32_to_bf16_rne(w_gpu))


def test_retrained_weights_feed_the_linear_layer_and_the_repack():
    """One retraining step on a pruned layer: the bf16 copy written by the step is the execution layout of
    bsp_linear_planned, and bsp_repack_values refreshes the packed tiles without touching the indices."""
    T, N, K, d = 192, 256, 384, 16
    spec = si.LinearSpec("retrain", N, K, True, 3.0, d)
    wp, keep = si.make_pruned_weight(52, spec)
    x = si.make_activations(52, spec.name, T, K)
    b = si.make_bias(52, spec)
    pk = bsp.PackedMatrix.allocate(N, K, d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(to_dev(wp), pk, 0.0)
    ptr0, idx0, _, _, _ = packed_to_host(pk)
    W = torch.from_numpy(si.bf16_bits_to_f32(wp).astype(np.float32)).to(DEV)
    M, V = torch.zeros_like(W), torch.zeros_like(W)
    g = si.bf16_bits_to_f32(si.normal_bf16(53, "retrain.g", (N, K), 1.0)).astype(np.float32)
    plan = torch.full((N, K), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_masked_adam_step(W, torch.from_numpy(g).to(DEV), M, V, pk.keep, d, bsp.ORIENT_C, 1e-3, 0.9, 0.999, 1e-8,
                             0.0, 1, plan)
    bsp.bsp_repack_values(plan, pk)
    y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_planned(plan, N, K, d, to_dev(x), to_dev(b), 1, y)
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    w_new = bits_of(plan)                                                # bf16 bits of the updated masked weights
    mask = O.mask_of(wp)
    assert not w_new[~mask].any() and (w_new[mask] != wp[mask]).mean() > 0.5    # a step of 1e-3 moves most weights
    ptr1, idx1, vals1, _, _ = packed_to_host(pk)
    assert np.array_equal(ptr1, ptr0) and np.array_equal(idx1, idx0)
    assert np.array_equal(vals1, O.repack_values(w_new, ptr0, idx0, d))
    y_ref = O.linear_masked_dense(x, w_new, mask, b, 1)
    assert_linear_close(bits_of(y), y_ref, O.row_scales(x, w_new, mask, b), "layer after one retraining step")


def test_repack_values_small_blocks_and_empty_blocks():
    rows, cols, d = 96, 50, 3
    spec = si.LinearSpec("repack3", rows, cols, False, 2.0, d)
    wp, keep = si.make_pruned_weight(54, spec)
    keep[2, :] = False
    wp = si.zero_groups(wp, keep, d, "C")
    pk = bsp.PackedMatrix.allocate(rows, cols, d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(to_dev(wp), pk, 0.0)
    ptr, idx, vals, _, _ = packed_to_host(pk)
    w2 = si.zero_groups(si.make_weight(55, spec), keep, d, "C")
    bsp.bsp_repack_values(to_dev(w2), pk)
    torch.cuda.synchronize()
    ptr2, idx2, vals2, _, _ = packed_to_host(pk)
    assert np.array_equal(ptr2, ptr) and np.array_equal(idx2, idx)
    assert np.array_equal(vals2, O.repack_values(w2, ptr, idx, d))


def test_dense_mask_is_algorithm_2s_mask():
    """Mask_ij = (W_ij != 0), negative zero included, on a ragged shape with a padded leading dimension; and
    its reduction over the groups is what bsp_prune_pack calls the keep flags at threshold 0."""
    rows, cols, d = 96, 50, 12
    spec = si.LinearSpec("dmask", rows, cols, False, 2.0, d)
    wp, keep = si.make_pruned_weight(56, spec)
    wp[5, 7] = 0x8000                                              # -0.0 is zero
    wide = np.zeros((rows, 64), dtype=np.uint16)
    wide[:, :cols] = wp
    wd = to_dev(wide)[:, :cols]                                    # leading dimension 64
    mask = torch.full((rows, cols), 9, dtype=torch.uint8, device=DEV)
    bsp.bsp_dense_mask(wd, mask)
    torch.cuda.synchronize()
    ref = O.mask_of(wp)
    assert np.array_equal(mask.cpu().numpy().astype(bool), ref) and mask.max().item() == 1
    pk = bsp.PackedMatrix.allocate(rows, cols, d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(to_dev(wp), pk, 0.0)
    torch.cuda.synchronize()
    assert np.array_equal(pk.keep.cpu().numpy().astype(bool), O.group_any(ref, d, "C"))
