"""GPU parity: bsp_group_norms, bsp_prune_pack, bsp_percentile_threshold, bsp_apply_mask against the oracle.

Norms / gamma / penalty: relative error <= 1e-5 (float32 device arithmetic vs float64 oracle).
Keep flags, blk_ptr, index lists, packed values, kept-weight count, thresholds: bit-exact.
"""
import numpy as np
import pytest
import torch

import paper_2009_08065_b200 as bsp
import synth_inputs as si
from oracle import bsp_oracle as O
from gpu_util import DEV, assert_linear_close, bits_of, packed_to_host, to_dev

pytestmark = pytest.mark.gpu
REL = 1e-5


def run_norms(w_bits, block, orient, eps, pen, gamma_in=None, w_dev=None):
    rows, cols = w_bits.shape
    shape = (rows // block, cols) if orient == bsp.ORIENT_C else (rows, cols // block)
    norms = torch.full(shape, -1.0, dtype=torch.float32, device=DEV)
    gout = torch.full(shape, -1.0, dtype=torch.float32, device=DEV)
    pen_out = torch.full((1,), 123.0, dtype=torch.float64, device=DEV)
    gin = None if gamma_in is None else torch.from_numpy(gamma_in.astype(np.float32)).to(DEV)
    bsp.bsp_group_norms(to_dev(w_bits) if w_dev is None else w_dev, block, orient, eps, pen, norms, gin, gout, pen_out)
    torch.cuda.synchronize()
    return norms.cpu().numpy(), gout.cpu().numpy(), float(pen_out.item())


def check_norms(w_bits, block, orient, eps=1e-3, w_dev=None):
    o = "C" if orient == bsp.ORIENT_C else "R"
    n_ref = O.group_norms(w_bits, block, o)
    s_ref = O.group_sumsq(w_bits, block, o)
    # the paper's form
    n, g, p = run_norms(w_bits, block, orient, eps, bsp.PEN_L2, w_dev=w_dev)
    assert np.allclose(n, n_ref, rtol=REL, atol=0)
    g_ref = O.gamma_update(n_ref, eps)
    assert np.allclose(g, g_ref, rtol=REL, atol=0)
    assert p == pytest.approx(O.penalty_l2(n_ref, g_ref), rel=REL)
    # squared-norm variant
    n2, a, p2 = run_norms(w_bits, block, orient, eps, bsp.PEN_L2SQ, w_dev=w_dev)
    assert np.array_equal(n2, n)
    a_ref = O.alpha_update_sq(s_ref, eps)
    assert np.allclose(a, a_ref, rtol=REL, atol=0)
    assert p2 == pytest.approx(O.penalty_l2sq(s_ref, a_ref), rel=REL)
    # stale gamma from an earlier W, and gamma == 1 (plain group Lasso)
    stale = O.gamma_update(O.group_norms(si.normal_bf16(99, "old", w_bits.shape, 0.02), block, o), eps)
    _, _, p3 = run_norms(w_bits, block, orient, eps, bsp.PEN_L2, gamma_in=stale, w_dev=w_dev)
    assert p3 == pytest.approx(O.penalty_l2(n_ref, stale.astype(np.float32).astype(np.float64)), rel=REL)
    _, _, p4 = run_norms(w_bits, block, orient, eps, bsp.PEN_L2, gamma_in=np.ones_like(n_ref), w_dev=w_dev)
    assert p4 == pytest.approx(O.penalty_l2(n_ref, None), rel=REL)


@pytest.mark.parametrize("block", [16, 3, 12, 96, 8, 32, 64, 1])
def test_norms_orientation_c_768(block):
    spec = si.LinearSpec("n768", 768, 768, False, 2.0, block)
    wp, _ = si.make_pruned_weight(si.DEFAULT_SEED, spec)          # half of the groups are exactly zero
    check_norms(wp, block, bsp.ORIENT_C)


@pytest.mark.parametrize("block", [16, 3, 12, 4])
def test_norms_orientation_r(block):
    spec = si.LinearSpec("nr", 768, 3072, False, 2.0, block)
    wp, _ = si.make_pruned_weight(si.DEFAULT_SEED, spec, orient="R")
    check_norms(wp, block, bsp.ORIENT_R)


def test_norms_odd_shapes_and_strides():
    # cols not a multiple of 8 (scalar path), a padded leading dimension, and an odd base offset
    w = si.normal_bf16(5, "odd", (36, 50), 0.02)
    check_norms(w, 12, bsp.ORIENT_C)
    check_norms(w, 5, bsp.ORIENT_R)
    big = si.normal_bf16(6, "pad", (48, 72), 0.02)
    big_dev = to_dev(big)
    check_norms(np.ascontiguousarray(big[:, :64]), 16, bsp.ORIENT_C, w_dev=big_dev[:, :64])     # ld 72, vector path
    check_norms(np.ascontiguousarray(big[:, 3:67]), 16, bsp.ORIENT_C, w_dev=big_dev[:, 3:67])   # misaligned base
    check_norms(np.ascontiguousarray(big[:, 3:67]), 8, bsp.ORIENT_R, w_dev=big_dev[:, 3:67])


def test_norms_heavy_tailed_ffn_shape():
    w = si.student_t_bf16(si.DEFAULT_SEED, "t3", (3072, 768), 3.0, 0.02)
    check_norms(w, 32, bsp.ORIENT_C)


def test_norms_outputs_are_optional():
    w = si.normal_bf16(8, "opt", (64, 64), 0.02)
    pen = torch.zeros(1, dtype=torch.float64, device=DEV)
    bsp.bsp_group_norms(to_dev(w), 16, bsp.ORIENT_C, 1e-3, bsp.PEN_L2, None, None, None, pen)
    n_ref = O.group_norms(w, 16, "C")
    assert float(pen.item()) == pytest.approx(O.penalty_l2(n_ref, O.gamma_update(n_ref, 1e-3)), rel=REL)
    with pytest.raises(bsp.BspError):
        bsp.bsp_group_norms(to_dev(w), 16, bsp.ORIENT_C, 1e-3, bsp.PEN_L2, None, None, None, None)


# ---------------------------------------------------------------------------------------- pack
def check_pack(w_bits, block, orient, t_b=0.0, keep_per_block=-1, thr_dev=None, keep_ref=None):
    o = "C" if orient == bsp.ORIENT_C else "R"
    rows, cols = w_bits.shape
    if keep_ref is None:
        keep_ref = (O.keep_topk_per_block(w_bits, block, o, keep_per_block) if keep_per_block >= 0
                    else O.keep_flags(w_bits, block, o, t_b))
    ref_ptr, ref_idx, ref_vals = O.pack(w_bits, keep_ref, block, o)
    pk = bsp.PackedMatrix.allocate(rows, cols, block, orient, DEV)
    pk.idx.fill_(-7)
    bsp.bsp_prune_pack(to_dev(w_bits), pk, t_b, thr_dev, keep_per_block)
    torch.cuda.synchronize()
    blk_ptr, idx, vals, keep, kept = packed_to_host(pk)
    assert np.array_equal(keep, keep_ref)
    assert np.array_equal(blk_ptr, ref_ptr)
    assert np.array_equal(idx, ref_idx)
    assert np.array_equal(vals, ref_vals)
    assert kept == block * int(keep_ref.sum())
    return pk, keep_ref


@pytest.mark.parametrize("block,orient", [(16, 0), (3, 0), (12, 0), (96, 0), (3, 1), (12, 1), (16, 1)])
def test_pack_seeded_sets_zero_threshold(block, orient):
    spec = si.LinearSpec("pk", 768, 768, False, 2.0, block)
    wp, keep = si.make_pruned_weight(si.DEFAULT_SEED, spec, orient="CR"[orient])
    _, keep_ref = check_pack(wp, block, orient, 0.0)
    assert np.array_equal(keep_ref, keep)                       # exactly the drawn sets: rate 2.0


def test_pack_ffn_shapes_rate_3():
    for n, k in [(3072, 768), (768, 3072), (2304, 768)]:
        spec = si.LinearSpec(f"ffn{n}x{k}", n, k, False, 3.0, 16)
        wp, keep = si.make_pruned_weight(si.DEFAULT_SEED, spec)
        pk, _ = check_pack(wp, 16, bsp.ORIENT_C, 0.0)
        assert int(pk.kept_weights.item()) * 3 == n * k


def test_pack_thresholds_ties_and_limits():
    g = si.stream(3, 1)
    wf = g.integers(-3, 4, size=(48, 64)).astype(np.float32) / 8      # many exact ties and zero groups
    w = si.f32_to_bf16_bits(wf)
    for orient, block in [(0, 4), (1, 4), (0, 2), (1, 8)]:
        for t in [0.0, 0.25, 0.375, 0.5, 0.75, -1.0, 100.0, float(np.sqrt(np.float32(0.5)))]:
            check_pack(w, block, orient, t)


def test_pack_percentile_threshold_pipeline():
    w = si.student_t_bf16(si.DEFAULT_SEED, "pct", (768, 768), 3.0, 0.02)
    for orient, block in [(0, 32), (1, 12)]:
        o = "CR"[orient]
        for rate in (1.79, 1.0, 5.0):
            t_ref = O.percentile_threshold(w, block, o, rate)
            _, _, ws_bytes = bsp.bsp_pack_bound(768, 768, block, orient)
            ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
            t_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
            bsp.bsp_percentile_threshold(to_dev(w), block, orient, rate, t_dev, ws)
            torch.cuda.synchronize()
            assert np.float32(t_dev.item()) == np.float32(t_ref)        # bit-exact threshold
            check_pack(w, block, orient, t_b=123.0, thr_dev=t_dev, keep_ref=O.keep_flags(w, block, o, t_ref))


def test_pack_keep_count_per_block():
    w = si.normal_bf16(4, "topk", (96, 768), 0.02)
    check_pack(w, 16, bsp.ORIENT_C, keep_per_block=256)
    check_pack(w, 16, bsp.ORIENT_C, keep_per_block=0)
    check_pack(w, 16, bsp.ORIENT_C, keep_per_block=768)
    check_pack(np.ascontiguousarray(w.T), 16, bsp.ORIENT_R, keep_per_block=300)
    g = si.stream(5, 2)
    ties = si.f32_to_bf16_bits(g.integers(-2, 3, size=(32, 40)).astype(np.float32))
    check_pack(ties, 4, bsp.ORIENT_C, keep_per_block=13)
    check_pack(ties, 4, bsp.ORIENT_R, keep_per_block=9)


def test_apply_mask_matches_pruned_weight():
    w = si.normal_bf16(6, "am", (96, 80), 0.02)
    for orient, block in [(0, 12), (1, 5)]:
        o = "CR"[orient]
        t = float(np.median(O.group_norms(w, block, o)))
        keep = O.keep_flags(w, block, o, t)
        wd = to_dev(w).clone()
        bsp.bsp_apply_mask(wd, block, orient, torch.from_numpy(keep.astype(np.uint8)).to(DEV))
        torch.cuda.synchronize()
        assert np.array_equal(bits_of(wd), O.prune(w, block, o, t))      # Algorithm 1's W_p = W * Mask


# ---------------------------------------------------------------------------------------- fused, batched
def test_prepare_batched_matches_oracle_and_single_calls():
    """One call for four matrices of different shapes: norms, gamma, penalty, flags, pack and plan."""
    eps, block = 1e-3, 16
    shapes = [(2304, 768), (768, 768), (3072, 768), (768, 3072)]
    jobs, refs = [], []
    for n, (rows, cols) in enumerate(shapes):
        w = si.student_t_bf16(50 + n, f"batched{n}", (rows, cols), 3.0, 0.02)
        t_b = float(np.quantile(O.group_norms(w, block, "C"), 0.55 + 0.1 * n))
        pk = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        pk.idx.fill_(-7)
        shape = (rows // block, cols)
        job = bsp.LayerJob(
            W=to_dev(w), out=pk, threshold=t_b,
            norms=torch.empty(shape, dtype=torch.float32, device=DEV),
            gamma_out=torch.empty(shape, dtype=torch.float32, device=DEV),
            penalty=torch.full((1,), -5.0, dtype=torch.float64, device=DEV),
            plan=torch.empty(bsp.bsp_linear_plan_bytes(rows, cols, block), dtype=torch.uint8, device=DEV))
        jobs.append(job)
        refs.append((w, t_b))
    bsp.bsp_prepare_batched(jobs, block, eps, bsp.PEN_L2)
    torch.cuda.synchronize()
    for job, (w, t_b) in zip(jobs, refs):
        rows, cols = w.shape
        n_ref = O.group_norms(w, block, "C")
        g_ref = O.gamma_update(n_ref, eps)
        assert np.allclose(job.norms.cpu().numpy(), n_ref, rtol=REL, atol=0)
        assert np.allclose(job.gamma_out.cpu().numpy(), g_ref, rtol=REL, atol=0)
        assert float(job.penalty.item()) == pytest.approx(O.penalty_l2(n_ref, g_ref), rel=REL)
        keep_ref = O.keep_flags(w, block, "C", t_b)
        ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
        blk_ptr, idx, vals, keep, kept = packed_to_host(job.out)
        assert np.array_equal(keep, keep_ref) and np.array_equal(blk_ptr, ref_ptr)
        assert np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)
        assert kept == block * int(keep_ref.sum())
        plan = bits_of(job.plan.view(torch.int16)[: rows * cols].reshape(rows, cols))
        assert np.array_equal(plan, O.prune(w, block, "C", t_b))          # W * Mask, densely laid out
        # and the per-matrix calls give the same bits
        single = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        bsp.bsp_prune_pack(job.W, single, t_b)
        plan1 = torch.empty_like(job.plan)
        bsp.bsp_linear_plan(single, plan1)
        norms1 = torch.empty_like(job.norms)
        bsp.bsp_group_norms(job.W, block, bsp.ORIENT_C, eps, bsp.PEN_L2, norms1)
        torch.cuda.synchronize()
        assert torch.equal(norms1, job.norms) and torch.equal(plan1[: rows * cols * 2], job.plan[: rows * cols * 2])
        assert torch.equal(single.blk_ptr, job.out.blk_ptr)
    # repeated call: penalty is reproducible bit for bit
    first = [float(j.penalty.item()) for j in jobs]
    bsp.bsp_prepare_batched(jobs, block, eps, bsp.PEN_L2)
    torch.cuda.synchronize()
    assert [float(j.penalty.item()) for j in jobs] == first


def test_prepare_batched_optional_outputs_and_many_jobs():
    """More jobs than one launch holds, outputs skipped, the squared-norm penalty, stale gamma."""
    eps, block = 1e-2, 8
    jobs, ws = [], []
    for n in range(100):
        w = si.normal_bf16(70 + n, f"many{n}", (64 + 8 * (n % 20), 72), 0.02)
        pk = bsp.PackedMatrix.allocate(w.shape[0], 72, block, bsp.ORIENT_C, DEV)
        stale = (np.abs(si.bf16_bits_to_f32(si.normal_bf16(90 + n, "g", (w.shape[0] // block, 72), 1.0))) + 0.5).astype(np.float32)
        jobs.append(bsp.LayerJob(W=to_dev(w), out=pk, threshold=0.05,
                                 gamma_in=torch.from_numpy(stale).to(DEV) if n % 2 else None,
                                 penalty=torch.zeros(1, dtype=torch.float64, device=DEV)))
        ws.append((w, stale if n % 2 else None))
    bsp.bsp_prepare_batched(jobs, block, eps, bsp.PEN_L2SQ)
    torch.cuda.synchronize()
    for job, (w, stale) in zip(jobs, ws):
        s_ref = O.group_sumsq(w, block, "C")
        alpha = stale.astype(np.float64) if stale is not None else O.alpha_update_sq(s_ref, eps)
        assert float(job.penalty.item()) == pytest.approx(O.penalty_l2sq(s_ref, alpha), rel=REL)
        keep_ref = O.keep_flags(w, block, "C", 0.05)
        ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
        blk_ptr, idx, vals, keep, kept = packed_to_host(job.out)
        assert np.array_equal(blk_ptr, ref_ptr) and np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)
    # shapes the fused kernels do not take are refused as a whole
    odd = si.normal_bf16(1, "odd", (16, 50), 0.02)
    pk = bsp.PackedMatrix.allocate(16, 50, 8, bsp.ORIENT_C, DEV)
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_prepare_batched([jobs[0], bsp.LayerJob(W=to_dev(odd), out=pk)], 8)
    assert e.value.status == -6


def test_prepare_batched_streaming_batch_larger_than_the_gpu():
    """More row-blocks than CTAs fit on the GPU at once, with wide matrices split into column ranges:
    the streaming one-pass kernel (ticket order, published counts) against the oracle, bit for bit."""
    eps, block = 1e-3, 16
    shapes = [(768, 768), (3072, 768), (768, 3072)] * 8
    jobs, refs = [], []
    for n, (rows, cols) in enumerate(shapes):
        w = si.student_t_bf16(300 + n, f"stream{n}", (rows, cols), 3.0, 0.02)
        t_b = float(np.quantile(O.group_norms(w, block, "C"), 0.3 + 0.02 * n))
        pk = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        shape = (rows // block, cols)
        jobs.append(bsp.LayerJob(
            W=to_dev(w), out=pk, threshold=t_b,
            norms=torch.empty(shape, dtype=torch.float32, device=DEV),
            gamma_out=torch.empty(shape, dtype=torch.float32, device=DEV),
            penalty=torch.full((1,), -5.0, dtype=torch.float64, device=DEV),
            plan=torch.empty(bsp.bsp_linear_plan_bytes(rows, cols, block), dtype=torch.uint8, device=DEV)))
        refs.append((w, t_b))
    for _ in range(2):                                   # the second call starts from the first one's scratch
        bsp.bsp_prepare_batched(jobs, block, eps, bsp.PEN_L2)
        bsp.bsp_linear_status()                          # no bounded wait expired
        torch.cuda.synchronize()
        for job, (w, t_b) in zip(jobs, refs):
            rows, cols = w.shape
            n_ref = O.group_norms(w, block, "C")
            g_ref = O.gamma_update(n_ref, eps)
            assert np.allclose(job.norms.cpu().numpy(), n_ref, rtol=REL, atol=0)
            assert np.allclose(job.gamma_out.cpu().numpy(), g_ref, rtol=REL, atol=0)
            assert float(job.penalty.item()) == pytest.approx(O.penalty_l2(n_ref, g_ref), rel=REL)
            keep_ref = O.keep_flags(w, block, "C", t_b)
            ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
            blk_ptr, idx, vals, keep, kept = packed_to_host(job.out)
            assert np.array_equal(keep, keep_ref) and np.array_equal(blk_ptr, ref_ptr)
            assert np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)
            assert kept == block * int(keep_ref.sum())
            plan = bits_of(job.plan.view(torch.int16)[: rows * cols].reshape(rows, cols))
            assert np.array_equal(plan, O.prune(w, block, "C", t_b))
            job.out.idx.fill_(-7)
            job.penalty.fill_(-5.0)


@pytest.mark.parametrize("block,n_jobs,seed", [(16, 40, 900), (8, 9, 901), (32, 7, 902)])
def test_prepare_batched_matrices_of_unequal_sizes(block, n_jobs, seed):
    """Matrices with different row-block counts and widths (some split into column ranges, some of one
    block) in one call: items are numbered round by round across the matrices, and the rounds thin
    out as the short matrices run out.  40 matrices make several waves (tickets); 9 and 7 fit one wave.
    Odd kept counts per block exercise the unaligned tile paths.  Pack against the oracle, bit for bit."""
    rng = np.random.default_rng(seed)
    eps = 1e-3
    jobs, refs = [], []
    for n in range(n_jobs):
        rows = block * int(rng.choice([1, 2, 3, 5, 24, 48, 96]))
        cols = 8 * int(rng.choice([1, 3, 12, 96, 97, 200, 384]))
        w = si.student_t_bf16(seed + n, f"mixed{n}", (rows, cols), 3.0, 0.02)
        t_b = float(np.quantile(O.group_norms(w, block, "C"), float(rng.uniform(0.1, 0.9))))
        pk = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        pk.idx.fill_(-7)
        jobs.append(bsp.LayerJob(W=to_dev(w), out=pk, threshold=t_b,
                                 penalty=torch.full((1,), -5.0, dtype=torch.float64, device=DEV)))
        refs.append((w, t_b))
    for _ in range(2):                                   # the second call starts from the first one's scratch
        bsp.bsp_prepare_batched(jobs, block, eps, bsp.PEN_L2)
        bsp.bsp_linear_status()
        torch.cuda.synchronize()
        for job, (w, t_b) in zip(jobs, refs):
            keep_ref = O.keep_flags(w, block, "C", t_b)
            ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
            blk_ptr, idx, vals, keep, kept = packed_to_host(job.out)
            assert np.array_equal(keep, keep_ref) and np.array_equal(blk_ptr, ref_ptr)
            assert np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)
            assert kept == block * int(keep_ref.sum())
            n_ref = O.group_norms(w, block, "C")
            assert float(job.penalty.item()) == pytest.approx(O.penalty_l2(n_ref, O.gamma_update(n_ref, eps)), rel=REL)
            job.out.idx.fill_(-7)
            job.penalty.fill_(-5.0)


def test_prepare_batched_in_place_masks_w_and_writes_nothing_else():
    """A job whose plan is its W: the pruned groups are zeroed inside W (Algorithm 2's W = W * Mask), every other
    output is what the separate-plan call gives, a second call on the now-masked W with threshold 0 leaves W
    as it is, and the masked W runs through the linear layer as its own execution layout."""
    eps = 1e-3
    # the last case is beyond the one-pass kernel (32 column ranges per row-block) and takes the two-stage path
    for rows, cols, block in [(768, 768, 16), (768, 3072, 16), (3072, 768, 16), (192, 4096, 96)]:
        w = si.student_t_bf16(610 + rows + cols, f"inplace{rows}x{cols}", (rows, cols), 3.0, 0.02)
        t_b = float(np.quantile(O.group_norms(w, block, "C"), 0.6))
        W = to_dev(w)
        pk = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        pen = torch.zeros(1, dtype=torch.float64, device=DEV)
        bsp.bsp_prepare_batched([bsp.LayerJob(W=W, out=pk, threshold=t_b, penalty=pen, plan=W)], block, eps, bsp.PEN_L2)
        bsp.bsp_linear_status()
        keep_ref = O.keep_flags(w, block, "C", t_b)
        w_masked = O.prune(w, block, "C", t_b)
        assert np.array_equal(bits_of(W), w_masked)
        ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
        blk_ptr, idx, vals, keep, kept = packed_to_host(pk)
        assert np.array_equal(keep, keep_ref) and np.array_equal(blk_ptr, ref_ptr)
        assert np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)
        n_ref = O.group_norms(w, block, "C")
        assert float(pen.item()) == pytest.approx(O.penalty_l2(n_ref, O.gamma_update(n_ref, eps)), rel=REL)
        # second pass, threshold 0 on the masked matrix: same kept sets, W untouched
        pk2 = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        bsp.bsp_prepare_batched([bsp.LayerJob(W=W, out=pk2, threshold=0.0, plan=W)], block, eps, bsp.PEN_L2)
        bsp.bsp_linear_status()
        assert np.array_equal(bits_of(W), w_masked)
        assert torch.equal(pk2.blk_ptr, pk.blk_ptr) and torch.equal(pk2.keep, pk.keep)
        # W is now its own execution layout
        x = si.normal_bf16(3, "inplace_x", (200, cols), 1.0)
        y = torch.full((200, rows), 0x7FC0, dtype=torch.int16, device=DEV)
        bsp.bsp_linear_planned(W, rows, cols, block, to_dev(x), None, bsp.ACT_NONE, y)
        bsp.bsp_linear_status()
        mask = O.mask_of(w_masked)
        assert_linear_close(bits_of(y), O.linear_masked_dense(x, w_masked, mask, None, 0), O.row_scales(x, w_masked, mask, None))


@pytest.mark.parametrize("block", [3, 12, 96])
def test_prepare_batched_paper_block_heights(block):
    """The paper's block sizes (3, 12 and 96 rows): at 96 rows a row-block no longer fits the kernel's row
    buffer and is split into six column ranges that wait for one another's counts."""
    eps = 1e-3
    jobs, refs = [], []
    for n, (rows, cols) in enumerate([(768, 768), (96 * 4, 3072), (96, 72)]):
        w = si.student_t_bf16(500 + n, f"paperblk{block}_{n}", (rows, cols), 3.0, 0.02)
        t_b = float(np.quantile(O.group_norms(w, block, "C"), 0.5))
        pk = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        shape = (rows // block, cols)
        jobs.append(bsp.LayerJob(W=to_dev(w), out=pk, threshold=t_b,
                                 norms=torch.empty(shape, dtype=torch.float32, device=DEV),
                                 gamma_out=torch.empty(shape, dtype=torch.float32, device=DEV),
                                 penalty=torch.zeros(1, dtype=torch.float64, device=DEV),
                                 plan=torch.empty(bsp.bsp_linear_plan_bytes(rows, cols, block), dtype=torch.uint8, device=DEV)))
        refs.append((w, t_b))
    bsp.bsp_prepare_batched(jobs, block, eps, bsp.PEN_L2)
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    for job, (w, t_b) in zip(jobs, refs):
        rows, cols = w.shape
        n_ref = O.group_norms(w, block, "C")
        assert np.allclose(job.norms.cpu().numpy(), n_ref, rtol=REL, atol=0)
        assert np.allclose(job.gamma_out.cpu().numpy(), O.gamma_update(n_ref, eps), rtol=REL, atol=0)
        assert float(job.penalty.item()) == pytest.approx(O.penalty_l2(n_ref, O.gamma_update(n_ref, eps)), rel=REL)
        keep_ref = O.keep_flags(w, block, "C", t_b)
        ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
        blk_ptr, idx, vals, keep, kept = packed_to_host(job.out)
        assert np.array_equal(keep, keep_ref) and np.array_equal(blk_ptr, ref_ptr)
        assert np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)
        plan = bits_of(job.plan.view(torch.int16)[: rows * cols].reshape(rows, cols))
        assert np.array_equal(plan, O.prune(w, block, "C", t_b))


def test_prepare_batched_with_device_side_percentile_thresholds():
    """The heavy-tailed workload's recipe in batched form (32-row blocks, 1.79x): every matrix's threshold is
    found on the device (bsp_percentile_threshold) and read from there by the one batched call; kept counts
    differ from block to block, and the wide matrix is split into column ranges."""
    eps, block, rate = 1e-3, 32, 1.79
    shapes = [(768, 768), (3072, 768), (768, 3072), (768, 768), (768, 3072), (3072, 768)]
    jobs, refs = [], []
    for n, (rows, cols) in enumerate(shapes):
        w = si.student_t_bf16(400 + n, f"distil_batched{n}", (rows, cols), 3.0, 0.02)
        wd = to_dev(w)
        pk = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        t_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
        bsp.bsp_percentile_threshold(wd, block, bsp.ORIENT_C, rate, t_dev, pk.ws)
        shape = (rows // block, cols)
        jobs.append(bsp.LayerJob(W=wd, out=pk, threshold=123.0, threshold_dev=t_dev,       # the host value must be ignored
                                 norms=torch.empty(shape, dtype=torch.float32, device=DEV),
                                 penalty=torch.zeros(1, dtype=torch.float64, device=DEV),
                                 plan=torch.empty(bsp.bsp_linear_plan_bytes(rows, cols, block), dtype=torch.uint8, device=DEV)))
        refs.append(w)
    bsp.bsp_prepare_batched(jobs, block, eps, bsp.PEN_L2)
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    for job, w in zip(jobs, refs):
        rows, cols = w.shape
        t_ref = O.percentile_threshold(w, block, "C", rate)
        assert np.float32(job.threshold_dev.item()) == np.float32(t_ref)
        n_ref = O.group_norms(w, block, "C")
        assert np.allclose(job.norms.cpu().numpy(), n_ref, rtol=REL, atol=0)
        assert float(job.penalty.item()) == pytest.approx(O.penalty_l2(n_ref, O.gamma_update(n_ref, eps)), rel=REL)
        keep_ref = O.keep_flags(w, block, "C", t_ref)
        ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
        blk_ptr, idx, vals, keep, kept = packed_to_host(job.out)
        assert np.array_equal(keep, keep_ref) and np.array_equal(blk_ptr, ref_ptr)
        assert np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)
        counts = np.diff(blk_ptr)
        assert counts.min() < counts.max()
        assert abs(float(O.compression_rate(rows, cols, kept)) - rate) < 1e-3 * rate
        plan = bits_of(job.plan.view(torch.int16)[: rows * cols].reshape(rows, cols))
        assert np.array_equal(plan, O.prune(w, block, "C", t_ref))


def test_percentile_thresholds_for_a_batch_of_matrices():
    """bsp_percentile_threshold_batched: one call finds every matrix's threshold (different rates, a rate of 1 that
    prunes nothing, heavy ties); the device floats equal the oracle's thresholds and the single-matrix call's, bit
    for bit, and feed bsp_prepare_batched."""
    block = 16
    cases = [((768, 768), 1.79, "t"), ((3072, 768), 3.0, "t"), ((768, 3072), 5.0, "t"), ((256, 512), 1.0, "t"),
             ((512, 256), 2.0, "ties"), ((64, 72), 8.0, "t")]
    jobs, refs, rates = [], [], []
    for n, ((rows, cols), rate, kind) in enumerate(cases):
        if kind == "ties":            # few distinct values: many groups share the selected sum of squares
            g = si.stream(700 + n, 1)
            w = si.f32_to_bf16_bits(g.integers(-2, 3, size=(rows, cols)).astype(np.float32) / 8)
        else:
            w = si.student_t_bf16(700 + n, f"pbatch{n}", (rows, cols), 3.0, 0.02)
        pk = bsp.PackedMatrix.allocate(rows, cols, block, bsp.ORIENT_C, DEV)
        jobs.append(bsp.LayerJob(W=to_dev(w), out=pk, threshold=0.0,
                                 threshold_dev=torch.full((1,), 77.0, dtype=torch.float32, device=DEV)))
        refs.append(w)
        rates.append(rate)
    bsp.bsp_percentile_threshold_batched(jobs, block, rates)
    single = torch.zeros(1, dtype=torch.float32, device=DEV)
    for job, w, rate in zip(jobs, refs, rates):
        t_ref = O.percentile_threshold(w, block, "C", rate)
        assert np.float32(job.threshold_dev.item()) == np.float32(t_ref), (w.shape, rate)
        bsp.bsp_percentile_threshold(job.W, block, bsp.ORIENT_C, rate, single, job.out.ws)
        assert torch.equal(single, job.threshold_dev)
    bsp.bsp_prepare_batched(jobs, block, 1e-3, bsp.PEN_L2)
    bsp.bsp_linear_status()
    for job, w, rate in zip(jobs, refs, rates):
        keep_ref = O.keep_flags(w, block, "C", O.percentile_threshold(w, block, "C", rate))
        ref_ptr, ref_idx, ref_vals = O.pack(w, keep_ref, block, "C")
        blk_ptr, idx, vals, keep, kept = packed_to_host(job.out)
        assert np.array_equal(keep, keep_ref) and np.array_equal(blk_ptr, ref_ptr)
        assert np.array_equal(idx, ref_idx) and np.array_equal(vals, ref_vals)


# ---------------------------------------------------------------------------------------- penalty gradient
@pytest.mark.parametrize("orient,block,shape", [(0, 16, (768, 768)), (0, 3, (96, 50)), (1, 12, (96, 768)), (1, 5, (33, 50))])
def test_penalty_gradient(orient, block, shape):
    """G = lambda * gamma_g * W / ||W_g|| (and the squared-norm variant), gamma fixed; relative 1e-5 in float32."""
    o = "CR"[orient]
    rows, cols = shape
    spec = si.LinearSpec("pg", rows, cols, False, 2.0, block)
    wp, _ = si.make_pruned_weight(19, spec, orient=o)                  # half of the groups are all-zero
    gshape = (rows // block, cols) if orient == 0 else (rows, cols // block)
    gamma = O.gamma_update(O.group_norms(si.make_weight(20, spec), block, o), 1e-3).astype(np.float32)
    assert gamma.shape == gshape
    lam = 3e-4                                                          # a penalty factor from the paper's range
    wd, gd = to_dev(wp), torch.from_numpy(gamma).to(DEV)
    for pen, squared in ((bsp.PEN_L2, False), (bsp.PEN_L2SQ, True)):
        ref = lam * O.penalty_grad(wp, block, o, gamma.astype(np.float64), squared)
        grad = torch.full((rows, cols), 7.0, dtype=torch.float32, device=DEV)
        bsp.bsp_penalty_grad(wd, block, orient, pen, gd, lam, grad)
        torch.cuda.synchronize()
        assert np.allclose(grad.cpu().numpy(), ref, rtol=REL, atol=1e-12)
        assert (ref[~O.mask_of(wp)] == 0).all() and (grad.cpu().numpy()[~O.mask_of(wp)] == 0).all()
        # accumulate onto an existing gradient
        base = torch.from_numpy(si.bf16_bits_to_f32(si.normal_bf16(21, "tg", (rows, cols), 1e-3))).to(DEV)
        acc = base.clone()
        bsp.bsp_penalty_grad(wd, block, orient, pen, gd, lam, acc, accumulate=True)
        torch.cuda.synchronize()
        assert np.allclose(acc.cpu().numpy(), base.cpu().numpy().astype(np.float64) + ref, rtol=REL, atol=1e-9)
