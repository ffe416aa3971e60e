"""Pins for the CPU oracle: closed forms, hand-built cases, brute force, library special cases and
the numbers the paper prints.  None of these tests touches the CUDA path."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import synth_inputs as si
from oracle import bsp_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(a):
    """bf16 bit patterns of values that are exactly representable (asserted)."""
    a = np.asarray(a, dtype=np.float32)
    b = si.f32_to_bf16_bits(a)
    assert np.array_equal(si.bf16_bits_to_f32(b), a), "test value is not a bf16 number"
    return b


def rand_w(seed, rows, cols, std=0.02):
    return si.normal_bf16(seed, f"w{rows}x{cols}", (rows, cols), std)


# ----------------------------------------------------------------------------- decoding
def test_bf16_decode_known_patterns():
    pat = np.array([0x3F80, 0xBF80, 0x4000, 0x3F00, 0x0000, 0x8000, 0x4049], dtype=np.uint16)
    want = [1.0, -1.0, 2.0, 0.5, 0.0, -0.0, 3.140625]
    assert O.bf16_to_f64(pat).tolist() == want


# ----------------------------------------------------------------------------- norms
@pytest.mark.parametrize("orient", ["C", "R"])
def test_norms_hand_built_groups(orient):
    d = 4
    # four groups: all-equal 0.5 -> 0.5*sqrt(4) = 1 ; (3,4,0,0) -> 5 ; zeros -> 0 ; (2,-2,2,-2)*2^k -> 4*2^k
    g = np.array([[0.5, 0.5, 0.5, 0.5], [3, 4, 0, 0], [0, 0, 0, 0], [16, -16, 16, -16]], dtype=np.float32)
    w = bits(g.T if orient == "C" else g)          # "C": groups run down columns; "R": along rows
    n = O.group_norms(w, d, orient).ravel()
    assert n.tolist() == [1.0, 5.0, 0.0, 32.0]
    s = O.group_sumsq(w, d, orient).ravel()
    assert s.tolist() == [1.0, 25.0, 0.0, 1024.0]


@pytest.mark.parametrize("orient,block", [("C", 3), ("C", 16), ("R", 12), ("R", 4)])
def test_norms_match_numpy_linalg_on_explicit_slices(orient, block):
    rows, cols = 48, 24
    w = rand_w(1, rows, cols)
    wf = si.bf16_bits_to_f32(w).astype(np.float64)
    n = O.group_norms(w, block, orient)
    if orient == "C":
        assert n.shape == (rows // block, cols)
        for b in range(rows // block):
            for j in range(cols):
                assert n[b, j] == pytest.approx(np.linalg.norm(wf[b * block:(b + 1) * block, j]), rel=1e-14)
    else:
        assert n.shape == (rows, cols // block)
        for i in range(rows):
            for a in range(cols // block):
                assert n[i, a] == pytest.approx(np.linalg.norm(wf[i, a * block:(a + 1) * block]), rel=1e-14)


def test_orientations_are_transposes_of_each_other():
    w = rand_w(2, 24, 36)
    nc = O.group_norms(w, 4, "C")                       # [6, 36]
    nr = O.group_norms(np.ascontiguousarray(w.T), 4, "R")  # [36, 6]
    assert np.array_equal(nc, nr.T)


def test_block_must_divide():
    w = rand_w(3, 10, 12)
    with pytest.raises(ValueError):
        O.group_norms(w, 3, "C")
    with pytest.raises(ValueError):
        O.group_norms(w, 5, "R")


def test_frobenius_identity():
    """Sum of all group sums of squares is the squared Frobenius norm, for any block size."""
    w = rand_w(4, 96, 48)
    fro2 = (si.bf16_bits_to_f32(w).astype(np.float64) ** 2).sum()
    for orient, blk in [("C", 3), ("C", 12), ("C", 96), ("R", 3), ("R", 16)]:
        assert O.group_sumsq(w, blk, orient).sum() == pytest.approx(fro2, rel=1e-13)


# ----------------------------------------------------------------------------- gamma / penalty
def test_gamma_closed_form_and_zero_group():
    n = np.array([0.0, 1.0, 3.0, 1e-3])
    g = O.gamma_update(n, 1e-3)
    assert g[0] == pytest.approx(1000.0)
    assert g[1] == pytest.approx(1 / 1.001)
    assert g[2] == pytest.approx(1 / 3.001)
    assert g[3] == pytest.approx(500.0)


def test_penalty_closed_forms():
    w = rand_w(5, 32, 40)
    w[0:8, 3] = 0            # one all-zero group for d=8, "C"
    n = O.group_norms(w, 8, "C")
    s = O.group_sumsq(w, 8, "C")
    eps = 1e-3
    # gamma from the same W: P = sum n/(n+eps); squared variant: sum S/(S+eps)
    assert O.penalty_l2(n, O.gamma_update(n, eps)) == pytest.approx((n / (n + eps)).sum(), rel=1e-14)
    assert O.penalty_l2sq(s, O.alpha_update_sq(s, eps)) == pytest.approx((s / (s + eps)).sum(), rel=1e-14)
    # eps -> 0: both count the non-zero groups
    nonzero = int((n > 0).sum())
    assert nonzero == n.size - 1
    assert O.penalty_l2(n, O.gamma_update(n, 1e-30)) == pytest.approx(nonzero, rel=1e-12)
    assert O.penalty_l2sq(s, O.alpha_update_sq(s, 1e-300)) == pytest.approx(nonzero, rel=1e-12)
    # every norm equal to eps: each term is 1/2
    e = np.full((4, 5), 0.25)
    assert O.penalty_l2(e, O.gamma_update(e, 0.25)) == pytest.approx(e.size / 2)
    assert O.penalty_l2sq(e, O.alpha_update_sq(e, 0.25)) == pytest.approx(e.size / 2)


def test_plain_group_lasso_reduces_to_l1_for_unit_blocks():
    """gamma == 1 and 1x1 groups: the regulariser is the l1 norm of W."""
    w = rand_w(6, 16, 20)
    l1 = np.abs(si.bf16_bits_to_f32(w).astype(np.float64)).sum()
    for orient in ("C", "R"):
        assert O.penalty_l2(O.group_norms(w, 1, orient), None) == pytest.approx(l1, rel=1e-14)


def test_penalty_scaling_law_with_fixed_gamma():
    """With gamma held fixed (between milestones of Algorithm 2), P(cW) = |c| P(W); c = -4 is exact in bf16."""
    w = rand_w(7, 24, 24)
    w4 = si.f32_to_bf16_bits(si.bf16_bits_to_f32(w) * np.float32(-4.0))
    gam = O.gamma_update(O.group_norms(w, 3, "C"), 1e-3)
    p1 = O.penalty_l2(O.group_norms(w, 3, "C"), gam)
    p4 = O.penalty_l2(O.group_norms(w4, 3, "C"), gam)
    assert p4 == pytest.approx(4 * p1, rel=1e-14)


def test_stale_gamma_differs_from_fresh():
    w_old, w_new = rand_w(8, 16, 16), rand_w(9, 16, 16)
    n_new = O.group_norms(w_new, 4, "R")
    stale = O.gamma_update(O.group_norms(w_old, 4, "R"), 1e-3)
    want = sum(stale[i, a] * n_new[i, a] for i in range(16) for a in range(4))
    assert O.penalty_l2(n_new, stale) == pytest.approx(want, rel=1e-14)
    assert abs(O.penalty_l2(n_new, stale) - O.penalty_l2(n_new, O.gamma_update(n_new, 1e-3))) > 1e-3


@pytest.mark.parametrize("orient,block,squared", [("C", 3, False), ("R", 4, False), ("C", 2, True), ("R", 3, True)])
def test_penalty_gradient_against_finite_differences(orient, block, squared):
    """Central differences of the penalty value (gamma fixed) reproduce the analytic gradient."""
    g = si.stream(17, 3)
    w = g.standard_normal((6, 12)) * 0.5
    shape = (6 // block, 12) if orient == "C" else (6, 12 // block)
    gamma = g.uniform(0.5, 2.0, size=shape)

    def value(x):
        s = O.group_sumsq_values(x, block, orient)
        return O.penalty_l2sq(s, gamma) if squared else O.penalty_l2(np.sqrt(s), gamma)

    grad = O.penalty_grad_values(w, block, orient, gamma, squared)
    h = 1e-6
    for i, j in [(0, 0), (1, 5), (5, 11), (3, 7), (2, 2)]:
        e = np.zeros_like(w)
        e[i, j] = h
        fd = (value(w + e) - value(w - e)) / (2 * h)
        assert grad[i, j] == pytest.approx(fd, rel=1e-6, abs=1e-9)
    # closed forms: a group (3, 4) with gamma 2 -> 2 * (0.6, 0.8); an all-zero group -> 0
    wz = np.zeros((2, 2))
    wz[:, 0] = [3.0, 4.0]
    gz = O.penalty_grad_values(wz, 2, "C", np.array([[2.0, 5.0]]))
    assert np.allclose(gz, [[1.2, 0.0], [1.6, 0.0]], rtol=1e-15, atol=0)
    assert np.array_equal(O.penalty_grad_values(wz, 2, "C", np.array([[2.0, 5.0]]), squared=True), [[12.0, 0.0], [16.0, 0.0]])
    # Euler: <W, grad> = penalty for the norm form (degree-1 homogeneous), 2 * penalty for the squared form
    assert (w * grad).sum() == pytest.approx((2.0 if squared else 1.0) * value(w), rel=1e-12)


# ----------------------------------------------------------------------------- decision quantity
def test_decision_sumsq32_is_sequential_float32():
    """A case where summation order matters in float32: 1 + 2^-24 + 2^-24 taken left to right stays 1."""
    one, tiny = 1.0, 2.0 ** -12           # squares: 1 and 2^-24
    col = bits([[one], [tiny], [tiny]])
    assert O.decision_sumsq32(col, 3, "C")[0, 0] == np.float32(1.0)          # (1 + 2^-24) rounds to even = 1, twice
    col2 = bits([[tiny], [tiny], [one]])
    assert O.decision_sumsq32(col2, 3, "C")[0, 0] == np.float32(1.0 + 2.0 ** -23)
    row = bits([[one, tiny, tiny]])
    assert O.decision_sumsq32(row, 3, "R")[0, 0] == np.float32(1.0)


def test_decision_quantity_close_to_float64():
    w = rand_w(10, 96, 64)
    for orient, blk in [("C", 96), ("C", 16), ("R", 16)]:
        s32 = O.decision_sumsq32(w, blk, orient).astype(np.float64)
        s64 = O.group_sumsq(w, blk, orient)
        assert np.allclose(s32, s64, rtol=blk * 2.0 ** -24, atol=0)


# ----------------------------------------------------------------------------- prune / mask
def brute_force_row_groups(wf, k, t_b):
    """Algorithm 1's rule in plain Python floats on a list-of-lists matrix: a row segment of a strip
    survives iff its l2 norm is not <= t_b."""
    n = len(wf[0])
    h = n // k
    gone = {(j, c // h) for j, row in enumerate(wf) for c in range(0, n, h)
            if math.sqrt(math.fsum(v * v for v in row[c:c + h])) <= t_b}
    return [[0.0 if (j, c // h) in gone else v for c, v in enumerate(row)] for j, row in enumerate(wf)]


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_prune_against_brute_force_alg1(seed):
    # small integers / 8 are exact in bf16 and their squares sum exactly in float32 and float64,
    # so float32 and float64 decide identically and `<=` ties really occur
    g = si.stream(seed, 1)
    wf = g.integers(-3, 4, size=(6, 8)).astype(np.float32) / 8
    w = bits(wf)
    for k, t_b in [(2, 0.0), (2, 0.5), (4, 0.375), (8, 0.25), (1, 0.7), (2, math.sqrt(3) * 0.375)]:
        h = 8 // k
        want = np.array(brute_force_row_groups(wf.astype(float).tolist(), k, t_b), dtype=np.float32)
        got_loops = si.bf16_bits_to_f32(O.prune_groupwise(w, h, "R", t_b))
        got_vec = si.bf16_bits_to_f32(O.prune(w, h, "R", t_b))
        assert np.array_equal(got_loops, want), (k, t_b)
        assert np.array_equal(got_vec, want), (k, t_b)
        # column variant = row variant on the transpose
        got_c = si.bf16_bits_to_f32(O.prune(np.ascontiguousarray(w.T), h, "C", t_b)).T
        assert np.array_equal(got_c, want), (k, t_b)
        got_c_groups = si.bf16_bits_to_f32(O.prune_groupwise(np.ascontiguousarray(w.T), h, "C", t_b)).T
        assert np.array_equal(got_c_groups, want), (k, t_b)


def test_threshold_is_inclusive():
    """Algorithm 1 prunes at norm == t_b (`<=`), keeps just above."""
    w = bits([[3.0], [4.0]])                       # one group of norm exactly 5 (d=2, "C")
    assert not O.keep_flags(w, 2, "C", 5.0)[0, 0]
    assert O.keep_flags(w, 2, "C", 4.96875)[0, 0]  # largest bf16-exact float below 5 used as t_b
    assert O.prune(w, 2, "C", 5.0).tolist() == [[0], [0]]


def test_prune_limits_and_monotonicity():
    w = rand_w(14, 48, 32)
    n = O.group_norms(w, 12, "C")
    assert O.keep_flags(w, 12, "C", -1.0).all()                    # negative threshold: nothing goes
    assert not O.keep_flags(w, 12, "C", float(n.max()) * 1.01).any()  # above the largest norm: everything goes
    k_prev = O.keep_flags(w, 12, "C", 0.0)
    assert k_prev.all()                                            # generator emits no zero weights
    for t in np.quantile(n, [0.1, 0.3, 0.5, 0.9]):
        k = O.keep_flags(w, 12, "C", float(t))
        assert not (k & ~k_prev).any()                             # kept(t2) subset of kept(t1) for t1 < t2
        assert k.sum() < k_prev.sum()
        k_prev = k


def test_mask_equals_group_flags_at_zero_threshold():
    """Algorithm 2's Mask = (W != 0) on a pruned matrix, seen per group, equals keep(t_b = 0)."""
    spec = si.LinearSpec("m", 48, 40, False, 2.0, 12)
    wp, keep = si.make_pruned_weight(3, spec)
    m = O.mask_of(wp)
    assert np.array_equal(O.group_any(m, 12, "C"), keep)
    assert np.array_equal(O.keep_flags(wp, 12, "C", 0.0), keep)
    assert np.array_equal(O.prune(wp, 12, "C", 0.0), wp)           # pruning twice changes nothing
    # negative zero counts as zero
    assert not O.mask_of(np.array([[0x8000]], dtype=np.uint16))[0, 0]


# ----------------------------------------------------------------------------- percentile / top-k
def test_percentile_threshold_hits_the_rate():
    w = si.student_t_bf16(5, "t", (64, 96), 3.0, 0.02)
    for rate in (1.25, 1.79, 2.0, 5.0):
        t = O.percentile_threshold(w, 8, "C", rate)
        keep = O.keep_flags(w, 8, "C", t)
        g = keep.size
        r = math.floor(g * (1 - 1 / rate))
        assert g - keep.sum() >= r                                  # ties may remove a few more
        assert g - keep.sum() <= r + 2
        # exactly the r smallest norms are gone (no ties here)
        order = np.argsort(O.decision_sumsq32(w, 8, "C").ravel(), kind="stable")
        assert not keep.ravel()[order[:r]].any()
    assert O.percentile_threshold(w, 8, "C", 1.0) == -1.0


def test_topk_per_block_with_ties():
    # a 2x6 matrix, d=2: column sums of squares 4,1,4,0,1,4 -> keep 3 largest: columns 0,2,5; 4 -> + column 1 (lower index wins tie)
    wf = np.array([[2, 1, 2, 0, 1, 2], [0, 0, 0, 0, 0, 0]], dtype=np.float32)
    assert O.keep_topk_per_block(bits(wf), 2, "C", 3).tolist() == [[True, False, True, False, False, True]]
    assert O.keep_topk_per_block(bits(wf), 2, "C", 4).tolist() == [[True, True, True, False, False, True]]
    got_r = O.keep_topk_per_block(bits(wf.T), 2, "R", 4)           # strips are blocks, rows are groups
    assert got_r.shape == (6, 1) and got_r[:, 0].tolist() == [True, True, True, False, False, True]


# ----------------------------------------------------------------------------- pack
@pytest.mark.parametrize("orient,block", [("C", 3), ("C", 16), ("R", 12), ("R", 4)])
def test_pack_roundtrip_and_structure(orient, block):
    rows, cols = 48, 36
    spec = si.LinearSpec("p", rows, cols, False, 2.0, block)
    wp, keep = si.make_pruned_weight(21, spec, orient=orient)
    blk_ptr, idx, vals = O.pack(wp, keep, block, orient)
    n_blocks = rows // block if orient == "C" else cols // block
    limit = cols if orient == "C" else rows
    assert blk_ptr.dtype == np.int32 and idx.dtype == np.int32 and vals.dtype == np.uint16
    assert blk_ptr[0] == 0 and len(blk_ptr) == n_blocks + 1 and (np.diff(blk_ptr) >= 0).all()
    assert blk_ptr[-1] == keep.sum() and vals.size == block * keep.sum()
    for b in range(n_blocks):
        seg = idx[blk_ptr[b]:blk_ptr[b + 1]]
        assert (np.diff(seg) > 0).all() and (seg >= 0).all() and (seg < limit).all()
    back = O.unpack(blk_ptr, idx, vals, rows, cols, block, orient)
    assert np.array_equal(back, wp)                                  # bit for bit = W * Mask
    assert O.compression_rate(rows, cols, int(O.mask_of(back).sum())) == Fraction(rows * cols, block * int(keep.sum()))


def test_pack_tile_layout_by_hand():
    # 4x4, d=2, "C": block 0 keeps columns 1,3; block 1 keeps column 0
    wf = np.array([[0, 1, 0, 2], [0, 3, 0, 4], [5, 0, 0, 0], [6, 0, 0, 0]], dtype=np.float32)
    w = bits(wf)
    keep = np.array([[False, True, False, True], [True, False, False, False]])
    blk_ptr, idx, vals = O.pack(w, keep, 2, "C")
    assert blk_ptr.tolist() == [0, 2, 3] and idx.tolist() == [1, 3, 0]
    assert si.bf16_bits_to_f32(vals).tolist() == [1, 2, 3, 4, 5, 6]   # [d, kc] row-major tiles, block after block
    # "R" on the transpose: strips of 2 columns; tiles are [kc, h]
    blk_ptr, idx, vals = O.pack(np.ascontiguousarray(w.T), np.ascontiguousarray(keep.T), 2, "R")
    assert blk_ptr.tolist() == [0, 2, 3] and idx.tolist() == [1, 3, 0]
    assert si.bf16_bits_to_f32(vals).tolist() == [1, 3, 2, 4, 5, 6]
    # an empty block is legal
    blk_ptr, idx, vals = O.pack(w, np.zeros((2, 4), bool), 2, "C")
    assert blk_ptr.tolist() == [0, 0, 0] and idx.size == 0 and vals.size == 0


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, v = line.split()
                out[k] = v
    return out


def test_paper_storage_example():
    """Section 4.4: 8x8, 4x4 blocks, 50% sparsity, rows pruned inside blocks: COO 96 words, block structured 48."""
    g = read_golden("storage_example.txt")
    rows, cols, blk = int(g["rows"]), int(g["cols"]), int(g["block"])
    spec = si.LinearSpec("ex", rows, cols, False, 1 / (1 - float(g["sparsity"])), blk)
    wp, keep = si.make_pruned_weight(1, spec, orient="R")            # half of each strip's row segments go
    nnz = int(O.mask_of(wp).sum())
    assert nnz == rows * cols * (1 - float(g["sparsity"]))
    assert O.storage_words_coo(nnz) == int(g["coo_words"])
    assert O.storage_words_block_structured(nnz, keep.size) == int(g["bsp_words"])
    blk_ptr, idx, vals = O.pack(wp, keep, blk, "R")
    assert vals.size + idx.size + blk_ptr.size <= int(g["bsp_words"])  # our layout needs no more than the paper counts


def test_compression_rate_values_the_paper_prints():
    with open(os.path.join(GOLDEN, "compression_rates.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for key, printed in rows:
        if key == "bert_row_mean":
            mean = (8 * O.compression_rate(10, 10, 70) + O.compression_rate(10, 10, 50)) / 9
            assert round(float(mean), 2) == float(printed)
        else:
            kept = 100 - int(key)
            rate = O.compression_rate(10, 10, kept)
            assert rate == Fraction(100, kept)
            assert abs(float(rate) - float(printed)) < 1e-3 + 1e-12
    # half the 768 columns of every 16-row block of a 768x768 matrix: exactly 2
    assert O.compression_rate(768, 768, 48 * 16 * 384) == 2


# ----------------------------------------------------------------------------- linear
def test_gelu_values():
    xs = np.array([0.0, 1.0, -1.0, 0.5, 10.0, -10.0, 3.0])
    got = O.gelu(xs)
    want = [0.5 * x * (1 + math.erf(x / math.sqrt(2))) for x in xs]
    assert np.allclose(got, want, rtol=1e-15, atol=0)
    assert got[0] == 0.0
    assert got[1] == pytest.approx(0.8413447460685429, rel=1e-14)       # Phi(1)
    assert got[2] == pytest.approx(-0.15865525393145707, rel=1e-13)     # -Phi(-1)
    assert got[4] == pytest.approx(10.0, rel=1e-15) and abs(got[5]) < 1e-20


def triple_loop(xf, wf, mf, bf, act):
    T, K = xf.shape
    N = wf.shape[0]
    y = [[0.0] * N for _ in range(T)]
    for t in range(T):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                if mf[n][k]:
                    acc += float(xf[t][k]) * float(wf[n][k])
            acc += float(bf[n])
            y[t][n] = 0.5 * acc * (1 + math.erf(acc / math.sqrt(2))) if act else acc
    return np.array(y)


@pytest.mark.parametrize("act", [0, 1])
def test_linear_against_triple_loop_and_packed_form(act):
    T, N, K, d = 5, 12, 16, 3
    spec = si.LinearSpec("lin", N, K, bool(act), 2.0, d)
    wp, keep = si.make_pruned_weight(31, spec)
    w_full = si.make_weight(31, spec)                 # unpruned weights: the mask must do the pruning
    x = si.make_activations(31, "lin", T, K)
    b = si.make_bias(31, spec)
    mask = np.repeat(keep, d, axis=0)
    xf, wf, bf = (si.bf16_bits_to_f32(a).astype(np.float64) for a in (x, w_full, b))
    want = triple_loop(xf, wf, mask, bf, act)
    got = O.linear_masked_dense(x, w_full, mask, b, act)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)
    # same thing from the pruned matrix with its own mask, and from the packed form
    got2 = O.linear_masked_dense(x, wp, O.mask_of(wp), b, act)
    assert np.allclose(got2, want, rtol=1e-13, atol=1e-15)
    blk_ptr, idx, vals = O.pack(wp, keep, d, "C")
    got3 = O.linear_from_packed(x, blk_ptr, idx, vals, N, d, b, act)
    assert np.allclose(got3, want, rtol=1e-12, atol=1e-15)


def test_linear_special_cases():
    T, N, K, d = 7, 32, 24, 8
    spec = si.LinearSpec("sp", N, K, False, 2.0, d)
    w = si.make_weight(32, spec)
    x = si.make_activations(32, "sp", T, K)
    b = si.make_bias(32, spec)
    xf, wf, bf = (si.bf16_bits_to_f32(a).astype(np.float64) for a in (x, w, b))
    ones = np.ones((N, K), bool)
    # nothing pruned: a plain GEMM
    assert np.allclose(O.linear_masked_dense(x, w, ones, b, 0), xf @ wf.T + bf, rtol=1e-14, atol=1e-16)
    assert np.allclose(O.linear_masked_dense(x, w, ones, None, 0), np.einsum("tk,nk->tn", xf, wf), rtol=1e-13, atol=1e-16)
    # everything pruned: act(b) in every row
    y0 = O.linear_masked_dense(x, w, ~ones, b, 1)
    assert np.allclose(y0, np.tile(O.gelu(bf), (T, 1)), rtol=0, atol=0)
    blk_ptr, idx, vals = O.pack(w, np.zeros((N // d, K), bool), d, "C")
    assert np.array_equal(O.linear_from_packed(x, blk_ptr, idx, vals, N, d, b, 1), y0)
    # linearity in X without bias: doubling X (exact in bf16) doubles Y
    x2 = si.f32_to_bf16_bits(si.bf16_bits_to_f32(x) * np.float32(2))
    keep = si.random_keep_sets(1, "k", N // d, K, 12)
    m = np.repeat(keep, d, axis=0)
    assert np.array_equal(O.linear_masked_dense(x2, w, m, None, 0), 2 * O.linear_masked_dense(x, w, m, None, 0))
    # a pruned column of X has no influence on its row-block, a kept one does
    xm = x.copy()
    j = int(np.flatnonzero(~keep[0])[0])
    xm[:, j] = si.f32_to_bf16_bits(np.full(T, 100.0, np.float32))
    ya, yb = O.linear_masked_dense(x, w, m, b, 0), O.linear_masked_dense(xm, w, m, b, 0)
    assert np.array_equal(ya[:, :d], yb[:, :d])
    jk = int(np.flatnonzero(keep[0])[0])
    xm = x.copy()
    xm[:, jk] = si.f32_to_bf16_bits(np.full(T, 100.0, np.float32))
    assert not np.allclose(ya[:, :d], O.linear_masked_dense(xm, w, m, b, 0)[:, :d])


def test_row_scales():
    x = bits([[3.0, 4.0]])
    w = bits([[1.0, 0.0], [0.5, 0.5]])
    b = bits([0.25, -2.0])
    m = np.array([[True, True], [True, False]])
    s = O.row_scales(x, w, m, b)
    assert s.tolist() == [[5.0 * 1.0 + 0.25, 5.0 * 0.5 + 2.0]]


def test_backward_input_is_the_adjoint_of_the_forward_layer():
    """<dY, X W^T> == <dY W, X> for the masked weight: pins the backward product to the forward one."""
    T, N, K, d = 6, 12, 16, 4
    spec = si.LinearSpec("adj", N, K, False, 2.0, d)
    wp, keep = si.make_pruned_weight(41, spec)
    x = si.make_activations(41, "adj", T, K)
    dy = si.make_activations(42, "adj.dy", T, N)
    m = O.mask_of(wp)
    y = O.linear_masked_dense(x, wp, m, None, 0)
    dx = O.linear_backward_input(dy, wp, m)
    assert (O.bf16_to_f64(dy) * y).sum() == pytest.approx((dx * O.bf16_to_f64(x)).sum(), rel=1e-13)
    # a pruned column of a row-block passes no gradient from that block's outputs
    dy1 = np.zeros_like(dy)
    dy1[:, :d] = dy[:, :d]                      # only row-block 0's outputs carry gradient
    dx1 = O.linear_backward_input(dy1, wp, m)
    assert (dx1[:, ~keep[0]] == 0).all() and (dx1[:, keep[0]] != 0).any()


def test_backward_weight_is_the_adjoint_in_w():
    """<dY, X (V*M)^T> == <(dY^T X)*M, V> for any V: pins the weight gradient to the forward layer; and a
    brute-force entry."""
    T, N, K, d = 7, 8, 12, 4
    spec = si.LinearSpec("adjw", N, K, False, 2.0, d)
    wp, keep = si.make_pruned_weight(43, spec)
    v = si.make_weight(44, spec)                       # an arbitrary direction in weight space
    x = si.make_activations(43, "adjw", T, K)
    dy = si.make_activations(44, "adjw.dy", T, N)
    m = O.mask_of(wp)
    dw = O.linear_backward_weight(dy, x, m)
    lhs = (O.bf16_to_f64(dy) * O.linear_masked_dense(x, v, m, None, 0)).sum()
    assert lhs == pytest.approx((dw * O.bf16_to_f64(v)).sum(), rel=1e-13)
    assert (dw[~m] == 0).all()
    n, k = [int(a[0]) for a in np.nonzero(m)]
    brute = sum(float(O.bf16_to_f64(dy)[t, n]) * float(O.bf16_to_f64(x)[t, k]) for t in range(T))
    assert dw[n, k] == pytest.approx(brute, rel=1e-14)


# ---------------------------------------------------------------------------------------- Algorithm 2's retraining update
def _adam_scalar_loop(w, g_seq, lr, b1, b2, eps):
    """Adam as printed by Kingma & Ba (Algorithm 1), one scalar at a time, plain Python floats."""
    m = v = 0.0
    out = []
    for t, g in enumerate(g_seq, start=1):
        m = b1 * m + (1 - b1) * g
        v = b2 * v + (1 - b2) * g * g
        w = w - lr * (m / (1 - b1 ** t)) / (math.sqrt(v / (1 - b2 ** t)) + eps)
        out.append(w)
    return out


def test_adam_step_first_step_moves_by_lr_against_the_gradient_sign():
    """With zero moments the bias-corrected first step is lr * g / (|g| + eps): a step of (almost) lr."""
    w = np.array([[0.5, -0.25, 0.125, 1.0]])
    g = np.array([[3.0, -7.0, 1e-3, 0.0]])
    z = np.zeros_like(w)
    w1, m1, v1 = O.adam_step_masked(w, g, z, z, 1, 1e-2, 0.9, 0.999, 1e-8, 0.0, None)
    assert np.allclose(w1[0, :3], w[0, :3] - 1e-2 * np.sign(g[0, :3]), rtol=0, atol=1e-6)
    assert w1[0, 3] == 1.0                                    # zero gradient, no decay: unchanged
    assert np.allclose(m1, 0.1 * g) and np.allclose(v1, 0.001 * g * g)


def test_adam_step_constant_gradient_closed_form_and_scalar_loop():
    """A constant gradient gives mhat = g and vhat = g^2 at every step, so W_t = W_0 - t lr g / (|g| + eps);
    a changing gradient is checked against the published algorithm written as a scalar loop."""
    lr, b1, b2, eps = 3e-5, 0.9, 0.999, 1e-8
    w = np.array([[0.02, -0.01]])
    g = np.array([[0.3, -0.004]])
    m = v = np.zeros_like(w)
    for t in range(1, 8):
        w, m, v = O.adam_step_masked(w, g, m, v, t, lr, b1, b2, eps, 0.0, None)
    assert np.allclose(w, np.array([[0.02, -0.01]]) - 7 * lr * g / (np.abs(g) + eps), rtol=1e-12, atol=0)
    g_seq = [0.5, -0.2, 0.05, 0.9, -1.5]
    w = np.array([[0.1]])
    m = v = np.zeros((1, 1))
    for t, gt in enumerate(g_seq, start=1):
        w, m, v = O.adam_step_masked(w, np.array([[gt]]), m, v, t, 1e-3, b1, b2, eps, 0.0, None)
    assert w[0, 0] == pytest.approx(_adam_scalar_loop(0.1, g_seq, 1e-3, b1, b2, eps)[-1], rel=1e-13)


def test_adam_step_mask_and_decoupled_weight_decay():
    """W = W * Mask after the update: pruned weights are exactly zero, their moments still move; the
    decay term is lr * wd * W_old, independent of the gradient."""
    w = np.array([[0.5, -0.25], [0.125, 1.0]])
    g = np.array([[1.0, 2.0], [3.0, 4.0]])
    mask = np.array([[True, False], [False, True]])
    z = np.zeros_like(w)
    w1, m1, v1 = O.adam_step_masked(w, g, z, z, 1, 1e-2, 0.9, 0.999, 1e-8, 0.0, mask)
    assert w1[0, 1] == 0.0 and w1[1, 0] == 0.0 and w1[0, 0] != 0.0
    assert (m1 != 0).all() and (v1 != 0).all()
    wd0, _, _ = O.adam_step_masked(w, np.zeros_like(g), z, z, 1, 1e-2, 0.9, 0.999, 1e-8, 0.1, None)
    assert np.allclose(wd0, w * (1 - 1e-2 * 0.1), rtol=1e-15)


def test_repack_values_equals_pack_of_the_updated_matrix():
    """With the kept sets fixed, re-packing the values of an updated W gives what a fresh pack of
    W * Mask gives, and leaves the indices alone."""
    spec = si.LinearSpec("repack", 96, 80, False, 2.0, 12)
    wp, keep = si.make_pruned_weight(5, spec)
    blk_ptr, idx, vals = O.pack(wp, keep, 12, "C")
    w2 = si.zero_groups(si.make_weight(6, spec), keep, 12, "C")          # new values, same mask
    ptr2, idx2, vals2 = O.pack(w2, keep, 12, "C")
    assert np.array_equal(ptr2, blk_ptr) and np.array_equal(idx2, idx)
    assert np.array_equal(O.repack_values(w2, blk_ptr, idx, 12), vals2)
    assert np.array_equal(O.repack_values(wp, blk_ptr, idx, 12), vals)
