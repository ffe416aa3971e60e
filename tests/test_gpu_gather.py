"""GPU parity of the gathering linear layer (bsp_linear_gathered: only the kept columns of X are fetched
and multiplied) and of bsp_transpose, against the oracle's masked dense product (float64).

Tolerances as for the other linear kernels (gpu_util): max |err| / (||x|| ||w|| + |b|) <= 2e-2 and
sum|err| / sum|ref| <= 5e-3; the transposed copy is bit-exact.
"""
import numpy as np
import pytest
import torch

import paper_2009_08065_b200 as bsp
import synth_inputs as si
from oracle import bsp_oracle as O
from gpu_util import DEV, assert_linear_close, bits_of, to_dev, upload_packed

pytestmark = pytest.mark.gpu


def oracle_linear(x, wp, b, act):
    m = O.mask_of(wp)
    return O.linear_masked_dense(x, wp, m, b, act), O.row_scales(x, wp, m, b)


def run_gathered(wp, d, x, b, act):
    """prune/pack on the GPU -> gather plan -> transposed activations -> bsp_linear_gathered."""
    N, K = wp.shape
    T = x.shape[0]
    pk = bsp.PackedMatrix.allocate(N, K, d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(to_dev(wp), pk, 0.0)
    gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, K, d), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_gather_plan(pk, gplan)
    xd = to_dev(x)
    xt = torch.full((K, T), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_transpose(xd, xt)
    y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)          # NaN pattern: every output must be written
    bsp.bsp_linear_gathered(gplan, N, K, d, xt, None if b is None else to_dev(b), act, y)
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    return bits_of(y), bits_of(xt)


@pytest.mark.parametrize("rows,cols", [(8, 8), (200, 72), (136, 320), (1024, 768)])
def test_transpose_is_bit_exact(rows, cols):
    x = si.make_activations(31, f"tr{rows}x{cols}", rows, cols)
    xt = torch.zeros((cols, rows), dtype=torch.int16, device=DEV)
    bsp.bsp_transpose(to_dev(x), xt)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(xt), np.ascontiguousarray(x.T))


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("d,rate", [(16, 2.0), (32, 3.0), (64, 5.0), (128, 8.0)])
def test_gathered_linear_fixed_keep_count(d, rate, act):
    """Several token tiles with a ragged last one, several row-blocks per run, kept counts that are not
    multiples of the 16-column step (K = 712: 356, 237, 142, 89 kept columns per block)."""
    T, N, K = 328, 512, 712
    spec = si.LinearSpec(f"gath{d}", N, K, bool(act), rate, d)
    wp, _ = si.make_pruned_weight(41, spec)
    x = si.make_activations(41, spec.name, T, K)
    b = si.make_bias(41, spec)
    y_ref, scales = oracle_linear(x, wp, b, act)
    y, xt = run_gathered(wp, d, x, b, act)
    assert np.array_equal(xt, np.ascontiguousarray(x.T))
    assert_linear_close(y, y_ref, scales, f"gathered d={d} rate={rate} act={act}")


def test_gathered_linear_uneven_blocks_and_empty_blocks():
    """Threshold pruning of heavy-tailed weights: every row-block keeps a different number of columns;
    two blocks keep nothing (their outputs are act(b)), one keeps everything, one keeps a single column."""
    T, N, K, d = 136, 384, 456, 32
    spec = si.LinearSpec("gath_uneven", N, K, True, 2.0, d)
    w = si.make_weight(43, spec, "student_t3")
    t_b = float(np.quantile(O.group_norms(w, d, "C"), 0.6))
    keep = O.keep_flags(w, d, "C", t_b)
    keep[1, :] = False
    keep[7, :] = False
    keep[4, :] = True
    keep[9, :] = False
    keep[9, 100] = True
    wp = si.zero_groups(w, keep, d, "C")
    x = si.make_activations(43, spec.name, T, K)
    b = si.make_bias(43, spec)
    for act in (0, 1):
        y_ref, scales = oracle_linear(x, wp, b, act)
        y, _ = run_gathered(wp, d, x, b, act)
        assert_linear_close(y, y_ref, scales, f"gathered uneven act={act}")
    # nothing kept at all and no bias: exact zeros
    y, _ = run_gathered(np.zeros_like(wp), d, x, None, 0)
    assert not (y & 0x7FFF).any()


def test_gathered_linear_oracle_made_pack_and_dense_route_agree():
    """The packed form is the contract: a pack made by the oracle drives the gather plan, and the result
    agrees with the zero-expanded dense route on the same inputs."""
    T, N, K, d = 256, 256, 512, 64
    spec = si.LinearSpec("gath_opk", N, K, False, 3.0, d)
    wp, keep = si.make_pruned_weight(44, spec)
    x = si.make_activations(44, spec.name, T, K)
    b = si.make_bias(44, spec)
    blk_ptr, idx, vals = O.pack(wp, keep, d, "C")
    pk = upload_packed(blk_ptr, idx, vals, N, K, d)
    gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, K, d), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_gather_plan(pk, gplan)
    xd, bd = to_dev(x), to_dev(b)
    xt = torch.empty((K, T), dtype=torch.int16, device=DEV)
    bsp.bsp_transpose(xd, xt)
    y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_gathered(gplan, N, K, d, xt, bd, 0, y)
    y2 = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    ws = torch.empty(bsp.bsp_linear_plan_bytes(N, K, d), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear(pk, xd, bd, 0, y2, ws)
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    y_ref, scales = oracle_linear(x, wp, b, 0)
    assert_linear_close(bits_of(y), y_ref, scales, "gathered, oracle pack")
    assert_linear_close(bits_of(y2), y_ref, scales, "dense route, oracle pack")


def test_gathered_linear_bert_large_shape_sampled_rows():
    """A sweep point of the BERT-large workload at full width (hidden 1024 -> 4096, 64-row blocks, 5x) with
    4096 tokens: many units per CTA, long runs of row-blocks; the oracle checks a sample of token rows."""
    T, N, K, d, rate = 4096, 4096, 1024, 64, 5.0
    spec = si.LinearSpec("gath_large", N, K, True, rate, d)
    wp, _ = si.make_pruned_weight(45, spec)
    x = si.make_activations(45, spec.name, T, K)
    b = si.make_bias(45, spec)
    y, _ = run_gathered(wp, d, x, b, 1)
    rows = np.sort(np.random.default_rng(45).choice(T, size=48, replace=False))
    y_ref, scales = oracle_linear(x[rows], wp, b, 1)
    assert_linear_close(y[rows], y_ref, scales, "gathered BERT-large FFN-up sample")
    assert np.isfinite(O.bf16_to_f64(y)).all()


def test_gelu_epilogue_is_tight_on_both_routes():
    """With an identity weight (one kept column per output row, value 1) and no bias the accumulator holds x
    itself, so the output is the epilogue's GELU of a bf16 number rounded to bf16: compared with the oracle's
    float64 erf form rounded the same way it may differ by one bf16 ulp (where the float32 evaluation lands on
    the other side of a rounding boundary) plus the 2.6e-6 the kernels' Phi allows in absolute terms, and
    matches bit for bit almost everywhere above 1e-3."""
    T, N, d = 512, 128, 16
    w = np.zeros((N, N), dtype=np.uint16)
    w[np.arange(N), np.arange(N)] = 0x3F80                      # 1.0
    grid = np.linspace(-8.0, 8.0, T * N).astype(np.float32)
    x = (np.ascontiguousarray(grid).view(np.uint32) >> 16).astype(np.uint16).reshape(T, N)   # truncation: still a bf16 grid
    ref = O.gelu(O.bf16_to_f64(x))
    ref_bits = (lambda u: ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16))(
        ref.astype(np.float32).view(np.uint32).astype(np.uint64))
    pk = bsp.PackedMatrix.allocate(N, N, d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(to_dev(w), pk, 0.0)
    xd = to_dev(x)
    outs = {}
    y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    ws = torch.empty(bsp.bsp_linear_plan_bytes(N, N, d), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear(pk, xd, None, 1, y, ws)
    outs["dense"] = y
    gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, N, d), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_gather_plan(pk, gplan)
    xt = torch.empty((N, T), dtype=torch.int16, device=DEV)
    bsp.bsp_transpose(xd, xt)
    y2 = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_gathered(gplan, N, N, d, xt, None, 1, y2)
    outs["gathered"] = y2
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    ref_r = O.bf16_to_f64(ref_bits)
    ulp_of_ref = np.abs(ref_r) * 2.0 ** -7                         # an upper bound of one bf16 ulp at that magnitude
    for name, t in outs.items():
        got_bits = bits_of(t)
        got = O.bf16_to_f64(got_bits)
        # the kernels evaluate Phi with an absolute error of at most 3.2e-7 (|x| <= 8 here), so x Phi(x) is
        # off by at most 2.6e-6 before rounding; on top of that one rounding boundary may be crossed
        assert (np.abs(got - ref_r) <= ulp_of_ref + 2.6e-6).all(), name
        big = np.abs(ref_r) > 1e-3                                  # where the absolute term is far below an ulp
        assert (got_bits[big] == ref_bits[big]).mean() > 0.99, (name, float((got_bits[big] == ref_bits[big]).mean()))


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("T,N,K,d", [(328, 512, 712, 32), (1000, 200, 256, 8), (4096, 768, 768, 16)])
def test_transposed_output_is_the_transpose_bit_for_bit(T, N, K, d, act):
    """BSP_LINEAR_OUT_TRANSPOSED on the zero-expanded route and out_transposed on the gathering kernel: YT [n_out, tokens]
    holds exactly the bits of Y^T (ragged token tiles and output tiles included), nothing outside it is written."""
    spec = si.LinearSpec(f"tr_out{T}_{N}_{d}", N, K, bool(act), 3.0, d)
    wp, _ = si.make_pruned_weight(43, spec)
    x = to_dev(si.make_activations(43, spec.name, T, K))
    b = to_dev(si.make_bias(43, spec))
    W = to_dev(wp)                                        # zero where pruned: its own execution layout
    y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    ld = (T + 7) // 8 * 8 + 8                             # a leading dimension wider than the tokens
    yt = torch.full((N, ld), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_planned_ex(W, N, K, d, x, b, act, y, bsp.LINEAR_ONE_CTA)
    bsp.bsp_linear_planned_ex(W, N, K, d, x, b, act, yt[:, :T], bsp.LINEAR_ONE_CTA | bsp.LINEAR_OUT_TRANSPOSED)
    bsp.bsp_linear_status()
    assert torch.equal(yt[:, :T], y.t())
    assert bool((yt[:, T:] == 0x7FC0).all())              # the padding columns keep their pattern
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_linear_planned_ex(W, N, K, d, x, b, act, yt[:, :T], bsp.LINEAR_CTA_PAIR | bsp.LINEAR_OUT_TRANSPOSED)
    assert e.value.status == -6
    if d in (16, 32) and T % 8 == 0:
        pk = bsp.PackedMatrix.allocate(N, K, d, bsp.ORIENT_C, DEV)
        bsp.bsp_prune_pack(W, pk, 0.0)
        gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, K, d), dtype=torch.uint8, device=DEV)
        bsp.bsp_linear_gather_plan(pk, gplan)
        xt = torch.empty((K, T), dtype=torch.int16, device=DEV)
        bsp.bsp_transpose(x, xt)
        yg = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
        ygt = torch.full((N, ld), 0x7FC0, dtype=torch.int16, device=DEV)
        bsp.bsp_linear_gathered(gplan, N, K, d, xt, b, act, yg)
        bsp.bsp_linear_gathered_ex(gplan, N, K, d, xt, b, act, ygt[:, :T], True)
        bsp.bsp_linear_status()
        assert torch.equal(ygt[:, :T], yg.t())
        assert bool((ygt[:, T:] == 0x7FC0).all())


def test_chain_hands_transposed_activations_on_without_a_transposing_pass():
    """Two layers with 64-row blocks at 8x: the first (zero-expanded route) writes its output transposed, the second
    (gathering kernel) reads that as its XT and writes transposed again; each layer is checked against the oracle on
    the bf16 input it consumed."""
    T, H, F, d, rate = 1024, 512, 1024, 64, 8.0
    s1 = si.LinearSpec("chain_t.up", F, H, True, rate, d)
    s2 = si.LinearSpec("chain_t.down", H, F, False, rate, d)
    w1, _ = si.make_pruned_weight(47, s1)
    w2, _ = si.make_pruned_weight(47, s2)
    b1, b2 = si.make_bias(47, s1), si.make_bias(47, s2)
    x = si.make_activations(47, "chain_t", T, H)
    h_t = torch.full((F, T), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_planned_ex(to_dev(w1), F, H, d, to_dev(x), to_dev(b1), 1, h_t, bsp.LINEAR_OUT_TRANSPOSED)
    pk = bsp.PackedMatrix.allocate(H, F, d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(to_dev(w2), pk, 0.0)
    gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(H, F, d), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_gather_plan(pk, gplan)
    y_t = torch.full((H, T), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_gathered_ex(gplan, H, F, d, h_t, to_dev(b2), 0, y_t, True)
    bsp.bsp_linear_status()
    h = np.ascontiguousarray(bits_of(h_t).T)
    ref1, sc1 = oracle_linear(x, w1, b1, 1)
    assert_linear_close(h, ref1, sc1, "first layer, transposed output")
    ref2, sc2 = oracle_linear(h, w2, b2, 0)
    assert_linear_close(np.ascontiguousarray(bits_of(y_t).T), ref2, sc2, "second layer, gathered from the transposed output")


def test_one_call_over_both_routes_run_and_tune():
    """bsp_linear_run takes the route it is told, or chooses one, and reports it; both routes and both output layouts
    give the bits of the per-route calls; bsp_linear_tune times the possible routes and names the faster."""
    T, N, K, d, rate = 2048, 512, 2048, 64, 8.0
    spec = si.LinearSpec("front_door", N, K, False, rate, d)
    wp, _ = si.make_pruned_weight(53, spec)
    x = to_dev(si.make_activations(53, spec.name, T, K))
    b = to_dev(si.make_bias(53, spec))
    W = to_dev(wp)
    pk = bsp.PackedMatrix.allocate(N, K, d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(W, pk, 0.0)
    gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, K, d), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_gather_plan(pk, gplan)
    xt = torch.empty((K, T), dtype=torch.int16, device=DEV)
    bsp.bsp_transpose(x, xt)
    kept = int(pk.kept_weights.item())
    ref_z = torch.empty((T, N), dtype=torch.int16, device=DEV)
    ref_g = torch.empty((T, N), dtype=torch.int16, device=DEV)
    bsp.bsp_linear_planned(W, N, K, d, x, b, 0, ref_z)
    bsp.bsp_linear_gathered(gplan, N, K, d, xt, b, 0, ref_g)
    for transposed in (False, True):
        for route, ref in ((bsp.ROUTE_ZERO_EXPANDED, ref_z), (bsp.ROUTE_GATHERED, ref_g)):
            out = torch.full((N, T) if transposed else (T, N), 0x7FC0, dtype=torch.int16, device=DEV)
            call = bsp.make_linear_call(N, K, d, T, plan=W, gplan=gplan, kept_weights=kept, X=x, XT=xt, bias=b,
                                        **({"YT": out} if transposed else {"Y": out}))
            assert bsp.bsp_linear_run(call, route) == route
            bsp.bsp_linear_status()
            assert torch.equal(out.t() if transposed else out, ref)
    y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    call = bsp.make_linear_call(N, K, d, T, plan=W, gplan=gplan, kept_weights=kept, X=x, XT=xt, bias=b, Y=y)
    taken = bsp.bsp_linear_run(call)                                   # automatic choice
    assert taken == bsp.bsp_linear_route(call) and taken in (bsp.ROUTE_ZERO_EXPANDED, bsp.ROUTE_GATHERED)
    bsp.bsp_linear_status()
    assert torch.equal(y, ref_z if taken == bsp.ROUTE_ZERO_EXPANDED else ref_g)
    best, ms_z, ms_g = bsp.bsp_linear_tune(call, 3)
    assert ms_z > 0 and ms_g > 0 and best == (bsp.ROUTE_GATHERED if ms_g < ms_z else bsp.ROUTE_ZERO_EXPANDED)
    only_z = bsp.make_linear_call(N, K, d, T, plan=W, kept_weights=kept, X=x, bias=b, Y=y)
    best, ms_z, ms_g = bsp.bsp_linear_tune(only_z, 2)
    assert best == bsp.ROUTE_ZERO_EXPANDED and ms_z > 0 and ms_g == -1.0
    with pytest.raises(bsp.BspError):
        bsp.bsp_linear_run(only_z, bsp.ROUTE_GATHERED)                 # that route's operands were not given
    bsp.bsp_linear_status()
