"""GPU parity of the pruned linear layer against the oracle's masked dense product (float64).

Tolerances (bf16 x bf16 products, float32 accumulation, bf16 output), see gpu_util:
max |err| / (||x|| ||w|| + |b|) <= 2e-2 and sum|err| / sum|ref| <= 5e-3.
"""
import numpy as np
import pytest
import torch

import paper_2009_08065_b200 as bsp
import synth_inputs as si
from oracle import bsp_oracle as O
from gpu_util import DEV, assert_linear_close, bits_of, to_dev, upload_packed

pytestmark = pytest.mark.gpu


def make_case(seed, name, T, N, K, d, rate, act, dist="normal"):
    spec = si.LinearSpec(name, N, K, bool(act), rate, d)
    wp, keep = si.make_pruned_weight(seed, spec, dist)
    x = si.make_activations(seed, name, T, K)
    b = si.make_bias(seed, spec)
    return spec, wp, keep, x, b


def oracle_linear(x, wp, b, act):
    m = O.mask_of(wp)
    return O.linear_masked_dense(x, wp, m, b, act), O.row_scales(x, wp, m, b)


def gpu_pack(wp, d):
    pk = bsp.PackedMatrix.allocate(wp.shape[0], wp.shape[1], d, bsp.ORIENT_C, DEV)
    bsp.bsp_prune_pack(to_dev(wp), pk, 0.0)
    return pk


def run_paths(pk, x, b, act, T, N, paths=("tc", "core")):
    out = {}
    xd = to_dev(x)
    bd = None if b is None else to_dev(b)
    for path in paths:
        y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)      # NaN pattern: every output must be written
        if path == "tc":
            ws = torch.empty(bsp.bsp_linear_plan_bytes(N, pk.cols, pk.block), dtype=torch.uint8, device=DEV)
            bsp.bsp_linear(pk, xd, bd, act, y, ws)
            bsp.bsp_linear_status()
        else:
            bsp.bsp_linear_cuda_core(pk, xd, bd, act, y)
        torch.cuda.synchronize()
        out[path] = bits_of(y)
    return out


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("d", [16, 3, 12, 96])
def test_single_layer_768_T128_rate2(d, act):
    spec, wp, keep, x, b = make_case(si.DEFAULT_SEED, "cfg1", 128, 768, 768, d, 2.0, act)
    y_ref, scales = oracle_linear(x, wp, b, act)
    pk = gpu_pack(wp, d)
    for path, y in run_paths(pk, x, b, act, 128, 768).items():
        assert_linear_close(y, y_ref, scales, f"{path} d={d} act={act}")


@pytest.mark.parametrize("T", [1, 3, 127, 129, 300])
def test_ragged_token_counts(T):
    spec, wp, keep, x, b = make_case(7, "ragT", T, 256, 192, 16, 2.0, 1)
    y_ref, scales = oracle_linear(x, wp, b, 1)
    pk = gpu_pack(wp, 16)
    for path, y in run_paths(pk, x, b, 1, T, 256).items():
        assert_linear_close(y, y_ref, scales, f"{path} T={T}")


@pytest.mark.parametrize("N,K,d", [(80, 72, 8), (200, 136, 8), (264, 8, 24), (96, 1000, 12), (520, 328, 8)])
def test_ragged_output_and_reduction_sizes(N, K, d):
    """Output and reduction sizes that are not multiples of the tile sizes."""
    spec, wp, keep, x, b = make_case(8, f"rag{N}x{K}", 150, N, K, d, 2.0, 0)
    y_ref, scales = oracle_linear(x, wp, b, 0)
    pk = gpu_pack(wp, d)
    for path, y in run_paths(pk, x, b, 0, 150, N).items():
        assert_linear_close(y, y_ref, scales, f"{path} N={N} K={K}")


def test_degenerate_blocks():
    """Row-blocks with no kept column give act(b); a matrix with nothing pruned is a plain GEMM."""
    T, N, K, d = 64, 128, 128, 16
    spec = si.LinearSpec("deg", N, K, True, 2.0, d)
    w = si.make_weight(9, spec)
    x = si.make_activations(9, "deg", T, K)
    b = si.make_bias(9, spec)
    keep = si.random_keep_sets(9, "deg.keep", N // d, K, 64)
    keep[0, :] = False
    keep[3, :] = False
    keep[5, :] = True
    wp = si.zero_groups(w, keep, d, "C")
    for act in (0, 1):
        y_ref, scales = oracle_linear(x, wp, b, act)
        pk = gpu_pack(wp, d)
        for path, y in run_paths(pk, x, b, act, T, N).items():
            assert_linear_close(y, y_ref, scales, f"{path} degenerate act={act}")
    # everything pruned, no bias: exact zeros
    pk = gpu_pack(np.zeros_like(wp), d)
    for path, y in run_paths(pk, x, None, 0, T, N).items():
        assert not (y & 0x7FFF).any(), path


def test_oracle_made_pack_feeds_the_gpu_linear():
    """The packed form is a contract: a pack made by the oracle drives the GPU layer as well."""
    spec, wp, keep, x, b = make_case(10, "opk", 96, 192, 256, 16, 3.0, 0)
    blk_ptr, idx, vals = O.pack(wp, keep, 16, "C")
    pk = upload_packed(blk_ptr, idx, vals, 192, 256, 16)
    y_ref, scales = oracle_linear(x, wp, b, 0)
    for path, y in run_paths(pk, x, b, 0, 96, 192).items():
        assert_linear_close(y, y_ref, scales, path)


def test_unaligned_inputs_take_the_cuda_core_path():
    spec, wp, keep, x, b = make_case(11, "una", 40, 64, 50, 16, 2.0, 1)     # K = 50 is not a multiple of 8
    y_ref, scales = oracle_linear(x, wp, b, 1)
    pk = gpu_pack(wp, 16)
    y = run_paths(pk, x, b, 1, 40, 64, paths=("tc",))["tc"]               # bsp_linear falls back by itself
    assert_linear_close(y, y_ref, scales, "fallback")


def test_bert_base_layer_T4096_rate3():
    """One encoder layer's four linears, chained; each is judged on the bf16 input the GPU consumed."""
    wl = si.bert_base_layer(4096, 3.0, 16)
    seed = si.DEFAULT_SEED
    acts = {"x": to_dev(si.make_activations(seed, "layer_in", wl.tokens, 768))}
    for spec in wl.linears:
        wp, keep = si.make_pruned_weight(seed, spec)
        b = si.make_bias(seed, spec)
        pk = gpu_pack(wp, spec.block)
        assert int(pk.kept_weights.item()) * 3 == spec.n_out * spec.k_in
        src = acts[spec.src]
        y = torch.empty((wl.tokens, spec.n_out), dtype=torch.int16, device=DEV)
        ws = torch.empty(bsp.bsp_linear_plan_bytes(spec.n_out, spec.k_in, spec.block), dtype=torch.uint8, device=DEV)
        bsp.bsp_linear(pk, src, to_dev(b), int(spec.gelu), y, ws)
        bsp.bsp_linear_status()
        short = spec.name.split(".")[1]
        acts[short] = y
        if short == "qkv":
            acts["qkv_v"] = y[:, 2 * 768:]                   # a strided view: ldx = 2304
        x_bits = bits_of(src.contiguous())
        y_ref, scales = oracle_linear(x_bits, wp, b, int(spec.gelu))
        assert_linear_close(bits_of(y), y_ref, scales, spec.name)


def test_tensor_core_path_is_deterministic():
    spec, wp, keep, x, b = make_case(12, "det", 512, 768, 768, 16, 3.0, 1)
    pk = gpu_pack(wp, 16)
    first = run_paths(pk, x, b, 1, 512, 768, paths=("tc",))["tc"]
    for _ in range(2):
        assert np.array_equal(run_paths(pk, x, b, 1, 512, 768, paths=("tc",))["tc"], first)


def test_plan_is_reusable():
    spec, wp, keep, x, b = make_case(13, "plan", 256, 384, 256, 32, 1.79, 0)
    pk = gpu_pack(wp, 32)
    plan = torch.empty(bsp.bsp_linear_plan_bytes(384, 256, 32), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_plan(pk, plan)
    y_ref, scales = oracle_linear(x, wp, b, 0)
    for _ in range(2):
        y = torch.empty((256, 384), dtype=torch.int16, device=DEV)
        bsp.bsp_linear_planned(plan, 384, 256, 32, to_dev(x), to_dev(b), 0, y)
        bsp.bsp_linear_status()
        assert_linear_close(bits_of(y), y_ref, scales, "planned")
    # the plan is W * Mask laid out densely
    assert np.array_equal(bits_of(plan.view(torch.int16)[: 384 * 256].reshape(384, 256)), wp)


@pytest.mark.parametrize("T,N,K,act", [(4096, 2304, 768, 0), (300, 520, 136, 1), (1, 256, 64, 0), (777, 768, 3072, 1)])
def test_cta_pair_kernel_matches_one_cta_kernel_and_oracle(T, N, K, act):
    """The two tensor-core variants (one CTA per 128 x BN tile, a CTA pair per 256 x 256 tile) agree bit for bit."""
    spec, wp, keep, x, b = make_case(14, f"pair{T}x{N}x{K}", T, N, K, 8, 2.0, act)
    pk = gpu_pack(wp, 8)
    plan = torch.empty(bsp.bsp_linear_plan_bytes(N, K, 8), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_plan(pk, plan)
    xd, bd = to_dev(x), to_dev(b)
    ys = []
    for algo in (bsp.LINEAR_ONE_CTA, bsp.LINEAR_CTA_PAIR):
        y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
        bsp.bsp_linear_planned_ex(plan, N, K, 8, xd, bd, act, y, algo)
        bsp.bsp_linear_status()
        ys.append(y)
    assert torch.equal(ys[0], ys[1])
    if T <= 1024:
        y_ref, scales = oracle_linear(x, wp, b, act)
        assert_linear_close(bits_of(ys[1]), y_ref, scales, "pair")


@pytest.mark.parametrize("h,rate", [(3, 2.0), (12, 1.428), (16, 5.0), (96, 2.0)])
def test_linear_on_row_pruned_strips(h, rate):
    """Algorithm 1's own geometry (orientation R): strips of h columns, row segments pruned by threshold.
    The packed form is expanded to the execution layout by bsp_linear_plan_r; the layer then matches the
    masked dense product."""
    T, N, K = 200, 384, 768
    spec = si.LinearSpec(f"rlin{h}", N, K, True, rate, h)
    w = si.make_weight(15, spec, "student_t3")
    b = si.make_bias(15, spec)
    x = si.make_activations(15, spec.name, T, K)
    t_b = O.percentile_threshold(w, h, "R", rate)
    wp = O.prune(w, h, "R", t_b)
    pk = bsp.PackedMatrix.allocate(N, K, h, bsp.ORIENT_R, DEV)
    bsp.bsp_prune_pack(to_dev(w), pk, t_b)
    plan = torch.full((bsp.bsp_linear_plan_bytes(N, K, 1),), 0x5A, dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_plan(pk, plan)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(plan.view(torch.int16)[: N * K].reshape(N, K)), wp)      # W * Mask, bit for bit
    y = torch.full((T, N), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_planned(plan, N, K, 1, to_dev(x), to_dev(b), 1, y)
    bsp.bsp_linear_status()
    y_ref, scales = oracle_linear(x, wp, b, 1)
    assert_linear_close(bits_of(y), y_ref, scales, f"orientation R, h={h}")


def test_backward_with_respect_to_activations():
    """dX = dY (W * Mask) through the transposed plan and the same tensor-core kernel."""
    T, N, K, d = 640, 768, 384, 16
    spec = si.LinearSpec("bwd", N, K, False, 3.0, d)
    wp, keep = si.make_pruned_weight(16, spec)
    dy = si.make_activations(16, "bwd.dy", T, N)
    pk = gpu_pack(wp, d)
    plan_t = torch.full((bsp.bsp_linear_plan_bytes(N, K, d),), 0x33, dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_plan_t(pk, plan_t)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(plan_t.view(torch.int16)[: N * K].reshape(K, N)), np.ascontiguousarray(wp.T))
    dx = torch.full((T, K), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_planned(plan_t, K, N, 1, to_dev(dy), None, 0, dx)
    bsp.bsp_linear_status()
    m = O.mask_of(wp)
    ref = O.linear_backward_input(dy, wp, m)
    # error scale: ||dY[t, :]|| * ||(W * Mask)[:, k]||
    scales = np.sqrt((O.bf16_to_f64(dy) ** 2).sum(1))[:, None] * np.sqrt(((O.bf16_to_f64(wp) * m) ** 2).sum(0))[None, :]
    assert_linear_close(bits_of(dx), ref, np.maximum(scales, 1e-30), "dX")


@pytest.mark.parametrize("T,N,K,d", [(4096, 768, 768, 16), (1000, 520, 264, 8), (130, 136, 72, 8), (50, 256, 3072, 32)])
def test_backward_with_respect_to_weights(T, N, K, d):
    """dW = (dY^T X) * Mask on the tensor cores (contraction over tokens, MN-major operand tiles)."""
    spec = si.LinearSpec(f"bww{T}", N, K, False, 2.0, d)
    wp, keep = si.make_pruned_weight(17, spec)
    x = si.make_activations(17, spec.name, T, K)
    dy = si.make_activations(18, spec.name + ".dy", T, N)
    keep_dev = torch.from_numpy(keep.astype(np.uint8)).to(DEV)
    dw = torch.full((N, K), 0x7FC0, dtype=torch.int16, device=DEV)
    bsp.bsp_linear_backward_weight(to_dev(dy), to_dev(x), d, keep_dev, dw)
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    m = O.mask_of(wp)
    ref = O.linear_backward_weight(dy, x, m)
    got = bits_of(dw)
    assert not (got[~m] & 0x7FFF).any()                                   # pruned positions carry no gradient
    scales = np.sqrt((O.bf16_to_f64(dy) ** 2).sum(0))[:, None] * np.sqrt((O.bf16_to_f64(x) ** 2).sum(0))[None, :]
    assert_linear_close(got, ref, np.maximum(scales, 1e-30), "dW")
    # without a mask: the plain product
    bsp.bsp_linear_backward_weight(to_dev(dy), to_dev(x), d, None, dw)
    bsp.bsp_linear_status()
    assert_linear_close(bits_of(dw), O.linear_backward_weight(dy, x, np.ones_like(m)), np.maximum(scales, 1e-30), "dW dense")
