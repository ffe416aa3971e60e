"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every function
include/bsp.h declares, answers its size queries, and rejects bad arguments before launching."""
import ctypes
import os
import re

import pytest

import paper_2009_08065_b200 as bsp
from paper_2009_08065_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bsp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bsp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported_and_bound():
    names = declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(bsp.lib, n), f"libbsp.so does not export {n}"
        assert n in binding.EXPORTED_SYMBOLS, f"binding has no signature for {n}"
    for n in binding.EXPORTED_SYMBOLS:
        assert n in names, f"{n} is bound but not declared in bsp.h"


def test_status_strings():
    assert bsp.bsp_status_string(0) == "BSP_OK"
    for code in range(-6, 0):
        assert bsp.bsp_status_string(code).startswith("BSP_ERR_")
    assert "unknown" in bsp.bsp_status_string(-99)


def test_pack_bound():
    idx, val, ws = bsp.bsp_pack_bound(768, 768, 16, bsp.ORIENT_C)
    assert idx == 48 * 768 and val == 768 * 768 and ws >= 48 * 768 * 5 and ws % 256 == 0
    idx, val, ws = bsp.bsp_pack_bound(768, 3072, 12, bsp.ORIENT_R)
    assert idx == 256 * 768 and val == 768 * 3072
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_pack_bound(770, 768, 16, bsp.ORIENT_C)
    assert e.value.status == -2
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_pack_bound(768, 768, 0, bsp.ORIENT_C)
    assert e.value.status == -1
    with pytest.raises(bsp.BspError):
        bsp.bsp_pack_bound(768, 768, 16, 7)
    # the part bsp_prune_pack itself touches: counts and one flag byte per group
    scratch = bsp.bsp_pack_scratch_bytes(768, 768, 16, bsp.ORIENT_C)
    assert 48 * 768 + 4 * 49 <= scratch < bsp.bsp_pack_bound(768, 768, 16, bsp.ORIENT_C)[2] and scratch % 256 == 0
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_pack_scratch_bytes(770, 768, 16, bsp.ORIENT_C)
    assert e.value.status == -2


def test_plan_bytes():
    assert bsp.bsp_linear_plan_bytes(768, 768, 16) == 768 * 768 * 2
    assert bsp.bsp_linear_plan_bytes(96, 72, 3) % 256 == 0
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_linear_plan_bytes(100, 64, 16)
    assert e.value.status == -2


def test_argument_errors_are_caught_before_any_launch():
    """Fake non-null pointers are safe here: each call must return before touching the device."""
    lib = bsp.lib
    p = ctypes.c_void_p(0x1000)
    # norms: block does not divide, null W, no outputs, bad enum, negative eps, ld too small
    assert lib.bsp_group_norms(p, 10, 8, 8, 3, 0, 1e-3, 0, p, None, None, None, None) == -2
    assert lib.bsp_group_norms(None, 8, 8, 8, 2, 0, 1e-3, 0, p, None, None, None, None) == -1
    assert lib.bsp_group_norms(p, 8, 8, 8, 2, 0, 1e-3, 0, None, None, None, None, None) == -1
    assert lib.bsp_group_norms(p, 8, 8, 8, 2, 5, 1e-3, 0, p, None, None, None, None) == -1
    assert lib.bsp_group_norms(p, 8, 8, 8, 2, 0, 1e-3, 9, p, None, None, None, None) == -1
    assert lib.bsp_group_norms(p, 8, 8, 8, 2, 0, -1.0, 0, p, None, None, None, None) == -1
    assert lib.bsp_group_norms(p, 8, 8, 4, 2, 0, 1e-3, 0, p, None, None, None, None) == -2
    assert lib.bsp_group_norms(p, 8, 9, 9, 2, 1, 1e-3, 0, p, None, None, None, None) == -2   # h does not divide cols
    # prune_pack: workspace too small, null outputs, misaligned workspace
    assert lib.bsp_prune_pack(p, 8, 8, 8, 2, 0, 0.0, None, -1, None, p, p, p, None, ctypes.c_void_p(0x1010), 1 << 20, None) == -1  # ws not 256-aligned
    ws = ctypes.c_void_p(0x10000)
    assert lib.bsp_prune_pack(p, 8, 8, 8, 2, 0, 0.0, None, -1, None, p, p, p, None, ws, 16, None) == -3
    assert lib.bsp_prune_pack(p, 8, 8, 8, 2, 0, 0.0, None, -1, None, None, p, p, None, ws, 1 << 20, None) == -1
    assert lib.bsp_prune_pack(p, 8, 8, 8, 3, 0, 0.0, None, -1, None, p, p, p, None, ws, 1 << 20, None) == -2
    assert lib.bsp_prune_pack(p, 16, 16384, 16384, 16, 0, 0.0, None, 4, None, p, p, p, None, ws, 1 << 30, None) == -6
    assert lib.bsp_percentile_threshold(p, 8, 8, 8, 2, 0, 0.5, p, ws, 1 << 20, None) == -1     # rate < 1
    assert lib.bsp_apply_mask(p, 8, 8, 8, 2, 0, None, None) == -1
    # linear: block does not divide n_out, bad act, ld too small, null X
    assert lib.bsp_linear_cuda_core(p, p, p, 10, 8, 4, p, 4, 8, None, 0, p, 16, None) == -2
    assert lib.bsp_linear_cuda_core(p, p, p, 8, 8, 4, p, 4, 8, None, 3, p, 8, None) == -1
    assert lib.bsp_linear_cuda_core(p, p, p, 8, 8, 4, p, 4, 4, None, 0, p, 8, None) == -2
    assert lib.bsp_linear_cuda_core(p, p, p, 8, 8, 4, None, 4, 8, None, 0, p, 8, None) == -1
    assert lib.bsp_linear(p, p, p, 10, 8, 4, p, 4, 8, None, 0, p, 16, ws, 1 << 20, None) == -2
    assert lib.bsp_linear_planned(ws, 8, 8, 4, p, 4, 8, None, 7, p, 8, None) == -1
    assert lib.bsp_linear_plan(p, p, p, 8, 8, 4, ws, 16, None) == -3
    # batched weight-side call: null / empty job list, bad enum
    assert lib.bsp_prepare_batched(None, 1, 16, 1e-3, 0, None) == -1
    job = binding._LayerJob()
    assert lib.bsp_prepare_batched(ctypes.pointer(job), 0, 16, 1e-3, 0, None) == -1
    assert lib.bsp_prepare_batched(ctypes.pointer(job), 1, 16, 1e-3, 5, None) == -1
    assert lib.bsp_prepare_batched(ctypes.pointer(job), 1, 16, 1e-3, 0, None) == -1      # W is NULL
    job.W, job.rows, job.cols, job.ldw = 0x1000, 40, 64, 64
    assert lib.bsp_prepare_batched(ctypes.pointer(job), 1, 16, 1e-3, 0, None) == -2      # 16 does not divide 40
    # penalty gradient, the other plans, the weight gradient, the chain: checked before any launch
    assert lib.bsp_penalty_grad(p, 8, 8, 8, 3, 0, 0, p, 1.0, p, 8, 0, None) == -2
    assert lib.bsp_penalty_grad(p, 8, 8, 8, 2, 0, 0, None, 1.0, p, 8, 0, None) == -1
    assert lib.bsp_penalty_grad(p, 8, 8, 8, 2, 0, 0, p, 1.0, p, 4, 0, None) == -2          # ldg < cols
    assert lib.bsp_linear_plan_r(p, p, p, 8, 9, 2, ws, 1 << 20, None) == -2                  # h does not divide k_in
    assert lib.bsp_linear_plan_r(p, p, p, 8, 8, 2, ws, 16, None) == -3
    assert lib.bsp_linear_plan_t(p, p, p, 10, 8, 4, ws, 1 << 20, None) == -2
    assert lib.bsp_linear_plan_t(None, p, p, 8, 8, 4, ws, 1 << 20, None) == -1
    assert lib.bsp_linear_backward_weight(p, 8, p, 8, 4, 10, 8, 4, None, p, 8, None) == -2  # block does not divide n_out
    assert lib.bsp_linear_backward_weight(p, 8, p, 8, 4, 8, 8, 4, None, None, 8, None) == -1
    assert lib.bsp_linear_backward_weight(p, 4, p, 8, 4, 8, 8, 4, None, p, 8, None) == -2   # ldy < n_out
    assert lib.bsp_linear_backward_weight(ctypes.c_void_p(0x1008), 8, p, 8, 4, 8, 8, 4, None, p, 8, None) == -6
    assert lib.bsp_linear_planned_ex(ws, 8, 8, 4, p, 4, 8, None, 0, p, 8, 9, None) == -1    # unknown variant
    n = ctypes.c_size_t()
    assert lib.bsp_linear_chain_ws_bytes(0, 128, ctypes.byref(n)) == -1
    assert lib.bsp_linear_chain_ws_bytes(9, 128, ctypes.byref(n)) == -1
    assert lib.bsp_linear_chain_ws_bytes(4, 4096, ctypes.byref(n)) == 0 and n.value == 768   # 4 x 32 counters and the ticket, rounded up to 256
    assert lib.bsp_linear_chain(None, 1, p, 4, 8, ws, 1 << 20, None) == -1
    # zero tokens is a valid no-op
    assert lib.bsp_linear_cuda_core(p, p, p, 8, 8, 4, p, 0, 8, None, 0, p, 8, None) == 0


def test_gather_entry_points_reject_bad_arguments_without_a_gpu():
    lib = bsp.lib
    p, ws = ctypes.c_void_p(0x10000), ctypes.c_void_p(0x20000)
    n = ctypes.c_size_t()
    assert lib.bsp_linear_gather_plan_bytes(4096, 1024, 64, ctypes.byref(n)) == 0
    # stage tables, two column arrays and one d x 64 tile per stage: above the weights themselves, below twice that
    assert 4096 * 1024 * 2 < n.value < 2 * 4096 * 1024 * 2 and n.value % 256 == 0
    assert bsp.bsp_linear_gather_plan_bytes(4096, 1024, 64) == n.value
    assert lib.bsp_linear_gather_plan_bytes(4096, 1024, 48, ctypes.byref(n)) == -2           # 48 does not divide 4096
    assert lib.bsp_linear_gather_plan_bytes(96, 1024, 48, ctypes.byref(n)) == -6             # block height not taken
    assert lib.bsp_linear_gather_plan_bytes(128, 40000, 64, ctypes.byref(n)) == -6           # columns do not fit int16
    assert lib.bsp_linear_gather_plan_bytes(128, 64, 64, None) == -1
    assert lib.bsp_linear_gather_plan(None, p, p, 128, 64, 64, ws, 1 << 20, None) == -1
    assert lib.bsp_linear_gather_plan(p, p, p, 128, 64, 64, ws, 16, None) == -3
    assert lib.bsp_linear_gather_plan(p, p, p, 128, 64, 64, ctypes.c_void_p(0x20010), 1 << 20, None) == -1
    assert lib.bsp_transpose(None, 8, 8, 8, p, 8, None) == -1
    assert lib.bsp_transpose(p, 8, 16, 8, ws, 8, None) == -2                                 # ldx < cols
    assert lib.bsp_transpose(p, 8, 12, 16, ws, 8, None) == -6                                # cols not a multiple of 8
    assert lib.bsp_transpose(p, 0, 8, 8, ws, 8, None) == 0
    assert lib.bsp_linear_gathered(None, 128, 64, 64, p, 8, 8, None, 0, p, 128, None) == -1
    assert lib.bsp_linear_gathered(ws, 128, 64, 64, p, 8, 8, None, 7, p, 128, None) == -1    # unknown activation
    assert lib.bsp_linear_gathered(ws, 100, 64, 64, p, 8, 8, None, 0, p, 128, None) == -2
    assert lib.bsp_linear_gathered(ws, 128, 64, 64, p, 16, 8, None, 0, p, 128, None) == -2   # ldxt < tokens
    assert lib.bsp_linear_gathered(ws, 128, 64, 24, p, 8, 8, None, 0, p, 128, None) == -2    # 24 does not divide 128
    assert lib.bsp_linear_gathered(ws, 96, 64, 48, p, 8, 8, None, 0, p, 96, None) == -6      # block height not taken
    assert lib.bsp_linear_gathered(ws, 128, 64, 64, p, 12, 16, None, 0, p, 128, None) == -6  # tokens not a multiple of 8
    assert lib.bsp_linear_gathered(ws, 128, 64, 64, p, 0, 8, None, 0, p, 128, None) == 0     # zero tokens: no-op


def test_retraining_entry_points_reject_bad_arguments_without_a_gpu():
    lib = bsp.lib
    p = ctypes.c_void_p(0x10000)
    args = lambda **kw: [kw.get("W", p), p, p, p, kw.get("rows", 8), kw.get("cols", 8), kw.get("ldw", 8), 8,      # noqa: E731
                         kw.get("keep", None), kw.get("block", 4), 0, 1e-3, kw.get("beta1", 0.9), 0.999, 1e-8, 0.0,
                         kw.get("step", 1), None, 0, None]
    assert lib.bsp_masked_adam_step(*args(W=None)) == -1
    assert lib.bsp_masked_adam_step(*args(step=0)) == -1
    assert lib.bsp_masked_adam_step(*args(beta1=1.0)) == -1
    assert lib.bsp_masked_adam_step(*args(ldw=4)) == -2
    assert lib.bsp_masked_adam_step(*args(keep=p, block=3)) == -2                            # 3 does not divide 8
    assert lib.bsp_masked_adam_step(*args(cols=6, ldw=8)) == -6                              # cols not a multiple of 4
    assert lib.bsp_repack_values(p, 8, 8, 8, 4, None, p, p, None) == -1
    assert lib.bsp_dense_mask(p, 8, 8, 8, None, 8, None) == -1
    assert lib.bsp_dense_mask(p, 8, 8, 4, p, 8, None) == -2
    assert lib.bsp_repack_values(p, 8, 8, 8, 3, p, p, p, None) == -2


def test_product_code_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2009_08065_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f"{f} mentions the oracle"
    assert "paper_2009_08065_b200" not in open(os.path.join(ROOT, "oracle", "bsp_oracle.py")).read()


def _fake_call(n, k, d, c, tokens=32768, act=0, z=True, g=True):
    p = ctypes.c_void_p(0x1000).value
    call = binding._LinearCall()
    call.plan, call.gplan = (p if z else None), (p if g else None)
    call.kept_weights = int(round(k / c)) * n
    call.n_out, call.k_in, call.block, call.tokens = n, k, d, tokens
    call.X, call.ldx, call.XT, call.ldxt = (p if z else None), k, (p if g else None), tokens
    call.act = act
    call.Y, call.ldy = p, n
    return call


def test_route_choice_follows_the_measured_crossovers():
    """bsp_linear_route is host-only: with both routes possible it takes the gathering kernel where it was measured
    to win on B200 (64-row blocks at 8x on the FFN shapes) and the zero-expanded route elsewhere."""
    lib = bsp.lib
    assert bsp.bsp_linear_route(_fake_call(1024, 4096, 64, 8.0)) == bsp.ROUTE_GATHERED             # FFN-down
    assert bsp.bsp_linear_route(_fake_call(4096, 1024, 64, 8.0, act=1)) == bsp.ROUTE_GATHERED      # FFN-up + GELU
    assert bsp.bsp_linear_route(_fake_call(3072, 1024, 64, 8.0)) == bsp.ROUTE_ZERO_EXPANDED        # QKV
    assert bsp.bsp_linear_route(_fake_call(1024, 4096, 64, 5.0)) == bsp.ROUTE_ZERO_EXPANDED
    assert bsp.bsp_linear_route(_fake_call(1024, 4096, 32, 8.0)) == bsp.ROUTE_ZERO_EXPANDED
    assert bsp.bsp_linear_route(_fake_call(2304, 768, 16, 3.0, tokens=4096)) == bsp.ROUTE_ZERO_EXPANDED
    # only one route possible: that one, whatever the estimate says
    assert bsp.bsp_linear_route(_fake_call(2304, 768, 16, 3.0, z=False)) == bsp.ROUTE_GATHERED
    assert bsp.bsp_linear_route(_fake_call(1024, 4096, 64, 8.0, g=False)) == bsp.ROUTE_ZERO_EXPANDED
    assert bsp.bsp_linear_route(_fake_call(1024, 4096, 8, 8.0)) == bsp.ROUTE_ZERO_EXPANDED         # block 8: no gathering kernel
    bad = _fake_call(1024, 4096, 64, 8.0)
    bad.YT, bad.ldyt = bad.Y, 32768                                                                # both outputs
    assert lib.bsp_linear_route(ctypes.byref(bad), ctypes.byref(ctypes.c_int())) == -1
    none = _fake_call(1024, 4096, 64, 8.0)
    none.X = None                                                                                  # plan without X, gplan with XT
    assert bsp.bsp_linear_route(none) == bsp.ROUTE_GATHERED
    none.XT = None
    assert lib.bsp_linear_route(ctypes.byref(none), ctypes.byref(ctypes.c_int())) == -1
    assert lib.bsp_linear_run(ctypes.byref(_fake_call(1024, 4096, 64, 8.0)), 7, None, None) == -1
