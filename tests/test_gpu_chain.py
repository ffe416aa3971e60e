"""bsp_linear_chain: an encoder layer's linears in one persistent launch.  Checked against the oracle
(per linear, on the bf16 input the GPU consumed) and bit for bit against bsp_linear_planned op by op."""
import numpy as np
import pytest
import torch

import paper_2009_08065_b200 as bsp
import synth_inputs as si
from oracle import bsp_oracle as O
from gpu_util import DEV, assert_linear_close, bits_of, to_dev

pytestmark = pytest.mark.gpu


def build_layer(seed, tokens, hidden, ffn, d, rate):
    """(ops, per-op host data) for QKV -> attention output (reads the V third) -> FFN-up + GELU -> FFN-down."""
    shapes = [("qkv", 3 * hidden, hidden, 0, -1, 0), ("attn_out", hidden, hidden, 0, 0, 2 * hidden),
              ("ffn_up", ffn, hidden, 1, 1, 0), ("ffn_down", hidden, ffn, 0, 2, 0)]
    ops, host = [], []
    for nm, n, k, act, src, col in shapes:
        spec = si.LinearSpec(f"chain.{nm}", n, k, bool(act), rate, d)
        wp, _ = si.make_pruned_weight(seed, spec)
        b = si.make_bias(seed, spec)
        pk = bsp.PackedMatrix.allocate(n, k, d, bsp.ORIENT_C, DEV)
        bsp.bsp_prune_pack(to_dev(wp), pk, 0.0)
        plan = torch.empty(bsp.bsp_linear_plan_bytes(n, k, d), dtype=torch.uint8, device=DEV)
        bsp.bsp_linear_plan(pk, plan)
        y = torch.full((tokens, n), 0x7FC0, dtype=torch.int16, device=DEV)
        ops.append(bsp.ChainOp(plan=plan, n_out=n, k_in=k, block=d, bias=to_dev(b), act=act, Y=y, src=src, src_col=col))
        host.append((spec, wp, b))
    return ops, host


def run_and_check(seed, tokens, hidden, ffn, d, rate, oracle_rows=None):
    ops, host = build_layer(seed, tokens, hidden, ffn, d, rate)
    x = to_dev(si.make_activations(seed, "chain_in", tokens, hidden))
    ws = torch.empty(bsp.bsp_linear_chain_ws_bytes(len(ops), tokens), dtype=torch.uint8, device=DEV)
    bsp.bsp_linear_chain(ops, x, ws)
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    rows = np.arange(tokens) if oracle_rows is None else oracle_rows
    sel = torch.from_numpy(rows).to(DEV)
    for op, (spec, wp, b) in zip(ops, host):
        src = x if op.src < 0 else ops[op.src].Y
        src = src[:, op.src_col: op.src_col + op.k_in]
        # bit-identical to the single-launch kernel on the same input
        y1 = torch.empty_like(op.Y)
        bsp.bsp_linear_planned(op.plan, op.n_out, op.k_in, op.block, src, op.bias, op.act, y1)
        bsp.bsp_linear_status()
        assert torch.equal(y1, op.Y), spec.name
        # and within tolerance of the oracle
        xs, ys = bits_of(src[sel].contiguous()), bits_of(op.Y[sel].contiguous())
        m = O.mask_of(wp)
        assert_linear_close(ys, O.linear_masked_dense(xs, wp, m, b, op.act), O.row_scales(xs, wp, m, b), spec.name)
    return ops


def test_chain_bert_base_layer_T4096():
    rows = np.sort(si.stream(5, 1).choice(4096, size=256, replace=False))
    run_and_check(si.DEFAULT_SEED, 4096, 768, 3072, 16, 3.0, rows)


@pytest.mark.parametrize("tokens,hidden,ffn,d", [(300, 128, 520, 8), (1, 64, 72, 8), (129, 264, 264, 12), (1000, 256, 1024, 32)])
def test_chain_ragged_shapes(tokens, hidden, ffn, d):
    """Token counts, widths and reduction sizes that are not multiples of the 128 x 256 x 64 tiles."""
    run_and_check(21, tokens, hidden, ffn, d, 2.0)


def test_chain_is_deterministic_and_reusable():
    ops, _ = build_layer(3, 2048, 768, 3072, 16, 3.0)
    x = to_dev(si.make_activations(3, "chain_in", 2048, 768))
    ws = torch.empty(bsp.bsp_linear_chain_ws_bytes(4, 2048), dtype=torch.uint8, device=DEV)
    arr = bsp.make_chain_array(ops)
    outs = []
    for _ in range(3):
        for op in ops:
            op.Y.fill_(0)
        bsp.bsp_linear_chain(arr, x, ws)
        bsp.bsp_linear_status()
        outs.append([op.Y.clone() for op in ops])
    for later in outs[1:]:
        for a, b in zip(outs[0], later):
            assert torch.equal(a, b)


def test_chain_argument_errors():
    ops, _ = build_layer(4, 64, 64, 128, 8, 2.0)
    x = to_dev(si.make_activations(4, "chain_in", 64, 64))
    ws = torch.empty(bsp.bsp_linear_chain_ws_bytes(4, 64), dtype=torch.uint8, device=DEV)
    bad = list(ops)
    bad[1] = bsp.ChainOp(**{**ops[1].__dict__, "src": 2})           # reads a later op
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_linear_chain(bad, x, ws)
    assert e.value.status == -1
    bad[1] = bsp.ChainOp(**{**ops[1].__dict__, "src_col": 160})     # 160 + 64 > 192 source columns
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_linear_chain(bad, x, ws)
    assert e.value.status == -2
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_linear_chain(ops, x, ws[:16])
    assert e.value.status == -3
