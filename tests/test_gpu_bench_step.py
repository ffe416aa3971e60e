"""The benchmark's own step (its buffers, its call sequence, replayed from its CUDA graph) checked
against the oracle at the full size of the bench workload: norms / gamma / penalty within 1e-5,
flags / blk_ptr / indices / tiles / plan bit for bit, every linear within the GEMM tolerances on
the bf16 input the GPU consumed."""
import numpy as np
import pytest
import torch

import bench
import paper_2009_08065_b200 as bsp
import synth_inputs as si
from oracle import bsp_oracle as O
from gpu_util import assert_linear_close, bits_of, packed_to_host

pytestmark = pytest.mark.gpu


def test_bench_step_from_its_graph_matches_the_oracle():
    dev = torch.device("cuda", 0)
    wl = bench.workload()
    layer = bench.LayerOnDevice(wl, si.DEFAULT_SEED, 0, dev)
    layer.step()                                   # first call outside the graph (sets function attributes)
    for e in layer.lin:                            # make sure the replay, not the warm-up, produces the outputs
        e["Y"].fill_(0x7FC0)
        e["pk"].idx.fill_(-1)
        e["penalty"].fill_(-1.0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        layer.step()
    for _ in range(3):                             # every replay has to redo all of the work: wipe the outputs first
        for e in layer.lin:
            e["Y"].fill_(0x7FC0)
            e["norms"].fill_(-1.0)
            e["gamma"].fill_(-1.0)
            e["penalty"].fill_(-1.0)
            e["pk"].idx.fill_(-1)
            e["pk"].vals.fill_(0x7FC0)
            e["pk"].blk_ptr.fill_(-1)
            e["pk"].keep.fill_(7)
        graph.replay()
    bsp.bsp_linear_status()
    torch.cuda.synchronize()

    rows = np.sort(si.stream(9, 9).choice(wl.tokens, size=256, replace=False))
    sel = torch.from_numpy(rows).to(dev)
    outs = {}
    for e in layer.lin:
        spec = e["spec"]
        wp, keep = si.make_pruned_weight(si.DEFAULT_SEED, spec)
        b = si.make_bias(si.DEFAULT_SEED, spec)
        # weight side
        n_ref = O.group_norms(wp, spec.block, "C")
        g_ref = O.gamma_update(n_ref, bench.EPS)
        assert np.allclose(e["norms"].cpu().numpy(), n_ref, rtol=1e-5, atol=0)
        assert np.allclose(e["gamma"].cpu().numpy(), g_ref, rtol=1e-5, atol=0)
        assert float(e["penalty"].item()) == pytest.approx(O.penalty_l2(n_ref, g_ref), rel=1e-5)
        ref = O.pack(wp, O.keep_flags(wp, spec.block, "C", 0.0), spec.block, "C")
        blk_ptr, idx, vals, keep_gpu, kept = packed_to_host(e["pk"])
        assert np.array_equal(keep_gpu, keep) and np.array_equal(blk_ptr, ref[0])
        assert np.array_equal(idx, ref[1]) and np.array_equal(vals, ref[2])
        assert O.compression_rate(spec.n_out, spec.k_in, kept) == 3
        plan = bits_of(e["plan"].view(torch.int16)[: spec.n_out * spec.k_in].reshape(spec.n_out, spec.k_in))
        assert np.array_equal(plan, wp)
        # the linear, on the sampled token rows
        src = layer.source(spec, outs)
        xs, ys = bits_of(src[sel].contiguous()), bits_of(e["Y"][sel].contiguous())
        m = O.mask_of(wp)
        assert_linear_close(ys, O.linear_masked_dense(xs, wp, m, b, int(spec.gelu)), O.row_scales(xs, wp, m, b), spec.name)
        outs[spec.name.split(".")[1]] = e["Y"]
