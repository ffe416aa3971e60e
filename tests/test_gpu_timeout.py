"""The bail-out path of the kernels' bounded waits, exercised without hanging or faulting anything: the wait limit
is lowered to a few milliseconds and a one-CTA self-test waits, through the helpers the tensor-core kernels use,
on a barrier and a counter that nothing signals.  The kernel must return by itself, report BSP_ERR_TIMEOUT once,
and leave the library usable."""
import numpy as np
import pytest
import torch

import paper_2009_08065_b200 as bsp
import synth_inputs as si
from gpu_util import DEV, to_dev, bits_of


@pytest.mark.gpu
def test_waits_run_out_at_the_limit_and_the_library_recovers():
    bsp.bsp_linear_status()                         # starts clean
    limit_ms = 5
    bsp.bsp_set_wait_limit_ms(limit_ms)
    try:
        expired, waited_ns = bsp.bsp_wait_selftest()
        assert expired == 2                          # the mbarrier wait and the counter wait
        assert limit_ms * 1e6 <= waited_ns < 100 * limit_ms * 1e6
        with pytest.raises(bsp.BspError) as e:
            bsp.bsp_linear_status()
        assert e.value.status == -5                  # BSP_ERR_TIMEOUT, reported once
        bsp.bsp_linear_status()                      # and cleared

        # the tensor-core kernel still runs (tensor memory was given back, the context is intact), here even
        # with the short limit in force, and agrees with the CUDA-core route
        spec = si.LinearSpec("after_timeout", 256, 512, True, 2.0, 16)
        wp, _ = si.make_pruned_weight(5, spec)
        x = si.make_activations(5, "after_timeout", 384, 512)
        pk = bsp.PackedMatrix.allocate(256, 512, 16, bsp.ORIENT_C, DEV)
        bsp.bsp_prune_pack(to_dev(wp), pk, 0.0)
        ws = torch.empty(bsp.bsp_linear_plan_bytes(256, 512, 16), dtype=torch.uint8, device=DEV)
        y = torch.full((384, 256), 0x7FC0, dtype=torch.int16, device=DEV)
        y2 = torch.full((384, 256), 0x7FC0, dtype=torch.int16, device=DEV)
        bsp.bsp_linear(pk, to_dev(x), None, bsp.ACT_NONE, y, ws)
        bsp.bsp_linear_cuda_core(pk, to_dev(x), None, bsp.ACT_NONE, y2)
        bsp.bsp_linear_status()
        a = si.bf16_bits_to_f32(bits_of(y)).astype(np.float64)
        b = si.bf16_bits_to_f32(bits_of(y2)).astype(np.float64)
        assert np.isfinite(a).all() and np.abs(a - b).max() <= 2.0 ** -7 * max(1.0, np.abs(b).max())
    finally:
        bsp.bsp_set_wait_limit_ms(2000)


def test_wait_limit_arguments():
    assert bsp.lib.bsp_set_wait_limit_ms(0) == -1
    assert bsp.lib.bsp_set_wait_limit_ms(10 ** 7) == -1
