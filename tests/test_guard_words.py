"""The guard zones that the GPU tests run under (tests/gpu_util.py) must themselves catch a stray write.
Checked here on CPU tensors: the allocator is told to treat every device as one it guards."""
import pytest
import torch

from gpu_util import GUARD_BYTES, GuardedAllocations


def guarded_on_cpu():
    g = GuardedAllocations()
    g._is_cuda = lambda device: device is not None
    return g


def test_guard_zones_pass_when_only_the_tensor_is_written():
    with guarded_on_cpu() as g:
        a = torch.empty((5, 7), dtype=torch.int16, device="cpu")
        b = torch.full((33,), 7, dtype=torch.float32, device="cpu")
        c = torch.zeros(3, 4, dtype=torch.float64, device="cpu")
        d = torch.empty_like(a)
        a.fill_(-1), b.fill_(1.0), c.fill_(2.0), d.fill_(3)
        assert a.data_ptr() % 2 == 0 and b.shape == (33,) and float(c.sum()) == 24.0
        assert g.check() == 4
    assert torch.empty is not None and torch.empty(2).shape == (2,)      # factories restored


@pytest.mark.parametrize("where", ["before", "after"])
def test_a_write_outside_the_tensor_is_caught(where):
    with guarded_on_cpu() as g:
        a = torch.empty((6,), dtype=torch.int16, device="cpu")
        raw, n, _ = g.live[0]
        if where == "before":
            raw[GUARD_BYTES - 1] = 0
        else:
            raw[GUARD_BYTES + n] = 0                 # first byte past the payload
        with pytest.raises(AssertionError, match=where):
            g.check()
