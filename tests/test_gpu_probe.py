"""The copy-mechanism probe moves bytes exactly, whichever mechanism it uses (128-bit, 256-bit,
TMA bulk), between HBM and device-mapped pinned host memory in both directions."""
import numpy as np
import pytest
import torch

from paper_2607_17181_b200 import binding as tb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mechanism", [0, 1, 2])
def test_probe_copies_are_exact(mechanism):
    ctx = tb.Talaria(0)
    try:
        n = 37 * 16384                                             # ragged against every grid used below
        gen = torch.Generator(device="cuda"); gen.manual_seed(5 + mechanism)
        src = torch.empty(n // 8, dtype=torch.int64, device="cuda").random_(generator=gen).view(torch.uint8)
        for ctas in (1, 3, 8, 40):
            dst = torch.zeros(n + 64, dtype=torch.uint8, device="cuda")
            ctx.probe_copy(mechanism, src, dst, n, ctas)
            ctx.sync()
            assert torch.equal(dst[:n], src) and not bool(dst[n:].any())
        host = torch.zeros(n + 64, dtype=torch.uint8, pin_memory=True)
        ctx.probe_copy(mechanism, src, host, n, 4)                  # device -> mapped host
        ctx.sync()
        assert torch.equal(host[:n], src.cpu()) and not bool(host[n:].any())
        back = torch.zeros(n, dtype=torch.uint8, device="cuda")
        ctx.probe_copy(mechanism, host, back, n, 4)                 # mapped host -> device
        ctx.sync()
        assert torch.equal(back, src)
        with pytest.raises(tb.TalariaError):
            ctx.probe_copy(mechanism, src, dst, 1000, 4)            # not a multiple of 16 KiB
        with pytest.raises(tb.TalariaError):
            ctx.probe_copy(3, src, dst, n, 4)
    finally:
        ctx.destroy()
