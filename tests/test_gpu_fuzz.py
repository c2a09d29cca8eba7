"""Seeded random sweep of block-table copies: shapes, image layouts (any nesting order of the
layer / plane / block dimensions, with and without padding), sub-ranges and variants, each
compared with the CPU oracle byte for byte.  Sec. 4.3 / App. C."""
import itertools

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import DevicePool, GuardedDevice, GuardedPinned, oshape

pytestmark = pytest.mark.gpu


def _random_layout(g, shape, n):
    """Nested strides in a random dimension order, optionally padded; returns (strides, size)."""
    C = shape.chunk_bytes
    ext = {"l": shape.num_layers, "p": shape.num_planes, "i": n}
    order = list(g.permutation(["l", "p", "i"]))             # innermost first
    pad_unit = 16 if C % 16 == 0 and g.uniform() < 0.7 else 1
    stride, span = {}, C
    for d in order:
        pad = int(g.integers(0, 4)) * pad_unit if g.uniform() < 0.5 else 0
        stride[d] = span + pad
        span = stride[d] * (ext[d] - 1) + span
    return (stride["l"], stride["p"], stride["i"]), span


@pytest.mark.parametrize("case", range(48))
def test_random_copy_cases(case):
    g = wl.rng(1000, case)
    shape = wl.KvShape(int(g.integers(1, 6)), int(g.choice([1, 2, 4])), int(g.choice([1, 2, 4, 16])),
                       int(g.choice([1, 3, 8, 64, 128])), elt_bytes=int(g.choice([1, 2, 4])),
                       num_planes=int(g.choice([1, 2])))
    nb = int(g.integers(4, 60))
    total = int(g.integers(1, nb // 2 + 1))
    first = int(g.integers(0, total))
    n = total - first
    planes = [g.integers(0, 256, size=nb * shape.chunk_bytes, dtype=np.uint8)
              for _ in range(shape.num_layers * shape.num_planes)]
    pool = DevicePool(shape, planes)
    src, dst = wl.disjoint_tables(g, nb, [total, total])
    strides, size = _random_layout(g, shape, n)
    variant = int(g.choice([tb.VARIANT_AUTO, tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE, tb.VARIANT_RUNS]))
    ctx = tb.Talaria(0, variant=variant, bounce_bytes=int(g.choice([1, 4])) << 20, dma_min_bytes=1 << 12)
    try:
        device_image = g.uniform() < 0.25
        want = np.full(size, 0x6B, np.uint8)
        if n:
            orc.kv_offload(oshape(shape), planes, src, first, n, want, strides)
        if device_image:
            img = GuardedDevice(size, np.full(size, 0x6B, np.uint8))
            hl = tb.host_layout(strides, size)
            ctx.kv_gather(pool.kv, src, first, n, img.ptr, hl)
            ctx.sync()
            assert np.array_equal(img.read(), want)
            ctx.kv_scatter(pool.kv, dst, first, n, img.ptr, hl)
        else:
            img = GuardedPinned(size, fill=0x6B)
            hl = tb.host_layout(strides, size)
            ctx.kv_offload(pool.kv, src, first, n, img.ptr, hl)
            ctx.sync()
            assert np.array_equal(img.np, want)
            if g.uniform() < 0.5 and n:
                ev = []
                import torch
                for _ in range(shape.num_layers):
                    e = torch.cuda.Event(); e.record(); ev.append(e)
                ctx.kv_restore_layered(pool.kv, dst, first, n, img.ptr, hl, ev)
            else:
                ctx.kv_restore(pool.kv, dst, first, n, img.ptr, hl)
        ctx.sync()
        if n:
            orc.kv_restore(oshape(shape), planes, dst, first, n, want, strides)
        for a, b in zip(pool.read(), planes):
            assert np.array_equal(a, b)
        assert pool.guards_ok() and img.guards_ok()
    finally:
        ctx.destroy()
