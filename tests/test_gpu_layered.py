"""GPU parity for the layer-ordered restore: same pool contents as the oracle's restore, and
each layer's event must not fire before that layer's K and V are in the pool (a consumer
stream snapshots the layer right after waiting on its event).  Sec. 4.3 restore; App. C
layer-first view."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import DevicePool, GuardedPinned, oshape

pytestmark = pytest.mark.gpu


def _events(n):
    ev = [torch.cuda.Event() for _ in range(n)]
    for e in ev:
        e.record()                       # creates the CUDA handle
    torch.cuda.synchronize()
    return ev


def _run(ctx, shape, nb, n, strides_fn, seed):
    g = wl.rng(700, seed)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    src, dst = wl.disjoint_tables(g, nb, [n, n])
    strides, size = strides_fn(shape, n)
    img = GuardedPinned(size, fill=0x3C)
    orc.kv_offload(oshape(shape), planes, src, 0, n, img.np, strides)          # a stored session image
    expect = [p.copy() for p in planes]
    orc.kv_restore(oshape(shape), expect, dst, 0, n, img.np, strides)
    ev = _events(shape.num_layers)
    consumer = torch.cuda.Stream()
    snaps = []
    torch.cuda.synchronize()
    ctx.kv_restore_layered(pool.kv, dst, 0, n, img.ptr, tb.host_layout(strides, img.n), ev)
    P = shape.num_planes
    with torch.cuda.stream(consumer):
        for l in range(shape.num_layers):
            consumer.wait_event(ev[l])
            snaps.append([pool.bufs[l * P + p].view().clone() for p in range(P)])
    ctx.sync()
    consumer.synchronize()
    for a, b in zip(pool.read(), expect):
        assert np.array_equal(a, b)
    for l in range(shape.num_layers):
        for p in range(P):
            assert np.array_equal(snaps[l][p].cpu().numpy(), expect[l * P + p]), (l, p)
    assert pool.guards_ok() and img.guards_ok()
    return ctx.get_counters()


def _dense(order):
    return lambda shape, n: (wl.dense_strides(shape, n, order), n * shape.bytes_per_block)


def _padded_pf(shape, n):
    C, L, P = shape.chunk_bytes, shape.num_layers, shape.num_planes
    return (P * C + 64, C, L * (P * C + 64) + 128), n * (L * (P * C + 64) + 128)


def _padded_lf(shape, n):
    C, L, P = shape.chunk_bytes, shape.num_layers, shape.num_planes
    return (P * (n * C + 256) + 512, n * C + 256, C), L * (P * (n * C + 256) + 512)


def _scattered(shape, n):          # neither planes nor blocks adjacent: falls back to one ordinary restore
    C, L, P = shape.chunk_bytes, shape.num_layers, shape.num_planes
    slot = C + 32
    return (P * slot, slot, L * P * slot), n * L * P * slot


@pytest.mark.parametrize("bounce", [2 << 20, 16 << 20])
@pytest.mark.parametrize("layout", [_dense("PF"), _dense("LF"), _padded_pf, _padded_lf, _scattered])
def test_layered_restore_matches_oracle_and_events_gate_layers(bounce, layout):
    # 16 KiB chunks; 40 blocks: a layer is 1.25 MiB, so a 1 MiB half splits layers and an 8 MiB half
    # carries six layers per piece
    ctx = tb.Talaria(0, variant=tb.VARIANT_BOUNCE, bounce_bytes=bounce)
    try:
        c = _run(ctx, wl.KvShape(7, 4, 16, 128), 128, 40, layout, 1)
        assert c.kernel_launches >= 1
        _run(ctx, wl.KvShape(3, 4, 16, 128, num_planes=1), 64, 9, layout, 2)      # single latent plane
        _run(ctx, wl.KvShape(2, 2, 16, 64), 64, 1, layout, 3)                     # one block
    finally:
        ctx.destroy()


def test_layered_restore_small_image_and_zero_copy_context_fall_back():
    for kwargs in ({}, {"variant": tb.VARIANT_ZEROCOPY}):
        ctx = tb.Talaria(0, **kwargs)
        try:
            _run(ctx, wl.TINY, 64, 19, _dense("PF"), 4)
            _run(ctx, wl.KvShape(3, 1, 4, 3), 40, 9, _dense("LF"), 5)            # 24-byte chunks: byte path
        finally:
            ctx.destroy()


def test_layered_restore_argument_errors():
    ctx = tb.Talaria(0)
    try:
        shape, nb = wl.TINY, 32
        pool = DevicePool(shape, wl.kv_pool(wl.rng(701), shape, nb))
        img = GuardedPinned(4 * shape.bytes_per_block)
        hl = tb.host_layout(wl.dense_strides(shape, 4, "PF"), img.n)
        ev = _events(shape.num_layers)
        for table, events, status in (([0, 1, 1, 2], ev, tb.ERR_DUP_BLOCK), ([0, 1, 2, 99], ev, tb.ERR_BAD_BLOCK_ID),
                                      ([0, 1, 2, 3], [0] * shape.num_layers, tb.ERR_INVALID_ARG)):
            with pytest.raises(tb.TalariaError) as e:
                ctx.kv_restore_layered(pool.kv, table, 0, 4, img.ptr, hl, events)
            assert e.value.status == status
        ctx.kv_restore_layered(pool.kv, [0, 1, 2, 3], 0, 0, img.ptr, hl, ev)      # zero blocks: events still fire
        ctx.sync()
        assert all(e.query() for e in ev)
    finally:
        ctx.destroy()
