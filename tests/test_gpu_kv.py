"""GPU parity: block-table copies through the C ABI against the CPU oracle, byte
for byte (tolerance 0).  Sec. 4.3 checkpoint / restore, App. C LF / PF layouts."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import DevicePool, GuardedDevice, GuardedPinned, oshape

pytestmark = pytest.mark.gpu

VARIANTS = [tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE, tb.VARIANT_RUNS, tb.VARIANT_AUTO]


@pytest.fixture(scope="module")
def ctxs():
    # a 2 MiB bounce buffer makes the bounce variant run many double-buffered pieces
    out = {v: tb.Talaria(0, variant=v, bounce_bytes=2 << 20, dma_min_bytes=1 << 20) for v in VARIANTS}
    yield out
    for c in out.values():
        c.destroy()


def _roundtrip(ctx, shape, num_blocks, sizes, order, config_id):
    g = wl.rng(config_id)
    planes = wl.kv_pool(g, shape, num_blocks)
    pool = DevicePool(shape, planes)
    tables = wl.disjoint_tables(g, num_blocks, sizes)
    used = np.concatenate(tables)
    new_tables = wl.disjoint_tables(g, num_blocks, sizes, exclude=used)
    expect = [p.copy() for p in planes]
    for bt, bt2 in zip(tables, new_tables):
        n = bt.size
        strides = wl.dense_strides(shape, n, order)
        img = GuardedPinned(n * shape.bytes_per_block)
        hl = tb.host_layout(strides, img.n)
        ctx.kv_offload(pool.kv, bt, 0, n, img.ptr, hl)
        ctx.sync()
        want = np.zeros(img.n, np.uint8)
        orc.kv_offload(oshape(shape), expect, bt, 0, n, want, strides)
        assert np.array_equal(img.np, want)
        assert img.guards_ok()
        ctx.kv_restore(pool.kv, bt2, 0, n, img.ptr, hl)
        ctx.sync()
        orc.kv_restore(oshape(shape), expect, bt2, 0, n, want, strides)
        got = pool.read()
        for a, b in zip(got, expect):
            assert np.array_equal(a, b)
        assert pool.guards_ok()
    c = ctx.get_counters()
    assert c.kernel_launches + c.memcpy_calls > 0


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("order", ["LF", "PF"])
def test_config1_tiny_offload_restore(ctxs, variant, order):
    # 4 layers, 2 KV heads, head_dim 64, 16-token blocks; sessions of 300 and 500 tokens
    _roundtrip(ctxs[variant], wl.TINY, 256, [wl.TINY.blocks_for(300), wl.TINY.blocks_for(500)], order, 1)


@pytest.mark.parametrize("variant", [tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE])
@pytest.mark.parametrize("order", ["LF", "PF"])
def test_qwen_chunk_size_several_tiles_and_ragged_tail(ctxs, variant, order):
    # 16 KiB chunks (4 KV heads x 16 tokens x 128 x bf16), 3 layers, 37 + 5 blocks: pieces and
    # warps end mid-image
    shape = wl.KvShape(3, 4, 16, 128)
    _roundtrip(ctxs[variant], shape, 128, [37, 5, 1], order, 11)


@pytest.mark.parametrize("shape", [wl.KvShape(3, 1, 4, 3), wl.KvShape(2, 3, 5, 6, elt_bytes=1, num_planes=1),
                                   wl.KvShape(2, 1, 1, 8, elt_bytes=2), wl.KvShape(1, 2, 3, 40, elt_bytes=2)])
@pytest.mark.parametrize("variant", [tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE, tb.VARIANT_RUNS])
def test_odd_shapes(ctxs, shape, variant):
    # chunk sizes 24, 90, 16 and 480 bytes: the byte path, a single plane, tiny vector chunks
    _roundtrip(ctxs[variant], shape, 40, [9, 4], "PF", 12)
    _roundtrip(ctxs[variant], shape, 40, [9, 4], "LF", 13)


@pytest.mark.parametrize("variant", [tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE, tb.VARIANT_RUNS])
def test_sub_range_padded_strides_and_duplicates_on_offload(ctxs, variant):
    ctx = ctxs[variant]
    shape, nb = wl.KvShape(3, 2, 4, 16), 50
    g = wl.rng(14)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    bt = wl.disjoint_tables(g, nb, [24])[0]
    bt[7] = bt[3]                                         # duplicates are legal when only reading
    C, L, P = shape.chunk_bytes, shape.num_layers, shape.num_planes
    first, n = 5, 11
    slot = C + 48
    strides = (P * slot, slot, L * P * slot)
    img = GuardedPinned(n * L * P * slot, fill=0x11)
    ctx.kv_offload(pool.kv, bt, first, n, img.ptr, tb.host_layout(strides, img.n))
    ctx.sync()
    want = np.full(img.n, 0x11, np.uint8)
    orc.kv_offload(oshape(shape), planes, bt, first, n, want, strides)
    assert np.array_equal(img.np, want) and img.guards_ok()


def test_gather_scatter_device_image(ctxs):
    ctx = ctxs[tb.VARIANT_AUTO]
    shape, nb = wl.KvShape(5, 4, 16, 128), 96
    g = wl.rng(15)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    bt, bt2 = wl.disjoint_tables(g, nb, [33, 33])
    for order in ("LF", "PF"):
        strides = wl.dense_strides(shape, 33, order)
        dimg = GuardedDevice(33 * shape.bytes_per_block, np.zeros(33 * shape.bytes_per_block, np.uint8))
        il = tb.host_layout(strides, dimg.n)
        ctx.kv_gather(pool.kv, bt, 0, 33, dimg.ptr, il)
        ctx.sync()
        want = np.zeros(dimg.n, np.uint8)
        orc.kv_offload(oshape(shape), planes, bt, 0, 33, want, strides)
        assert np.array_equal(dimg.read(), want) and dimg.guards_ok()
        ctx.kv_scatter(pool.kv, bt2, 0, 33, dimg.ptr, il)
        ctx.sync()
        orc.kv_restore(oshape(shape), planes, bt2, 0, 33, want, strides)
        for a, b in zip(pool.read(), planes):
            assert np.array_equal(a, b)
        bt, bt2 = bt2, bt
    assert pool.guards_ok()


def test_registered_host_memory_and_batch_forms(ctxs):
    ctx = ctxs[tb.VARIANT_ZEROCOPY]
    shape, nb = wl.TINY, 128
    g = wl.rng(16)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    sizes = [7, 19, 1, 12]
    tables = wl.disjoint_tables(g, nb, sizes)
    new_tables = wl.disjoint_tables(g, nb, sizes, exclude=np.concatenate(tables))
    raw = np.zeros(sum(sizes) * shape.bytes_per_block + 4096, np.uint8)   # ordinary numpy memory
    ctx.host_register(raw)
    try:
        xfers, at, imgs = [], 0, []
        for k, bt in enumerate(tables):
            n = bt.size
            strides = wl.dense_strides(shape, n, "PF" if k % 2 else "LF")
            view = raw[at:at + n * shape.bytes_per_block]
            imgs.append((view, strides))
            xfers.append((bt, 0, n, view, tb.host_layout(strides, view.size)))
            at += view.size
        ctx.kv_offload_batch(pool.kv, xfers)
        ctx.sync()
        for (view, strides), bt in zip(imgs, tables):
            want = np.zeros(view.size, np.uint8)
            orc.kv_offload(oshape(shape), planes, bt, 0, bt.size, want, strides)
            assert np.array_equal(view, want)
        ctx.kv_restore_batch(pool.kv, [(bt2, 0, bt2.size, view, x[4]) for bt2, (view, _), x in zip(new_tables, imgs, xfers)])
        ctx.sync()
        for (view, strides), bt2 in zip(imgs, new_tables):
            orc.kv_restore(oshape(shape), planes, bt2, 0, bt2.size, view, strides)
        for a, b in zip(pool.read(), planes):
            assert np.array_equal(a, b)
        # two sessions that claim the same new block are rejected before anything runs
        clash = [(new_tables[0], 0, 7, imgs[0][0], xfers[0][4]), (new_tables[0], 0, 7, imgs[0][0], xfers[0][4])]
        with pytest.raises(tb.TalariaError) as e:
            ctx.kv_restore_batch(pool.kv, clash)
        assert e.value.status == tb.ERR_DUP_BLOCK
    finally:
        ctx.sync()
        ctx.host_unregister(raw)


@pytest.mark.parametrize("order", ["PF", "LF"])
def test_batch_of_many_small_sessions_is_one_fused_launch(ctxs, order):
    ctx = ctxs[tb.VARIANT_AUTO]
    shape, nb = wl.TINY, 1536
    g = wl.rng(18)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    expect = [p.copy() for p in planes]
    for sizes in ([1] * 64, [3] * 40 + [1] * 50, [5, 1, 9, 2, 30, 1, 1, 7] * 10):     # <= 256 blocks inline, then beyond
        tables = wl.disjoint_tables(g, nb, sizes)
        new_tables = wl.disjoint_tables(g, nb, sizes, exclude=np.concatenate(tables))[::-1]
        imgs = [GuardedPinned(n * shape.bytes_per_block) for n in sizes]
        xf = [(bt, 0, bt.size, im.ptr, tb.host_layout(wl.dense_strides(shape, bt.size, order), im.n))
              for bt, im in zip(tables, imgs)]
        ctx.reset_counters()
        ctx.kv_offload_batch(pool.kv, xf)
        ctx.sync()
        c = ctx.get_counters()
        # page-first images all share their layer / plane strides; layer-first ones only at equal block counts
        per_group = [sum(sizes)] if order == "PF" else [sum(n for n in sizes if n == k) for k in set(sizes)]
        groups = len(per_group)
        assert c.kernel_launches == groups, (order, sizes[:4], c.kernel_launches)
        assert c.memcpy_calls == sum(1 for b in per_group if b > 256)               # up to 256 blocks: no upload
        for bt, im in zip(tables, imgs):
            want = np.zeros(im.n, np.uint8)
            orc.kv_offload(oshape(shape), expect, bt, 0, bt.size, want, wl.dense_strides(shape, bt.size, order))
            assert np.array_equal(im.np, want) and im.guards_ok()
        ctx.reset_counters()
        ctx.kv_restore_batch(pool.kv, [(bt2, 0, bt2.size, im.ptr, x[4]) for bt2, im, x in zip(new_tables[::-1], imgs, xf)])
        ctx.sync()
        assert ctx.get_counters().kernel_launches == groups
        for bt2, im in zip(new_tables[::-1], imgs):
            orc.kv_restore(oshape(shape), expect, bt2, 0, bt2.size, im.np, wl.dense_strides(shape, bt2.size, order))
        for a, b in zip(pool.read(), expect):
            assert np.array_equal(a, b)
        assert pool.guards_ok()


def test_small_transfers_carry_their_descriptor_in_the_launch(ctxs):
    ctx = ctxs[tb.VARIANT_ZEROCOPY]
    shape, nb = wl.TINY, 64
    g = wl.rng(19)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    for n, uploads in ((1, 0), (256 if nb >= 256 else nb, 0)):
        bt = wl.disjoint_tables(g, nb, [n])[0]
        img = GuardedPinned(n * shape.bytes_per_block)
        strides = wl.dense_strides(shape, n, "PF")
        ctx.reset_counters()
        ctx.kv_offload(pool.kv, bt, 0, n, img.ptr, tb.host_layout(strides, img.n))
        ctx.sync()
        c = ctx.get_counters()
        assert (c.kernel_launches, c.memcpy_calls) == (1, uploads)
        want = np.zeros(img.n, np.uint8)
        orc.kv_offload(oshape(shape), planes, bt, 0, n, want, strides)
        assert np.array_equal(img.np, want) and img.guards_ok()


def test_argument_errors_never_reach_the_gpu(ctxs):
    ctx = ctxs[tb.VARIANT_AUTO]
    shape, nb = wl.TINY, 32
    planes = wl.kv_pool(wl.rng(17), shape, nb)
    pool = DevicePool(shape, planes)
    n = 4
    strides = wl.dense_strides(shape, n, "PF")
    img = GuardedPinned(n * shape.bytes_per_block)
    hl = tb.host_layout(strides, img.n)

    def status(fn, *a):
        with pytest.raises(tb.TalariaError) as e:
            fn(*a)
        return e.value.status

    assert status(ctx.kv_offload, pool.kv, [0, 1, 2, nb], 0, n, img.ptr, hl) == tb.ERR_BAD_BLOCK_ID
    assert status(ctx.kv_offload, pool.kv, [0, -1, 2, 3], 0, n, img.ptr, hl) == tb.ERR_BAD_BLOCK_ID
    assert status(ctx.kv_restore, pool.kv, [0, 1, 2, 1], 0, n, img.ptr, hl) == tb.ERR_DUP_BLOCK
    assert status(ctx.kv_offload, pool.kv, [0, 1, 2, 3], 0, n, img.ptr, tb.host_layout(strides, img.n - 1)) == tb.ERR_EXTENT
    bad = (strides[0], strides[1], strides[2] - 16)
    assert status(ctx.kv_offload, pool.kv, [0, 1, 2, 3], 0, n, img.ptr, tb.host_layout(bad, img.n)) == tb.ERR_INVALID_ARG
    pageable = np.zeros(img.n, np.uint8)
    assert status(ctx.kv_offload, pool.kv, [0, 1, 2, 3], 0, n, pageable, hl) == tb.ERR_HOST_NOT_PINNED
    assert status(ctx.kv_gather, pool.kv, [0, 1, 2, 3], 0, n, img.ptr, hl) == tb.ERR_INVALID_ARG
    assert status(ctx.kv_offload, pool.kv, [0, 1, 2, 3], -1, n, img.ptr, hl) == tb.ERR_INVALID_ARG
    ctx.kv_offload(pool.kv, [0, 1, 2, 3], 0, 0, img.ptr, hl)          # zero blocks: a no-op
    ctx.sync()
    assert not img.np.any() and img.guards_ok()
    for a, b in zip(pool.read(), planes):
        assert np.array_equal(a, b)
    # the context is still healthy after every rejected call
    ctx.kv_offload(pool.kv, [3, 2, 1, 0], 0, n, img.ptr, hl)
    ctx.sync()
    want = np.zeros(img.n, np.uint8)
    orc.kv_offload(oshape(shape), planes, np.array([3, 2, 1, 0], np.int32), 0, n, want, strides)
    assert np.array_equal(img.np, want)


def test_two_streams_offload_and_restore_overlap(ctxs):
    # Sec. 4.3: checkpoints are issued as turns finish while other sessions are restored
    ctx = ctxs[tb.VARIANT_BOUNCE]
    shape, nb = wl.KvShape(4, 4, 16, 128), 160
    g = wl.rng(18)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    a, b, b_new = wl.disjoint_tables(g, nb, [40, 30, 30])
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    stra, strb = wl.dense_strides(shape, 40, "PF"), wl.dense_strides(shape, 30, "PF")
    img_a = GuardedPinned(40 * shape.bytes_per_block)
    img_b = GuardedPinned(30 * shape.bytes_per_block)
    orc.kv_offload(oshape(shape), planes, b, 0, 30, img_b.np, strb)       # session B was offloaded earlier
    torch.cuda.synchronize()
    ctx.kv_offload(pool.kv, a, 0, 40, img_a.ptr, tb.host_layout(stra, img_a.n), stream=sa)
    ctx.kv_restore(pool.kv, b_new, 0, 30, img_b.ptr, tb.host_layout(strb, img_b.n), stream=sb)
    ctx.sync(sa)
    ctx.sync(sb)
    want = np.zeros(img_a.n, np.uint8)
    orc.kv_offload(oshape(shape), planes, a, 0, 40, want, stra)
    assert np.array_equal(img_a.np, want)
    orc.kv_restore(oshape(shape), planes, b_new, 0, 30, img_b.np, strb)
    for x, y in zip(pool.read(), planes):
        assert np.array_equal(x, y)
    assert pool.guards_ok() and img_a.guards_ok() and img_b.guards_ok()


def test_device_side_guard_skips_bad_entries_when_host_validation_is_off():
    """With validate=0 a bad table reaches the kernel; it must skip the entry (no access outside the
    pool), leave everything else exact, and report through talaria_sync.  The bad id used here is
    num_blocks itself, whose chunk would start right at the end of each plane."""
    shape, nb = wl.TINY, 16
    g = wl.rng(19)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    ctx = tb.Talaria(0, variant=tb.VARIANT_ZEROCOPY, validate=False)
    try:
        n = 6
        table = np.array([3, 1, nb, 7, -1, 2], np.int32)              # entries 2 and 4 are outside the pool
        strides = wl.dense_strides(shape, n, "PF")
        img = GuardedPinned(n * shape.bytes_per_block, fill=0x99)
        hl = tb.host_layout(strides, img.n)
        ctx.kv_offload(pool.kv, table, 0, n, img.ptr, hl)
        with pytest.raises(tb.TalariaError) as e:
            ctx.sync()
        assert e.value.status == tb.ERR_BAD_BLOCK_ID
        ctx.sync()                                                     # reported once, then clear
        good = np.array([0, 1, 3, 5])
        want = np.full(img.n, 0x99, np.uint8)
        full = np.zeros(img.n, np.uint8)
        orc.kv_offload(oshape(shape), planes, np.where(table < 0, 0, np.minimum(table, nb - 1)).astype(np.int32),
                       0, n, full, strides)
        v_want, v_full = want.reshape(n, -1), full.reshape(n, -1)
        v_want[good] = v_full[good]                                    # skipped blocks keep the fill
        assert np.array_equal(img.np, want) and img.guards_ok()
        # the scatter direction: bad entries are skipped, the pool and its guard bands stay intact
        ctx.kv_restore(pool.kv, table, 0, n, img.ptr, hl)
        with pytest.raises(tb.TalariaError):
            ctx.sync()
        for a, b in zip(pool.read(), planes):
            assert np.array_equal(a, b)                               # good entries were restored onto themselves
        assert pool.guards_ok()
    finally:
        ctx.destroy()
