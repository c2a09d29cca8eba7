"""GPU parity for page-first registry slabs: one slab per logical block anywhere in a pinned
host pool (App. C page-first view; Sec. 4.3 unified pinned pool), against the CPU oracle."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import DevicePool, GuardedPinned, oshape

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctxs():
    out = {v: tb.Talaria(0, variant=v, bounce_bytes=8 << 20, dma_min_bytes=1 << 20)
           for v in (tb.VARIANT_AUTO, tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE)}
    yield out
    for c in out.values():
        c.destroy()


def _roundtrip(ctx, shape, nb, n, seed, gap, adjacent_runs=False):
    g = wl.rng(800, seed)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    src, dst = wl.disjoint_tables(g, nb, [n, n])
    slab = shape.bytes_per_block
    pitch = slab + gap
    order = np.sort(g.permutation(2 * n)[:n]) if adjacent_runs else g.permutation(2 * n)[:n]
    offs = order.astype(np.int64) * pitch + (gap // 2)
    host = GuardedPinned(2 * n * pitch + 64, fill=0x42)
    ctx.kv_offload_pages(pool.kv, src, 0, n, host.ptr, host.n, offs)
    ctx.sync()
    want = np.full(host.n, 0x42, np.uint8)
    orc.kv_pages(oshape(shape), planes, src, 0, n, want, offs, True)
    assert np.array_equal(host.np, want) and host.guards_ok()
    ctx.kv_restore_pages(pool.kv, dst, 0, n, host.ptr, host.n, offs)
    ctx.sync()
    orc.kv_pages(oshape(shape), planes, dst, 0, n, want, offs, False)
    for a, b in zip(pool.read(), planes):
        assert np.array_equal(a, b)
    assert pool.guards_ok()
    return int(ctx.get_counters().last_variant)


@pytest.mark.parametrize("variant", [tb.VARIANT_AUTO, tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE])
def test_qwen_sized_slabs_shuffled_with_gaps(ctxs, variant):
    # 12 layers x 2 planes x 16 KiB = 384 KiB slabs; AUTO stays zero-copy below 1 MiB slabs
    used = _roundtrip(ctxs[variant], wl.KvShape(12, 4, 16, 128), 96, 30, 1, gap=256)
    assert used == (tb.VARIANT_BOUNCE if variant == tb.VARIANT_BOUNCE else tb.VARIANT_ZEROCOPY)
    _roundtrip(ctxs[variant], wl.KvShape(12, 4, 16, 128), 96, 30, 2, gap=0, adjacent_runs=True)


def test_auto_takes_the_copy_engine_only_for_long_runs_of_adjacent_slabs(ctxs):
    # 40 layers: 1.25 MiB slabs.  37 consecutive slabs = one 46 MiB run -> copy engine, several
    # bounce pieces; the same slabs scattered -> zero-copy kernel
    shape = wl.KvShape(40, 4, 16, 128)
    g = wl.rng(802)
    planes = wl.kv_pool(g, shape, 80)
    pool = DevicePool(shape, planes)
    src = wl.disjoint_tables(g, 80, [37])[0]
    host = GuardedPinned(37 * shape.bytes_per_block)
    ctx = ctxs[tb.VARIANT_AUTO]
    offs = np.arange(37, dtype=np.int64) * shape.bytes_per_block
    ctx.kv_offload_pages(pool.kv, src, 0, 37, host.ptr, host.n, offs)
    ctx.sync()
    assert int(ctx.get_counters().last_variant) == tb.VARIANT_BOUNCE
    want = np.zeros(host.n, np.uint8)
    orc.kv_pages(oshape(shape), planes, src, 0, 37, want, offs, True)
    assert np.array_equal(host.np, want)
    assert _roundtrip(ctx, shape, 80, 37, 4, gap=4096) == tb.VARIANT_ZEROCOPY


@pytest.mark.parametrize("shape,gap", [(wl.TINY, 0), (wl.KvShape(3, 1, 4, 3), 10), (wl.KvShape(2, 3, 5, 6, elt_bytes=1, num_planes=1), 3),
                                       (wl.KvShape(2, 1, 1, 8), 16)])
def test_odd_shapes_and_unaligned_slabs(ctxs, shape, gap):
    for v in (tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE):
        _roundtrip(ctxs[v], shape, 40, 9, 5, gap=gap)
        _roundtrip(ctxs[v], shape, 40, 1, 6, gap=gap)


def test_page_argument_errors(ctxs):
    ctx = ctxs[tb.VARIANT_AUTO]
    shape, nb = wl.TINY, 32
    pool = DevicePool(shape, wl.kv_pool(wl.rng(801), shape, nb))
    slab = shape.bytes_per_block
    host = GuardedPinned(8 * slab)

    def status(fn, *a):
        with pytest.raises(tb.TalariaError) as e:
            fn(*a)
        return e.value.status

    offs = np.arange(4, dtype=np.int64) * slab
    assert status(ctx.kv_offload_pages, pool.kv, [0, 1, 2, 3], 0, 4, host.ptr, host.n, [0, slab, slab + 16, 5 * slab]) == tb.ERR_OVERLAP
    assert status(ctx.kv_offload_pages, pool.kv, [0, 1, 2, 3], 0, 4, host.ptr, host.n, [0, slab, 2 * slab, 7 * slab + 1]) == tb.ERR_EXTENT
    assert status(ctx.kv_offload_pages, pool.kv, [0, 1, 2, 3], 0, 4, host.ptr, host.n, [0, slab, 2 * slab, -1]) == tb.ERR_EXTENT
    assert status(ctx.kv_restore_pages, pool.kv, [0, 1, 1, 3], 0, 4, host.ptr, host.n, offs) == tb.ERR_DUP_BLOCK
    assert status(ctx.kv_offload_pages, pool.kv, [0, 1, 2, 40], 0, 4, host.ptr, host.n, offs) == tb.ERR_BAD_BLOCK_ID
    assert status(ctx.kv_offload_pages, pool.kv, [0, 1, 2, 3], 0, 4, np.zeros(8 * slab, np.uint8), 8 * slab, offs) == tb.ERR_HOST_NOT_PINNED
    ctx.kv_restore_pages(pool.kv, [3, 2, 1, 0], 0, 4, host.ptr, host.n, [0, 0, 0, 0])     # reading one slab four times is fine
    ctx.sync()


def test_registry_keyed_restore_end_to_end(ctxs):
    """Turn finishes: pages are checkpointed and registered under their cumulative hashes.  The
    session returns with a longer prompt: its hashes are computed on the GPU, the registry gives
    the longest run of pages present, and exactly those pages are restored into new blocks."""
    ctx = ctxs[tb.VARIANT_AUTO]
    shape, nb = wl.TINY, 256
    g = wl.rng(1)
    wl.tokens(g, 300)
    sess = wl.tokens(g, 500)
    cont = wl.continuation(g, sess, 560, 350)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    n_full = 500 // 16
    src, dst = wl.disjoint_tables(g, nb, [n_full, 560 // 16 + 1])
    slab = shape.bytes_per_block
    host = GuardedPinned(64 * slab)
    offs = g.permutation(64)[:n_full].astype(np.int64) * slab
    # checkpoint + register (GPU hashes of the stored stream, read back to the host)
    ctx.kv_offload_pages(pool.kv, src, 0, n_full, host.ptr, host.n, offs)
    res = np.zeros(1, tb.MATCH_DTYPE)
    hs = np.zeros(n_full, np.uint64)
    ctx.prefix_match_host(1, sess, [0, 500], sess[:0], [0, 0], None, 16, wl.HASH_SEED, hs, res)
    reg, ref = tb.Registry(), orc.Registry()
    assert reg.insert(hs, offs) == ref.insert(orc.block_hash(sess, 16, wl.HASH_SEED), offs) == n_full
    # the session returns
    hc = np.zeros(560 // 16, np.uint64)
    ctx.prefix_match_host(1, cont, [0, 560], sess, [0, 500], hs, 16, wl.HASH_SEED, hc, res)
    k, pages = reg.lookup_prefix(hc)
    k_ref, pages_ref = ref.lookup_prefix(orc.block_hash(cont, 16, wl.HASH_SEED))
    assert k == k_ref == 21 == int(res[0]["matched_blocks"]) and np.array_equal(pages, pages_ref)
    ctx.kv_restore_pages(pool.kv, dst, 0, k, host.ptr, host.n, pages)
    ctx.sync()
    want_host = np.zeros(host.n, np.uint8)
    orc.kv_pages(oshape(shape), planes, src, 0, n_full, want_host, offs, True)
    assert np.array_equal(host.np, want_host)
    orc.kv_pages(oshape(shape), planes, dst, 0, k_ref, want_host, pages_ref, False)
    for a, b in zip(pool.read(), planes):
        assert np.array_equal(a, b)
    reg.destroy()
