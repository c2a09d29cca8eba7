"""Extents are checked on the host, like tables: an image, a pinned pool, a pool plane or a stage
range that runs off the allocation (or registration) holding its first byte is rejected with
ERR_EXTENT before anything is launched.  Every failure here is a host-side argument error; the
GPU never sees the bad range (the kernel-launch and copy counters stay where they were)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import DevicePool, GuardedPinned, oshape

pytestmark = pytest.mark.gpu

HUGE = 1 << 40          # far beyond any allocation of this process


def _status(fn, *a, **kw):
    with pytest.raises(tb.TalariaError) as e:
        fn(*a, **kw)
    return e.value.status


def _launched(ctx):
    c = ctx.get_counters()
    return c.kernel_launches, c.memcpy_calls


@pytest.mark.parametrize("variant", [tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE, tb.VARIANT_AUTO])
def test_image_that_runs_off_a_registration_is_rejected(variant):
    ctx = tb.Talaria(0, variant=variant, bounce_bytes=2 << 20, dma_min_bytes=1 << 20)
    shape, nb, n = wl.TINY, 64, 8
    planes = wl.kv_pool(wl.rng(40), shape, nb)
    pool = DevicePool(shape, planes)
    size = n * shape.bytes_per_block
    raw = np.zeros(size + (1 << 20), np.uint8)                 # the buffer is large enough ...
    reg = raw[: size - shape.chunk_bytes]                      # ... but only this much is page-locked
    ctx.host_register(reg)
    try:
        strides = wl.dense_strides(shape, n, "PF")
        table = np.arange(n, dtype=np.int32)
        before = _launched(ctx)
        # the declared capacity is larger than the registration
        assert _status(ctx.kv_offload, pool.kv, table, 0, n, raw, tb.host_layout(strides, size)) == tb.ERR_EXTENT
        assert _status(ctx.kv_restore, pool.kv, table, 0, n, raw, tb.host_layout(strides, size)) == tb.ERR_EXTENT
        evs = [torch.cuda.Event() for _ in range(shape.num_layers)]
        for e in evs:
            e.record()
        assert _status(ctx.kv_restore_layered, pool.kv, table, 0, n, raw, tb.host_layout(strides, size), evs) == tb.ERR_EXTENT
        offs = np.arange(n, dtype=np.int64) * shape.bytes_per_block
        assert _status(ctx.kv_offload_pages, pool.kv, table, 0, n, raw, size, offs) == tb.ERR_EXTENT
        assert _launched(ctx) == before                         # nothing was enqueued
        assert not raw.any()
        # one block fewer fits the registration and goes through
        m = n - 1
        hl = tb.host_layout(wl.dense_strides(shape, m, "PF"), m * shape.bytes_per_block)
        ctx.kv_offload(pool.kv, table, 0, m, raw, hl)
        ctx.sync()
        want = np.zeros(m * shape.bytes_per_block, np.uint8)
        orc.kv_offload(oshape(shape), planes, table, 0, m, want, wl.dense_strides(shape, m, "PF"))
        assert np.array_equal(raw[: want.size], want)
    finally:
        ctx.sync()
        ctx.host_unregister(reg)
        ctx.destroy()


def test_overstated_capacity_of_a_pinned_or_device_image_is_rejected():
    ctx = tb.Talaria(0)
    try:
        shape, nb, n = wl.TINY, 64, 4
        pool = DevicePool(shape, wl.kv_pool(wl.rng(41), shape, nb))
        img = GuardedPinned(n * shape.bytes_per_block)
        strides = wl.dense_strides(shape, n, "LF")
        table = np.arange(n, dtype=np.int32)
        before = _launched(ctx)
        assert _status(ctx.kv_offload, pool.kv, table, 0, n, img.ptr, tb.host_layout(strides, HUGE)) == tb.ERR_EXTENT
        torch.cuda.empty_cache()
        d_img = torch.zeros(n * shape.bytes_per_block, dtype=torch.uint8, device="cuda")
        assert _status(ctx.kv_gather, pool.kv, table, 0, n, d_img, tb.host_layout(strides, HUGE)) == tb.ERR_EXTENT
        assert _status(ctx.kv_scatter, pool.kv, table, 0, n, d_img, tb.host_layout(strides, HUGE)) == tb.ERR_EXTENT
        assert _launched(ctx) == before
        assert img.guards_ok() and not img.np.any()
        ctx.kv_offload(pool.kv, table, 0, n, img.ptr, tb.host_layout(strides, img.n))    # the honest size works
        ctx.kv_gather(pool.kv, table, 0, n, d_img, tb.host_layout(strides, d_img.numel()))
        ctx.sync()
        assert np.array_equal(d_img.cpu().numpy(), img.np)
    finally:
        ctx.destroy()


def test_plane_smaller_than_the_declared_pool_is_rejected():
    ctx = tb.Talaria(0)
    try:
        shape, nb, n = wl.TINY, 64, 4
        planes_np = wl.kv_pool(wl.rng(42), shape, nb)
        pool = DevicePool(shape, planes_np)
        ptrs = [b.ptr for b in pool.bufs]
        lying, keep = tb.kv_layout(shape, ptrs, HUGE // shape.chunk_bytes)     # claims a 1 TiB plane
        img = GuardedPinned(n * shape.bytes_per_block)
        hl = tb.host_layout(wl.dense_strides(shape, n, "PF"), img.n)
        table = np.arange(n, dtype=np.int32)
        before = _launched(ctx)
        for fn in (ctx.kv_offload, ctx.kv_restore):
            assert _status(fn, lying, table, 0, n, img.ptr, hl) == tb.ERR_EXTENT
        offs = np.arange(n, dtype=np.int64) * shape.bytes_per_block
        assert _status(ctx.kv_restore_pages, lying, table, 0, n, img.ptr, img.n, offs) == tb.ERR_EXTENT
        assert _launched(ctx) == before
        assert pool.guards_ok()
        for a, b in zip(pool.read(), planes_np):
            assert np.array_equal(a, b)
    finally:
        ctx.destroy()


def test_stage_ranges_that_leave_their_allocation_are_rejected():
    ctx = tb.Talaria(0)
    try:
        # 32 MiB tensors are allocations of their own.  The over-long ranges below run 4 MiB past
        # their tensor; the other end of each copy sits in the middle of a 192 MiB tensor, so the
        # two ranges of an entry can never meet (that would be an overlap error instead).
        nbytes, too_long, mid = 32 << 20, 36 << 20, 64 << 20
        torch.cuda.empty_cache()          # no cached block may be larger than the tensor it is handed to
        staging = torch.arange(nbytes // 8, dtype=torch.int64, device="cuda").view(torch.uint8)
        slots = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        big = torch.zeros(192 << 20, dtype=torch.uint8, device="cuda")
        host = torch.zeros(64 << 20, dtype=torch.uint8, pin_memory=True)
        small_host = torch.zeros(nbytes, dtype=torch.uint8, pin_memory=True)

        def plan(src_dev, src_host, dst, nb):
            a = np.zeros(1, tb.COPY_DTYPE)
            a[0] = (src_dev, src_host, dst, nb, 0, 0)
            return a

        before = _launched(ctx)
        dirty = np.array([1], np.uint8)
        src_runs_off = plan(staging.data_ptr(), 0, big.data_ptr() + mid, too_long)
        dst_runs_off = plan(big.data_ptr() + mid, 0, slots.data_ptr(), too_long)
        dst_runs_off_from_host = plan(0, host.data_ptr(), slots.data_ptr(), too_long)
        host_runs_off = plan(big.data_ptr() + mid, small_host.data_ptr(), big.data_ptr(), too_long)
        assert _status(ctx.stage, src_runs_off) == tb.ERR_EXTENT
        assert _status(ctx.stage, dst_runs_off) == tb.ERR_EXTENT
        assert _status(ctx.stage, dst_runs_off_from_host) == tb.ERR_EXTENT
        assert _status(ctx.stage, host_runs_off, dirty) == tb.ERR_EXTENT
        assert _status(ctx.stage_plan_create, src_runs_off) == tb.ERR_EXTENT
        assert _status(ctx.stage_plan_create, dst_runs_off) == tb.ERR_EXTENT
        staged, dbits = np.zeros(1, np.uint8), np.zeros(1, np.uint8)
        # pre-staging writes host bytes to src_dev: both of its ranges are checked too
        assert _status(ctx.prestage, plan(staging.data_ptr(), host.data_ptr(), 0, too_long), None, staged, dbits) == tb.ERR_EXTENT
        assert _status(ctx.prestage, plan(big.data_ptr(), small_host.data_ptr(), 0, too_long), None, staged, dbits) == tb.ERR_EXTENT
        assert _launched(ctx) == before and not staged.any()
        assert not slots.any().item() and not big.any().item()
        ctx.stage(plan(staging.data_ptr(), 0, slots.data_ptr(), nbytes))          # the honest plan works
        ctx.sync()
        assert torch.equal(slots, staging)
    finally:
        ctx.destroy()


def test_extent_checks_follow_memory_that_was_freed_and_allocated_again():
    """A cached description of an allocation must never reject a later, larger one at the same address."""
    ctx = tb.Talaria(0)
    try:
        shape, n = wl.TINY, 4
        pool = DevicePool(shape, wl.kv_pool(wl.rng(43), shape, 64))
        table = np.arange(n, dtype=np.int32)
        for blocks in (n, 4 * n, 64 * n):                # growing device images; torch may reuse addresses
            torch.cuda.empty_cache()
            d_img = torch.zeros(blocks * shape.bytes_per_block, dtype=torch.uint8, device="cuda")
            il = tb.host_layout(wl.dense_strides(shape, n, "PF"), d_img.numel())
            ctx.kv_gather(pool.kv, table, 0, n, d_img, il)
            ctx.sync()
            del d_img
    finally:
        ctx.destroy()
