"""GPU parity: staged-switch copy plan through the C ABI against the CPU oracle
(Sec. 4.4: D2D for clean staged chunks, host reload for dirty / missing ones)."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import GuardedDevice, GuardedPinned

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = tb.Talaria(0)
    yield c
    c.destroy()


def _run(ctx, sizes, chunk, dirty_frac, missing_frac, seed, align=256, shift_src=0, shift_dst=0):
    plan, total = wl.stage_plan(sizes, chunk, align=align)
    g = wl.rng(600, seed)
    weights = g.integers(0, 256, size=total + 64, dtype=np.uint8)
    n = len(plan)
    dirty = g.uniform(size=n) < dirty_frac
    missing = (~dirty) & (g.uniform(size=n) < missing_frac)
    staged = weights.copy()
    for off, nb, cid in plan:
        if dirty[cid]:
            staged[off:off + nb] ^= 0xFF
    host = GuardedPinned(total + 64)
    host.np[:] = weights
    staging = GuardedDevice(total + 64, staged, align_off=shift_src)
    slots = GuardedDevice(total + 64, np.full(total + 64, 0xEE, np.uint8), align_off=shift_dst)
    arr = np.zeros(n, tb.COPY_DTYPE)
    for k, (off, nb, cid) in enumerate(plan):
        arr[k] = (0 if missing[cid] else staging.ptr + off, host.ptr + off, slots.ptr + off, nb, cid, 0)
    bitmap = np.packbits(dirty, bitorder="little") if n else None
    st = ctx.stage(arr, bitmap)
    ctx.sync()
    # oracle on host copies of the same buffers
    o_slots = np.full(total + 64, 0xEE, np.uint8)
    entries = [(None if missing[cid] else off, off, off, nb, cid) for off, nb, cid in plan]
    ost = orc.stage(staged, weights, o_slots, entries, bitmap)
    assert np.array_equal(slots.read(), o_slots)
    assert np.array_equal(staging.read(), staged)                      # sources are never written
    assert (st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks) == \
        (ost.d2d_bytes, ost.h2d_bytes, ost.dirty_chunks, ost.missing_chunks)
    assert slots.guards_ok() and staging.guards_ok() and host.guards_ok()
    return st


def test_all_clean_many_tiles(ctx):
    # expert-matrix sized tensors (1.5 MiB) cut into 256 KiB chunks plus small norm vectors
    sizes = [4096 * 192 * 2] * 5 + [256, 8192, 4096 * 192 * 2, 2, 100_000]
    st = _run(ctx, sizes, 256 << 10, 0.0, 0.0, 1)
    assert st.h2d_bytes == 0 and st.d2d_bytes == sum(sizes)


@pytest.mark.parametrize("dirty,missing", [(0.01, 0.0), (0.36, 0.0), (0.2, 0.2), (1.0, 0.0), (0.0, 1.0)])
def test_dirty_and_missing_chunks_come_from_host(ctx, dirty, missing):
    sizes = [300_000, 70_001, 5, 1 << 20, 33_333]
    _run(ctx, sizes, 64 << 10, dirty, missing, 2)


@pytest.mark.parametrize("shift_src,shift_dst", [(0, 0), (16, 32), (4, 4), (1, 3), (0, 8)])
def test_unaligned_entries(ctx, shift_src, shift_dst):
    sizes = [100_003, 17, 65_536, 32_768 + 15, 1]
    _run(ctx, sizes, 48 << 10, 0.1, 0.05, 3, align=1, shift_src=shift_src, shift_dst=shift_dst)


@pytest.mark.parametrize("prepared", [False, True])
@pytest.mark.parametrize("shift", [(0, 0), (16, 0), (1, 3)])
def test_many_scattered_reloads_take_the_kernels_host_leg(ctx, prepared, shift):
    """More than 32 separate host-sourced runs: the reload is the staging kernel's second leg, reading
    the device-mapped pinned copies (aligned, 16-byte and byte paths), not one copy-engine call per run."""
    sizes = [24_001] * 40 + [300_000, 7, 65_536 * 3, 1 << 20] + [4096] * 60
    plan, total = wl.stage_plan(sizes, 32 << 10, align=1 if shift != (0, 0) else 256)
    g = wl.rng(602, 7 * shift[0] + shift[1] + (100 if prepared else 0))
    n = len(plan)
    weights = g.integers(0, 256, size=total + 64, dtype=np.uint8)
    dirty = np.zeros(n, bool)
    dirty[::2] = True                                                  # every other chunk: no two host runs merge
    missing = (~dirty) & (g.uniform(size=n) < 0.1)
    staged = weights.copy()
    for off, nb, cid in plan:
        if dirty[cid]:
            staged[off:off + nb] ^= 0xFF
    host = GuardedPinned(total + 64); host.np[:] = weights
    staging = GuardedDevice(total + 64, staged, align_off=shift[0])
    slots = GuardedDevice(total + 64, np.full(total + 64, 0xEE, np.uint8), align_off=shift[1])
    arr = np.zeros(n, tb.COPY_DTYPE)
    for k, (off, nb, cid) in enumerate(plan):
        arr[k] = (0 if missing[cid] else staging.ptr + off, host.ptr + off, slots.ptr + off, nb, cid, 0)
    bitmap = np.packbits(dirty, bitorder="little")
    assert int(dirty.sum() + missing.sum()) > 40
    ctx.sync()
    ctx.reset_counters()
    if prepared:
        h = ctx.stage_plan_create(arr)
        st = ctx.stage_plan_run(h, bitmap)
    else:
        st = ctx.stage(arr, bitmap)
    ctx.sync()
    c = ctx.get_counters()
    assert c.kernel_launches == 2                                      # the D2D leg and the host leg
    assert c.memcpy_calls <= 2                                         # descriptor / bitmap uploads only, no per-run copies
    o_slots = np.full(total + 64, 0xEE, np.uint8)
    entries = [(None if missing[cid] else off, off, off, nb, cid) for off, nb, cid in plan]
    ost = orc.stage(staged, weights, o_slots, entries, bitmap)
    assert np.array_equal(slots.read(), o_slots)
    assert (st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks) == \
        (ost.d2d_bytes, ost.h2d_bytes, ost.dirty_chunks, ost.missing_chunks)
    assert np.array_equal(staging.read(), staged) and np.array_equal(host.np, weights)
    assert slots.guards_ok() and staging.guards_ok() and host.guards_ok()
    if prepared:
        # the same plan, next switch: everything clean except what was never staged
        slots.write(np.full(total + 64, 0xEE, np.uint8))
        st2 = ctx.stage_plan_run(h, None)
        ctx.sync()
        o2 = np.full(total + 64, 0xEE, np.uint8)
        orc.stage(staged, weights, o2, entries, None)
        assert np.array_equal(slots.read(), o2) and st2.dirty_chunks == 0
        ctx.stage_plan_destroy(h)


def test_empty_plan_and_zero_byte_entries(ctx):
    st = ctx.stage(np.zeros(0, tb.COPY_DTYPE), None)
    assert (st.d2d_bytes, st.h2d_bytes) == (0, 0)
    a = GuardedDevice(4096, np.arange(4096, dtype=np.uint8))
    b = GuardedDevice(4096, np.zeros(4096, np.uint8))
    arr = np.zeros(3, tb.COPY_DTYPE)
    arr[0] = (a.ptr, 0, b.ptr, 0, 0, 0)
    arr[1] = (a.ptr + 100, 0, b.ptr + 100, 1000, 1, 0)
    arr[2] = (a.ptr + 2000, 0, b.ptr + 2000, 0, 2, 0)
    st = ctx.stage(arr, None)
    ctx.sync()
    want = np.zeros(4096, np.uint8); want[100:1100] = np.arange(4096, dtype=np.uint8)[100:1100]
    assert np.array_equal(b.read(), want) and st.d2d_bytes == 1000


def test_plan_errors(ctx):
    a = GuardedDevice(8192, np.zeros(8192, np.uint8))
    host = GuardedPinned(8192)

    def status(arr, bm=None):
        with pytest.raises(tb.TalariaError) as e:
            ctx.stage(arr, bm)
        return e.value.status

    arr = np.zeros(2, tb.COPY_DTYPE)
    arr[0] = (a.ptr, 0, a.ptr + 4096, 512, 0, 0)
    arr[1] = (a.ptr + 512, 0, a.ptr + 4096 + 256, 512, 1, 0)
    assert status(arr) == tb.ERR_OVERLAP                                   # destinations overlap
    arr[1] = (a.ptr + 4096 + 600, 0, a.ptr + 6000, 512, 1, 0)
    ctx.stage(arr, None)                                                   # dst 0 = [4096,4608), src 1 = [4696,5208): disjoint
    ctx.sync()
    arr[1] = (a.ptr + 4096 + 100, 0, a.ptr + 6000, 512, 1, 0)
    assert status(arr) == tb.ERR_OVERLAP                                   # a destination covers a live source
    arr[1] = (a.ptr + 4096 + 100, host.ptr, a.ptr + 6000, 512, 1, 0)
    st = ctx.stage(arr, np.array([0b10], np.uint8))                        # ... fine once that source is dirty
    ctx.sync()
    assert st.dirty_chunks == 1
    arr[1] = (0, 0, a.ptr + 6000, 512, 1, 0)
    assert status(arr) == tb.ERR_INVALID_ARG                               # missing chunk without a host copy
    pageable = np.zeros(512, np.uint8)
    arr[1] = (0, pageable.ctypes.data, a.ptr + 6000, 512, 1, 0)
    assert status(arr) == tb.ERR_HOST_NOT_PINNED
    arr[1] = (a.ptr, 0, 0, 512, 1, 0)
    assert status(arr) == tb.ERR_INVALID_ARG


def test_prestage_then_dirty_marking_then_switch(ctx):
    """The whole Sec. 4.4 protocol: pre-stage what is not blocked, a KV allocation scribbles over
    part of the staging region and marks those chunks dirty, the switch then takes clean chunks
    D2D and dirty / unstaged ones from host; every slot must end up with the authoritative bytes."""
    sizes = [300_000, 70_001, 5, 1 << 20, 33_333, 4096 * 192 * 2]
    plan, total = wl.stage_plan(sizes, 64 << 10)
    g = wl.rng(601)
    n = len(plan)
    weights = g.integers(0, 256, size=total, dtype=np.uint8)
    host = GuardedPinned(total); host.np[:] = weights
    staging = GuardedDevice(total, np.full(total, 0x77, np.uint8))
    slots = GuardedDevice(total, np.full(total, 0xEE, np.uint8))
    arr = np.zeros(n, tb.COPY_DTYPE)
    for k, (off, nb, cid) in enumerate(plan):
        arr[k] = (staging.ptr + off, host.ptr + off, slots.ptr + off, nb, cid, 0)
    blocked = g.uniform(size=n) < 0.25
    staged, dirty = np.zeros((n + 7) // 8, np.uint8), np.zeros((n + 7) // 8, np.uint8)
    st = ctx.prestage(arr, np.packbits(blocked, bitorder="little"), staged, dirty)
    ctx.sync()
    # oracle mirror
    o_staging = np.full(total, 0x77, np.uint8)
    o_staged, o_dirty = np.zeros_like(staged), np.zeros_like(dirty)
    entries = [(off, off, off, nb, cid) for off, nb, cid in plan]
    ost = orc.prestage(o_staging, weights, entries, np.packbits(blocked, bitorder="little"), o_staged, o_dirty)
    assert np.array_equal(staging.read(), o_staging) and np.array_equal(staged, o_staged)
    assert (st.h2d_bytes, st.missing_chunks, st.dirty_chunks) == (ost.h2d_bytes, ost.missing_chunks, ost.dirty_chunks)
    # a prefill allocation takes rows in the middle of the staging region
    a_off, a_len = total // 3, 200_000
    junk = g.integers(0, 256, size=a_len, dtype=np.uint8)
    view = staging.read(); view[a_off:a_off + a_len] = junk; staging.write(view)
    o_staging[a_off:a_off + a_len] = junk
    changed = tb.Talaria.mark_dirty(arr, staging.ptr + a_off, a_len, staged, dirty)
    assert changed == orc.mark_dirty(o_staging, entries, a_off, a_len, o_staged, o_dirty) > 0
    assert np.array_equal(dirty, o_dirty)
    # switch: unstaged chunks are "missing"
    is_staged = np.unpackbits(staged, bitorder="little")[:n].astype(bool)
    sw = arr.copy()
    sw["src_dev"][~is_staged] = 0
    sst = ctx.stage(sw, dirty)
    ctx.sync()
    covered = np.zeros(total, bool)                      # alignment gaps between tensors are never copied
    for off, nb, _ in plan:
        covered[off:off + nb] = True
    assert np.array_equal(slots.read(), np.where(covered, weights, 0xEE))
    assert sst.missing_chunks == int((~is_staged).sum()) and sst.dirty_chunks == changed
    # staging again clears the dirty bits of rewritten chunks
    st2 = ctx.prestage(arr, None, staged, dirty)
    ctx.sync()
    assert st2.dirty_chunks == changed and not dirty.any()
    assert np.array_equal(staging.read()[covered], weights[covered])
    assert slots.guards_ok() and staging.guards_ok() and host.guards_ok()


def test_prestage_errors(ctx):
    a = GuardedDevice(8192, np.zeros(8192, np.uint8))
    host = GuardedPinned(8192)
    arr = np.zeros(2, tb.COPY_DTYPE)
    arr[0] = (a.ptr, host.ptr, 0, 1024, 0, 0)
    arr[1] = (a.ptr + 512, host.ptr + 2048, 0, 1024, 1, 0)
    bm = np.zeros(1, np.uint8)
    with pytest.raises(tb.TalariaError) as e:
        ctx.prestage(arr, None, bm, bm.copy())
    assert e.value.status == tb.ERR_OVERLAP and not bm.any()
    arr[1] = (a.ptr + 2048, np.zeros(1024, np.uint8).ctypes.data, 0, 1024, 1, 0)
    with pytest.raises(tb.TalariaError) as e:
        ctx.prestage(arr, None, bm, bm.copy())
    assert e.value.status == tb.ERR_HOST_NOT_PINNED and not bm.any()
    arr[1] = (a.ptr + 2048, host.ptr + 2048, 0, 1024, -1, 0)
    with pytest.raises(tb.TalariaError) as e:
        ctx.prestage(arr, None, bm, bm.copy())
    assert e.value.status == tb.ERR_INVALID_ARG


def test_prepared_plan_runs_match_the_oracle_for_changing_bitmaps(ctx):
    """One prepared plan, several switches: all clean, 1 % dirty, 36 % dirty, all dirty; some chunks
    were never staged.  Every run must leave the slots as the oracle's stage() does."""
    sizes = [300_000, 70_001, 5, 1 << 20, 33_333, 4096 * 192 * 2, 64]
    plan, total = wl.stage_plan(sizes, 64 << 10)
    g = wl.rng(602)
    n = len(plan)
    weights = g.integers(0, 256, size=total, dtype=np.uint8)
    missing = g.uniform(size=n) < 0.05
    host = GuardedPinned(total); host.np[:] = weights
    staging = GuardedDevice(total, weights)
    slots = GuardedDevice(total, np.zeros(total, np.uint8))
    arr = np.zeros(n, tb.COPY_DTYPE)
    for k, (off, nb, cid) in enumerate(plan):
        arr[k] = (0 if missing[k] else staging.ptr + off, host.ptr + off, slots.ptr + off, nb, cid, 0)
    prepared = ctx.stage_plan_create(arr)
    try:
        for frac in (0.0, 0.01, 0.36, 1.0, 0.0):
            dirty = g.uniform(size=n) < frac
            staged = weights.copy()
            for (off, nb, cid) in plan:
                if dirty[cid]:
                    staged[off:off + nb] ^= 0x5A                    # a KV allocation scribbled over these chunks
            staging.write(staged)
            slots.write(np.full(total, 0xEE, np.uint8))
            bitmap = np.packbits(dirty, bitorder="little")
            st = ctx.stage_plan_run(prepared, bitmap if frac else None if not dirty.any() else bitmap)
            ctx.sync()
            o_slots = np.full(total, 0xEE, np.uint8)
            entries = [(None if missing[c] else off, off, off, nb, c) for off, nb, c in plan]
            ost = orc.stage(staged, weights, o_slots, entries, bitmap)
            assert np.array_equal(slots.read(), o_slots), frac
            assert (st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks) == \
                (ost.d2d_bytes, ost.h2d_bytes, ost.dirty_chunks, ost.missing_chunks)
            # and the one-shot call agrees with the prepared one
            slots.write(np.full(total, 0xEE, np.uint8))
            ctx.stage(arr, bitmap)
            ctx.sync()
            assert np.array_equal(slots.read(), o_slots)
        assert slots.guards_ok() and staging.guards_ok()
    finally:
        ctx.stage_plan_destroy(prepared)
    bad = arr[:2].copy()
    bad[1]["dst_dev"] = bad[0]["dst_dev"]
    bad[1]["bytes"] = bad[0]["bytes"] = 1024
    with pytest.raises(tb.TalariaError) as e:
        ctx.stage_plan_create(bad)
    assert e.value.status == tb.ERR_OVERLAP
