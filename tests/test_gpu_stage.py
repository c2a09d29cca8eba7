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
