"""Pins for the oracle's staged-switch copy plan (Sec. 4.4: clean staged chunks
move device-to-device, dirty or missing chunks are reloaded from host; App. D
path classification: staged-byte coverage and dirty bytes per switch)."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import workloads as wl


def _setup(seed, sizes, chunk):
    plan, total = wl.stage_plan(sizes, chunk)
    g = wl.rng(400, seed)
    weights = g.integers(0, 256, size=total, dtype=np.uint8)      # authoritative host copy
    staging = weights.copy()
    slots = np.full(total, 0xEE, np.uint8)
    return plan, total, weights, staging, slots


def test_plan_covers_every_tensor_byte_once():
    sizes = [1000, 4096, 1, 8191, 8192, 8193]
    plan, total = wl.stage_plan(sizes, 4096, align=256)
    covered = np.zeros(total, np.int32)
    for off, n, _ in plan:
        assert 0 < n <= 4096
        covered[off:off + n] += 1
    at = 0
    for s in sizes:
        assert np.all(covered[at:at + s] == 1)
        pad = -(-s // 256) * 256
        assert np.all(covered[at + s:at + pad] == 0)
        at += pad
    assert [c for _, _, c in plan] == list(range(len(plan)))


def test_all_clean_is_plain_slices():
    plan, total, weights, staging, slots = _setup(1, [5000, 300, 70000], 4096)
    entries = [(off, off, off, n, cid) for off, n, cid in plan]
    st = orc.stage(staging, weights, slots, entries, None)
    want = np.full(total, 0xEE, np.uint8)
    for off, n, _ in plan:
        want[off:off + n] = staging[off:off + n]
    assert np.array_equal(slots, want)
    assert (st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks) == (sum(n for _, n, _ in plan), 0, 0, 0)


def test_dirty_chunks_take_host_bytes_even_when_staging_is_corrupt():
    plan, total, weights, staging, slots = _setup(2, [20000, 9000, 123], 2048)
    g = wl.rng(401)
    nchunks = len(plan)
    dirty = g.uniform(size=nchunks) < 0.36
    missing = (~dirty) & (g.uniform(size=nchunks) < 0.1)
    bitmap = np.packbits(dirty, bitorder="little")
    for (off, n, cid) in plan:
        if dirty[cid]:
            staging[off:off + n] ^= 0xFF                 # an overlapping allocation scribbled here
    entries = [(None if missing[cid] else off, off, off, n, cid) for off, n, cid in plan]
    st = orc.stage(staging, weights, slots, entries, bitmap)
    for off, n, _ in plan:
        assert np.array_equal(slots[off:off + n], weights[off:off + n])
    h2d = sum(n for _, n, c in plan if dirty[c] or missing[c])
    assert st.h2d_bytes == h2d and st.d2d_bytes == sum(n for _, n, _ in plan) - h2d
    assert st.dirty_chunks == int(dirty.sum()) and st.missing_chunks == int(missing.sum())
    assert np.array_equal(staging != weights, np.isin(np.arange(total), np.concatenate(
        [np.arange(off, off + n) for off, n, c in plan if dirty[c]])))   # the source side is never written


def test_bitmap_is_lsb_first():
    plan, total, weights, staging, slots = _setup(3, [64] * 10, 64, )
    staging[:] = 0
    bitmap = np.array([0b00000100, 0b00000010], np.uint8)   # chunks 2 and 9
    entries = [(off, off, off, n, cid) for off, n, cid in plan]
    st = orc.stage(staging, weights, slots, entries, bitmap)
    assert st.dirty_chunks == 2
    for off, n, cid in plan:
        src = weights if cid in (2, 9) else staging
        assert np.array_equal(slots[off:off + n], src[off:off + n])


def test_missing_host_copy_is_an_error_and_empty_plan_is_fine():
    plan, total, weights, staging, slots = _setup(4, [100], 64)
    with pytest.raises(ValueError):
        orc.stage(staging, None, slots, [(None, None, 0, 64, 0)], None)
    st = orc.stage(staging, weights, slots, [], None)
    assert (st.d2d_bytes, st.h2d_bytes) == (0, 0)


def test_validate_rejects_overlapping_destinations_and_dst_over_live_source():
    buf = np.zeros(4096, np.uint8)
    ok = [(0, 0, 2048, 512, 0), (512, 512, 2560, 512, 1)]
    assert orc.stage_validate(buf, buf, buf, ok, None)
    assert not orc.stage_validate(buf, buf, buf, [(0, 0, 2048, 512, 0), (512, 512, 2300, 512, 1)], None)
    assert not orc.stage_validate(buf, buf, buf, [(0, 0, 2048, 512, 0), (2100, 512, 3000, 512, 1)], None)
    # the same plan is fine once the clashing source chunk is dirty (it is then not read)
    bm = np.array([0b10], np.uint8)
    assert orc.stage_validate(buf, buf, buf, [(0, 0, 2048, 512, 0), (2100, 512, 3000, 512, 1)], bm)


def test_prestage_writes_unblocked_chunks_and_updates_bitmaps():
    plan, total, weights, staging, slots = _setup(5, [9000, 4096, 100, 20000], 2048)
    staging[:] = 0x77
    n = len(plan)
    g = wl.rng(402)
    blocked = g.uniform(size=n) < 0.3
    staged = np.zeros((n + 7) // 8, np.uint8)
    dirty = np.packbits(g.uniform(size=n) < 0.5, bitorder="little")
    dirty0 = np.unpackbits(dirty, bitorder="little")[:n].astype(bool)
    entries = [(off, off, off, nb, cid) for off, nb, cid in plan]
    st = orc.prestage(staging, weights, entries, np.packbits(blocked, bitorder="little"), staged, dirty)
    want = np.full(total, 0x77, np.uint8)
    for off, nb, cid in plan:
        if not blocked[cid]:
            want[off:off + nb] = weights[off:off + nb]
    assert np.array_equal(staging, want)
    assert np.array_equal(np.unpackbits(staged, bitorder="little")[:n].astype(bool), ~blocked)
    assert np.array_equal(np.unpackbits(dirty, bitorder="little")[:n].astype(bool), dirty0 & blocked)
    assert st.h2d_bytes == sum(nb for _, nb, c in plan if not blocked[c])
    assert st.missing_chunks == int(blocked.sum()) and st.dirty_chunks == int((dirty0 & ~blocked).sum())


def test_mark_dirty_is_interval_overlap_over_staged_chunks():
    plan, total, weights, staging, slots = _setup(6, [5000, 300, 12000], 1024)
    n = len(plan)
    g = wl.rng(403)
    entries = [(off, off, off, nb, cid) for off, nb, cid in plan]
    for _ in range(60):
        staged_b = g.uniform(size=n) < 0.7
        staged = np.packbits(staged_b, bitorder="little")
        dirty = np.zeros_like(staged)
        a = int(g.integers(0, total)); b = int(g.integers(0, 4000))
        changed = orc.mark_dirty(staging, entries, a, b, staged, dirty)
        want = np.array([staged_b[c] and b > 0 and off < a + b and a < off + nb for off, nb, c in plan])
        assert np.array_equal(np.unpackbits(dirty, bitorder="little")[:n].astype(bool), want)
        assert changed == int(want.sum())
        assert orc.mark_dirty(staging, entries, a, b, staged, dirty) == 0      # idempotent
    # a staged chunk next to, but not touching, the allocation stays clean
    dirty = np.zeros((n + 7) // 8, np.uint8)
    off, nb, cid = plan[3]
    assert orc.mark_dirty(staging, entries, off + nb, 10, None, dirty) == (1 if plan[4][0] == off + nb else 0)
    assert not (dirty[cid >> 3] >> (cid & 7)) & 1
