"""The Sec. 4.4 protocol end to end with every address coming from the stable-address layout of
Sec. 4.2: model A serves from KV planes placed by the allocator, model B's weights are pre-staged
into the tails of those planes (rows under the write are passed over by the allocator), prefill
allocations reach into the tails and dirty some chunks, the switch gathers clean chunks device to
device into B's weights region and reloads dirty / unplaced ones from the host, and after switching
back A finds every region where it was.  The whole region is mirrored on the host and every step
is replayed with the CPU oracle; the two must agree byte for byte."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import GuardedDevice, GuardedPinned, oshape

pytestmark = pytest.mark.gpu


def test_prestage_allocate_switch_through_allocator_addresses():
    g = wl.rng(720)
    shape_a, shape_b = wl.KvShape(2, 2, 16, 64), wl.KvShape(3, 2, 16, 64)
    Cb = shape_a.chunk_bytes
    S = 24 << 20
    W_a, W_b = 3 << 20, (5 << 20) + 1234
    models = [(W_a, 1 << 20, shape_a.num_layers, shape_a.num_planes, Cb),
              (W_b, 2 << 20, shape_b.num_layers, shape_b.num_planes, shape_b.chunk_bytes)]
    region = GuardedDevice(S, g.integers(0, 256, size=S, dtype=np.uint8))
    mirror = region.read().copy()
    base = region.ptr
    assert base % 256 == 0
    bump = tb.Bump(base, S, models)
    ob = orc.BumpLayout(S, 256, models)
    ctx = tb.Talaria(0)
    try:
        # ---- model A is active: its KV planes come from the layout -----------------------------
        va = bump.activate(0); ob.activate(0)
        _, planes_a = bump.view(0)
        NB = va.num_blocks
        kv, keep = tb.kv_layout(shape_a, planes_a, NB)
        m_planes = [mirror[p - base:p - base + NB * Cb] for p in planes_a]       # views into the mirror

        def prefill(n, staged_bm=None, dirty_bm=None):
            """A call's KV: n new blocks from the allocator, filled with seeded bytes."""
            ids, nd = bump.alloc_blocks(n, staged_bm, dirty_bm)
            img = g.integers(0, 256, size=n * shape_a.bytes_per_block, dtype=np.uint8)
            strides = wl.dense_strides(shape_a, n, "PF")
            ctx.kv_scatter(kv, ids, 0, n, torch.from_numpy(img).cuda(), tb.host_layout(strides, img.size))
            ctx.sync()
            orc.kv_restore(oshape(shape_a), m_planes, ids, 0, n, img, strides)
            return ids, nd

        ids1, _ = prefill(NB // 4)
        assert list(ids1) == list(range(NB // 4))                                # low addresses first
        # ---- pre-stage model B's weights into the plane tails ------------------------------------
        weights = g.integers(0, 256, size=W_b, dtype=np.uint8)
        host = GuardedPinned(W_b); host.np[:] = weights
        chunk = 64 << 10
        plan, placed = bump.stage_place(1, chunk, host_weights=host.ptr)
        n_chunks = plan.size
        assert placed == n_chunks == -(-W_b // chunk)                            # the tails have room for all of B
        slack0 = bump.staging_slack(1, chunk)
        staged, dirty = np.zeros((n_chunks + 7) // 8, np.uint8), np.zeros((n_chunks + 7) // 8, np.uint8)
        for c in range(n_chunks):
            bump.lock_chunk(c, True)                                             # the write is in flight ...
        ctx.prestage(plan, None, staged, dirty)
        rows_per_chunk = chunk // Cb
        lowest_staged_row = NB - -(-n_chunks // (shape_a.num_layers * shape_a.num_planes)) * rows_per_chunk
        ids2, _ = prefill(NB // 4)                                               # ... so an allocation made now stays below it
        assert max(ids2) < lowest_staged_row
        with pytest.raises(tb.TalariaError) as e:                                # and cannot take the rows being written
            bump.alloc_blocks(NB - NB // 2 - (NB - lowest_staged_row) + 1)
        assert e.value.status == tb.ERR_NO_MEMORY
        ctx.sync()
        for c in range(n_chunks):
            bump.lock_chunk(c, False)
        entries = [(int(e["src_dev"]) - base, int(e["src_host"]) - host.ptr, int(e["dst_dev"]) - base, int(e["bytes"]),
                    int(e["chunk_id"])) for e in plan]
        o_staged, o_dirty = np.zeros_like(staged), np.zeros_like(dirty)
        orc.prestage(mirror, weights, entries, None, o_staged, o_dirty)
        assert np.array_equal(region.read(), mirror) and np.array_equal(staged, o_staged)
        # ---- prefill allocations reach into the tails: those chunks become dirty --------------------
        want_dirty = dirty.copy()
        n3 = (lowest_staged_row - NB // 2) + 2 * rows_per_chunk + 3              # past the first two tail slots of every plane
        ids3, nd = prefill(n3, staged, dirty)
        changed = 0
        for bid in ids3:                                                          # the interval definition, range by range
            for p in planes_a:
                changed += tb.Talaria.mark_dirty(plan, p + int(bid) * Cb, Cb, staged, want_dirty)
                orc.mark_dirty(mirror, entries, p - base + int(bid) * Cb, Cb, o_staged, o_dirty)
        assert nd == changed > 0 and np.array_equal(dirty, want_dirty) and np.array_equal(dirty, o_dirty)
        assert 0 < int(np.unpackbits(dirty, bitorder="little").sum()) < n_chunks
        assert bump.staging_slack(1, chunk) <= slack0
        # ---- the switch: clean chunks D2D, dirty ones from host, into B's weights region -------------
        vb, planes_b = bump.view(1)
        assert vb.weights_base == base and int(plan[0]["dst_dev"]) == base
        st = ctx.stage(plan, dirty)
        ctx.sync()
        ost = orc.stage(mirror, weights, mirror, entries, dirty)
        assert (st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks) == \
            (ost.d2d_bytes, ost.h2d_bytes, ost.dirty_chunks, ost.missing_chunks)
        got = region.read()
        assert np.array_equal(got[:W_b], weights)                                # B's weights are exactly the authoritative bytes
        assert np.array_equal(got, mirror) and region.guards_ok() and host.guards_ok()
        # ---- B serves from its own planes; switching back, A finds everything where it was ------------
        bump.activate(1); ob.activate(1)
        kv_b, keep_b = tb.kv_layout(shape_b, planes_b, vb.num_blocks)
        idb, _ = bump.alloc_blocks(5)
        img = g.integers(0, 256, size=5 * shape_b.bytes_per_block, dtype=np.uint8)
        sb = wl.dense_strides(shape_b, 5, "LF")
        ctx.kv_scatter(kv_b, idb, 0, 5, torch.from_numpy(img).cuda(), tb.host_layout(sb, img.size))
        ctx.sync()
        mb = [mirror[p - base:p - base + vb.num_blocks * shape_b.chunk_bytes] for p in planes_b]
        orc.kv_restore(oshape(shape_b), mb, idb, 0, 5, img, sb)
        assert np.array_equal(region.read(), mirror)
        assert np.array_equal(region.read()[:W_b], weights)                      # the pool never reaches into the weights
        va2 = bump.activate(0)
        _, planes_a2 = bump.view(0)
        assert (va2.weights_base, va2.kv_base, va2.runtime_base, va2.num_blocks, planes_a2) == \
            (va.weights_base, va.kv_base, va.runtime_base, va.num_blocks, planes_a)
    finally:
        ctx.destroy()
