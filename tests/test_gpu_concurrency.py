"""Many calls in flight at once: batches longer than the descriptor ring, and offload / restore /
staging / prefix match interleaved on several streams over disjoint data.  Operations on
disjoint data commute, so the final state must equal the oracle's whatever the interleaving."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import DevicePool, GuardedDevice, GuardedPinned, oshape

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant", [tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE])
def test_batches_longer_than_the_descriptor_ring(variant):
    shape, nb = wl.KvShape(3, 4, 16, 128), 400
    g = wl.rng(1100, variant)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    sizes = [int(x) for x in g.integers(1, 12, size=21)]                  # 21 sessions > 8 ring slots
    tables = wl.disjoint_tables(g, nb, sizes)
    new_tables = wl.disjoint_tables(g, nb, sizes, exclude=np.concatenate(tables))
    ctx = tb.Talaria(0, variant=variant, bounce_bytes=2 << 20)
    try:
        imgs, xo, xr = [], [], []
        for k, (bt, bt2) in enumerate(zip(tables, new_tables)):
            n = bt.size
            strides = wl.dense_strides(shape, n, "PF" if k % 2 else "LF")
            img = GuardedPinned(n * shape.bytes_per_block)
            hl = tb.host_layout(strides, img.n)
            imgs.append((img, strides))
            xo.append((bt, 0, n, img.ptr, hl))
            xr.append((bt2, 0, n, img.ptr, hl))
        ctx.kv_offload_batch(pool.kv, xo)
        ctx.kv_restore_batch(pool.kv, xr)                                 # same stream: ordered after the offloads
        ctx.sync()
        for (img, strides), bt, bt2 in zip(imgs, tables, new_tables):
            want = np.zeros(img.n, np.uint8)
            orc.kv_offload(oshape(shape), planes, bt, 0, bt.size, want, strides)
            assert np.array_equal(img.np, want) and img.guards_ok()
            orc.kv_restore(oshape(shape), planes, bt2, 0, bt2.size, want, strides)
        for a, b in zip(pool.read(), planes):
            assert np.array_equal(a, b)
        assert pool.guards_ok()
    finally:
        ctx.destroy()


def test_mixed_operations_on_three_streams():
    shape, nb = wl.KvShape(4, 4, 16, 128), 600
    g = wl.rng(1101)
    planes = wl.kv_pool(g, shape, nb)
    pool = DevicePool(shape, planes)
    ctx = tb.Talaria(0, bounce_bytes=4 << 20, dma_min_bytes=1 << 20)       # both variants get used
    streams = [torch.cuda.Stream() for _ in range(3)]
    try:
        n_jobs = 9
        sizes = [int(x) for x in g.integers(2, 40, size=n_jobs)]
        src = wl.disjoint_tables(g, nb, sizes)
        dst = wl.disjoint_tables(g, nb, sizes, exclude=np.concatenate(src))
        jobs = []
        for k in range(n_jobs):
            n = sizes[k]
            strides = wl.dense_strides(shape, n, "PF" if k % 3 else "LF")
            img = GuardedPinned(n * shape.bytes_per_block)
            jobs.append((src[k], dst[k], n, strides, img, tb.host_layout(strides, img.n)))
        # a staging plan and prefix pairs to run in between
        plan, total = wl.stage_plan([300_000, 70_001, 1 << 20], 64 << 10)
        weights = g.integers(0, 256, size=total, dtype=np.uint8)
        staging, slots = GuardedDevice(total, weights), GuardedDevice(total, np.zeros(total, np.uint8))
        arr = np.zeros(len(plan), tb.COPY_DTYPE)
        for k, (off, nbytes, cid) in enumerate(plan):
            arr[k] = (staging.ptr + off, 0, slots.ptr + off, nbytes, cid, 0)
        toks = [(wl.tokens(g, 20_000 + 700 * k), None) for k in range(3)]
        toks = [(s, wl.continuation(g, s, 21_000, 9_000 + 333 * k)) for k, (s, _) in enumerate(toks)]
        d_tok = [(torch.from_numpy(s).cuda(), torch.from_numpy(c).cuda(),
                  torch.zeros(21_000 // 16, dtype=torch.int64, device="cuda"),
                  torch.zeros(4, dtype=torch.int64, device="cuda")) for s, c in toks]
        torch.cuda.synchronize()
        for k, (bt, bt2, n, strides, img, hl) in enumerate(jobs):
            st = streams[k % 3]
            ctx.kv_offload(pool.kv, bt, 0, n, img.ptr, hl, stream=st)
            if k % 3 == 0:
                ctx.stage(arr, None, stream=streams[(k + 1) % 3])
            ds, dc, dh, dr = d_tok[k % 3]
            ctx.prefix_match(1, dc, [0, 21_000], ds, [0, toks[k % 3][0].size], None, 16, wl.HASH_SEED, dh, dr,
                             stream=streams[(k + 2) % 3])
            ctx.kv_restore(pool.kv, bt2, 0, n, img.ptr, hl, stream=st)      # same stream as its offload
        for st in streams:
            ctx.sync(st)
        expect = [p.copy() for p in planes]
        for bt, bt2, n, strides, img, hl in jobs:
            want = np.zeros(img.n, np.uint8)
            orc.kv_offload(oshape(shape), planes, bt, 0, n, want, strides)   # sources are never overwritten
            assert np.array_equal(img.np, want) and img.guards_ok()
            orc.kv_restore(oshape(shape), expect, bt2, 0, n, want, strides)
        for a, b in zip(pool.read(), expect):
            assert np.array_equal(a, b)
        covered = np.zeros(total, bool)
        for off, nbytes, _ in plan:
            covered[off:off + nbytes] = True
        assert np.array_equal(slots.read(), np.where(covered, weights, 0))
        for (s, c), (ds, dc, dh, dr) in zip(toks, d_tok):
            m, hc = orc.prefix_match(c, s, 16, wl.HASH_SEED)
            r = dr.cpu().numpy()
            assert [int(r[0]), int(r[1]), int(r[2])] == [m.lcp_tokens, m.matched_blocks, m.reusable_tokens]
            assert np.array_equal(dh.cpu().numpy().view(np.uint64), hc)
        assert pool.guards_ok() and slots.guards_ok()
    finally:
        ctx.destroy()
