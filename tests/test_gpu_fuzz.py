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


@pytest.mark.parametrize("case", range(16))
def test_random_batches_mix_fused_and_single_transfers(case):
    """Batches of sessions with random sizes, layouts (dense or padded, any nesting), sub-ranges and
    alignment: small ones are fused into shared launches, large ones take the copy-engine variants;
    offload then restore into new blocks, against the oracle."""
    g = wl.rng(1001, case)
    shape = wl.KvShape(int(g.integers(1, 5)), int(g.choice([1, 2])), 16, int(g.choice([8, 64])),
                       elt_bytes=int(g.choice([1, 2])), num_planes=int(g.choice([1, 2])))
    nb = 640                                      # room for the largest draw: 13 sessions x 23 blocks, twice
    planes = [g.integers(0, 256, size=nb * shape.chunk_bytes, dtype=np.uint8)
              for _ in range(shape.num_layers * shape.num_planes)]
    pool = DevicePool(shape, planes)
    n_sess = int(g.integers(1, 14))
    totals = [int(g.integers(1, 24)) for _ in range(n_sess)]
    src = wl.disjoint_tables(g, nb, totals)
    dst = wl.disjoint_tables(g, nb, totals, exclude=np.concatenate(src))
    # a small dma threshold sends the larger sessions through the bounce / run variants
    ctx = tb.Talaria(0, bounce_bytes=1 << 20, dma_min_bytes=int(g.choice([1 << 12, 1 << 16, 1 << 30])))
    try:
        xo, xr, imgs, meta = [], [], [], []
        for s in range(n_sess):
            first = int(g.integers(0, totals[s]))
            n = totals[s] - first
            if g.uniform() < 0.6:
                strides = wl.dense_strides(shape, n, "PF" if g.uniform() < 0.6 else "LF")
                size = n * shape.bytes_per_block
            else:
                strides, size = _random_layout(g, shape, n)
            img = GuardedPinned(size, fill=0x3C)
            hl = tb.host_layout(strides, size)
            xo.append((src[s], first, n, img.ptr, hl))
            xr.append((dst[s], first, n, img.ptr, hl))
            imgs.append(img)
            meta.append((first, n, strides, size))
        ctx.kv_offload_batch(pool.kv, xo)
        ctx.sync()
        for s, (first, n, strides, size) in enumerate(meta):
            want = np.full(size, 0x3C, np.uint8)
            orc.kv_offload(oshape(shape), planes, src[s], first, n, want, strides)
            assert np.array_equal(imgs[s].np, want), (case, s)
            assert imgs[s].guards_ok()
        ctx.kv_restore_batch(pool.kv, xr)
        ctx.sync()
        for s, (first, n, strides, size) in enumerate(meta):
            orc.kv_restore(oshape(shape), planes, dst[s], first, n, imgs[s].np, strides)
        for a, b in zip(pool.read(), planes):
            assert np.array_equal(a, b)
        assert pool.guards_ok()
    finally:
        ctx.destroy()


@pytest.mark.parametrize("case", range(8))
def test_random_large_prefix_batches(case):
    """At least one pair per SM (the one-CTA-per-pair kernel): random block size among 4 / 8 / 16 / 32,
    ragged lengths around the kernel's round and chunk boundaries, random alignment of both token
    arrays, stored or derived session hashes -- every record and hash against the oracle."""
    import torch
    g = wl.rng(1002, case)
    B = int(g.choice([4, 8, 16, 32]))
    chunk, rnd = 1024 * B, 256 * B
    edges = [0, 1, B - 1, B, B + 1, rnd - 1, rnd, rnd + 1, chunk - B, chunk - 1, chunk, chunk + 1, chunk + rnd, 2 * chunk + 3]
    pairs = []
    for q in range(int(g.integers(150, 260))):
        def length():
            if g.uniform() < 0.15:
                return max(0, int(g.choice(edges)) + int(g.integers(-2, 3)))
            return int(g.integers(0, 2500))
        ts, tc = length(), length()
        s = wl.tokens(g, ts)
        shared = min(ts, tc) if g.uniform() < 0.3 else int(g.integers(0, min(ts, tc) + 1))
        pairs.append((wl.continuation(g, s, tc, shared), s))
    pad_c, pad_s = int(g.integers(0, 9)), int(g.integers(0, 9))
    cont = np.concatenate([np.zeros(pad_c, np.int32)] + [c for c, _ in pairs])
    sess = np.concatenate([np.zeros(pad_s, np.int32)] + [s for _, s in pairs])
    co = np.cumsum([pad_c] + [c.size for c, _ in pairs]).astype(np.int64)
    so = np.cumsum([pad_s] + [s.size for _, s in pairs]).astype(np.int64)
    stored = [orc.block_hash(s, B, wl.HASH_SEED) for _, s in pairs]
    with_stored = case % 2 == 1
    d_stored = None
    if with_stored:
        allh = np.concatenate(stored)
        d_stored = torch.from_numpy(allh.view(np.int64).copy()).cuda() if allh.size else torch.zeros(1, dtype=torch.int64, device="cuda")
    nbc = sum(c.size // B for c, _ in pairs)
    d_h = torch.full((max(nbc, 1) + 1,), -1, dtype=torch.int64, device="cuda")
    d_r = torch.zeros(len(pairs) * 4, dtype=torch.int64, device="cuda")
    ctx = tb.Talaria(0)
    try:
        before = ctx.get_counters().kernel_launches
        ctx.prefix_match(len(pairs), torch.from_numpy(cont).cuda(), co, torch.from_numpy(sess).cuda(), so, d_stored, B,
                         wl.HASH_SEED, d_h, d_r)
        ctx.sync()
        assert ctx.get_counters().kernel_launches - before == 1          # the single-launch path really ran
        res = d_r.cpu().numpy().view(tb.MATCH_DTYPE)
        hashes = d_h.cpu().numpy().view(np.uint64)
        assert hashes[nbc] == np.uint64(0xFFFFFFFFFFFFFFFF)              # nothing written past the last hash
        at = 0
        for q, (c, s) in enumerate(pairs):
            m, hc = orc.prefix_match(c, s, B, wl.HASH_SEED)
            r = res[q]
            assert (int(r["lcp_tokens"]), int(r["matched_blocks"]), int(r["reusable_tokens"]), int(r["hash_token_disagree"])) \
                == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree), (case, q, B)
            assert np.array_equal(hashes[at:at + hc.size], hc), (case, q)
            at += hc.size
    finally:
        ctx.destroy()
