"""GPU parity at the full sizes of the benchmark configurations, in the launch
configuration `bench.py` times (default context: AUTO variant, 128 MiB bounce, page-first).

At these sizes (4.8 - 59 GB) the oracle cannot mirror everything in seconds, so each test checks
  (a) sampled layers / plan entries against the CPU oracle, byte for byte, and
  (b) properties that hold at any size, evaluated for EVERY chunk with torch indexing on the
      device as an independent routine: image[l,p,i] == pool[l,p][table[i]] after offload,
      pool[l,p][new_table[i]] == image[l,p,i] after restore, and per-block checksums of every
      untouched block unchanged.
Sec. 4.3 (checkpoint / restore into new slots), Sec. 4.4 (staged switch), App. A (prefix reuse).
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _need(host_gb: float, device_gb: float):
    """Skip (rather than fail half-way) when the box cannot hold the full-size case right now."""
    import psutil
    free_dev, _ = torch.cuda.mem_get_info()
    torch.cuda.empty_cache()
    free_dev = max(free_dev, torch.cuda.mem_get_info()[0])
    avail = psutil.virtual_memory().available
    if avail < host_gb * 1.25e9:
        pytest.skip(f"needs {host_gb * 1.25:.0f} GB of free host memory for pinned images, the box has {avail / 1e9:.0f} GB available")
    if free_dev < device_gb * 1.02e9:
        pytest.skip(f"needs {device_gb * 1.02:.0f} GB of free device memory, the GPU has {free_dev / 1e9:.0f} GB free")


def _pool(shape, num_blocks, seed):
    torch.cuda.empty_cache()
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    planes = []
    for _ in range(shape.num_layers * shape.num_planes):
        t = torch.empty(num_blocks * shape.chunk_bytes // 2, dtype=torch.bfloat16, device=DEV)
        t.normal_(generator=gen)
        planes.append(t.view(torch.uint8))
    kv, keep = tb.kv_layout(shape, [t.data_ptr() for t in planes], num_blocks)
    return planes, kv, keep


def _block_sums(planes, num_blocks):
    """One 64-bit checksum per (plane, block)."""
    return torch.stack([p.view(torch.int64).view(num_blocks, -1).sum(1) for p in planes])


def _image_chunks(image_dev, shape, n, strides, l, p):
    """[n, C] view of plane (l, p) inside a dense device copy of the image."""
    C = shape.chunk_bytes
    base = l * strides[0] + p * strides[1]
    return torch.as_strided(image_dev, (n, C), (strides[2], 1), base)


def _check_image_against_pool(image_pinned, planes, shape, num_blocks, table, n, strides, layers_dev_check=None):
    """Property (b): every chunk of the image equals the pool chunk its table entry names."""
    C = shape.chunk_bytes
    idx = torch.from_numpy(np.ascontiguousarray(table[:n]).astype(np.int64)).to(DEV)
    image_dev = image_pinned.to(DEV, non_blocking=True)
    for l in range(shape.num_layers):
        for p in range(shape.num_planes):
            want = planes[l * shape.num_planes + p].view(num_blocks, C)[idx]
            got = _image_chunks(image_dev, shape, n, strides, l, p)
            assert torch.equal(got, want), (l, p)
    del image_dev


def _oracle_layers(image_np, planes, shape, table, n, strides, layers, restored_into=None, n_restore=0):
    """(a): one-layer oracle runs on sampled layers."""
    one = orc.KvShape(1, shape.num_kv_heads, shape.block_tokens, shape.head_dim, shape.elt_bytes, shape.num_planes)
    C, P = shape.chunk_bytes, shape.num_planes
    for l in layers:
        host_planes = [planes[l * P + p].cpu().numpy() for p in range(P)]
        lo = l * strides[0]
        size = (P - 1) * strides[1] + (n - 1) * strides[2] + C
        view = image_np[lo:lo + size]
        if restored_into is None:
            want = np.zeros(size, np.uint8)
            orc.kv_offload(one, host_planes, table, 0, n, want, strides)
            for p in range(P):
                a = np.lib.stride_tricks.as_strided(view[p * strides[1]:], (n, C), (strides[2], 1))
                b = np.lib.stride_tricks.as_strided(want[p * strides[1]:], (n, C), (strides[2], 1))
                assert np.array_equal(a, b), (l, p)
        else:
            # the device planes must already equal "oracle restore applied to the device planes"
            after = [hp.copy() for hp in host_planes]
            orc.kv_restore(one, after, restored_into, 0, n_restore, view, strides)
            for a, b in zip(after, host_planes):
                assert np.array_equal(a, b), l


@pytest.mark.parametrize("variant", [tb.VARIANT_AUTO, tb.VARIANT_ZEROCOPY])
def test_config2_qwen235_one_session(variant):
    _need(host_gb=6, device_gb=20)
    shape, NB = wl.QWEN235, 4096
    g = wl.rng(2)
    sess = wl.tokens(g, 25_000)
    cont = wl.continuation(g, sess, 27_000, 24_000)
    perm = g.permutation(NB).astype(np.int32)
    n = shape.blocks_for(25_000)
    assert n == 1563 and n * shape.bytes_per_block == 4_814_340_096
    bt, bt2 = np.ascontiguousarray(perm[:n]), np.ascontiguousarray(perm[n:2 * n])
    planes, kv, keep = _pool(shape, NB, 22)
    sums_before = _block_sums(planes, NB)
    strides = wl.dense_strides(shape, n, "PF")
    image = torch.zeros(n * shape.bytes_per_block + 4096, dtype=torch.uint8, pin_memory=True)
    image[-4096:] = 0xA5
    hl = tb.host_layout(strides, image.numel() - 4096)
    ctx = tb.Talaria(0, variant=variant)
    try:
        ctx.kv_offload(kv, bt, 0, n, image, hl)
        ctx.sync()
        assert int(ctx.get_counters().last_variant) == (tb.VARIANT_BOUNCE if variant == tb.VARIANT_AUTO else variant)
        assert torch.equal(_block_sums(planes, NB), sums_before)               # offload only reads the pool
        assert bool((image[-4096:] == 0xA5).all())
        _check_image_against_pool(image[:-4096], planes, shape, NB, bt, n, strides)
        _oracle_layers(image.numpy(), planes, shape, bt, n, strides, layers=(0, 31, 93))
        # match on the device, restore the matched prefix into NEW slots
        d_res = torch.zeros(4, dtype=torch.int64, device=DEV)
        d_hashes = torch.zeros(27_000 // 16, dtype=torch.int64, device=DEV)
        ctx.prefix_match(1, torch.from_numpy(cont).to(DEV), [0, 27_000], torch.from_numpy(sess).to(DEV),
                         [0, 25_000], None, 16, wl.HASH_SEED, d_hashes, d_res)
        ctx.sync()
        m, hc = orc.prefix_match(cont, sess, 16, wl.HASH_SEED)
        r = d_res.cpu().numpy()
        assert [int(r[0]), int(r[1]), int(r[2]), int(r[3])] == [24_000, 1_500, 24_000, 0] == \
            [m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree]
        assert np.array_equal(d_hashes.cpu().numpy().view(np.uint64), hc)
        nr = int(r[2]) // 16
        ctx.kv_restore(kv, bt2, 0, nr, image, hl)
        ctx.sync()
        _check_image_against_pool(image[:-4096], planes, shape, NB, bt2, nr, strides)
        _oracle_layers(image.numpy(), planes, shape, bt, n, strides, layers=(5, 60), restored_into=bt2, n_restore=nr)
        untouched = torch.ones(NB, dtype=torch.bool, device=DEV)
        untouched[torch.from_numpy(bt2[:nr].astype(np.int64)).to(DEV)] = False
        assert torch.equal(_block_sums(planes, NB)[:, untouched], sums_before[:, untouched])
    finally:
        ctx.destroy()


@pytest.fixture(scope="module")
def big_pinned():
    _need(host_gb=27, device_gb=80)
    t = torch.empty(20_218_380_288 + 4096, dtype=torch.uint8, pin_memory=True)
    yield t
    del t


@pytest.mark.parametrize("B,order", [(16, "PF"), (32, "LF")])
def test_config3_long_context_fragmented_restore_with_overlapped_offload(big_pinned, B, order):
    shape = wl.QWEN235 if B == 16 else wl.QWEN235_B32
    NB = 16_384 if B == 16 else 8_192
    n = shape.blocks_for(105_000)
    assert (n, n * shape.bytes_per_block) == ((6563, 20_215_300_096) if B == 16 else (3282, 20_218_380_288))
    g = wl.rng(3, B)
    planes, kv, keep = _pool(shape, NB, 30 + B)
    even = np.arange(0, NB, 2, dtype=np.int32)
    src = np.ascontiguousarray(g.permutation(even)[:n])                     # the session's current blocks
    n2 = shape.blocks_for(25_000)
    second = np.ascontiguousarray(g.permutation(np.setdiff1d(even, src))[:n2])   # another session, offloaded meanwhile
    dst = wl.isolated_table(g, NB, n)                                       # isolated single free blocks
    assert not np.any(np.diff(np.sort(dst)) == 1)
    strides = wl.dense_strides(shape, n, order)
    size = n * shape.bytes_per_block
    image = big_pinned[:size + 4096]
    image[size:] = 0x5A
    hl = tb.host_layout(strides, size)
    strides2 = wl.dense_strides(shape, n2, "PF")
    image2 = torch.zeros(n2 * shape.bytes_per_block, dtype=torch.uint8, pin_memory=True)
    hl2 = tb.host_layout(strides2, image2.numel())
    ctx = tb.Talaria(0)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    try:
        sums0 = _block_sums(planes, NB)
        ctx.kv_offload(kv, src, 0, n, image, hl)
        ctx.sync()
        _check_image_against_pool(image[:size], planes, shape, NB, src, n, strides)
        _oracle_layers(image.numpy(), planes, shape, src, n, strides, layers=(0, 93))
        # restore into the fragmented free list while the second session is checkpointed
        torch.cuda.synchronize()
        ctx.kv_restore(kv, dst, 0, n, image, hl, stream=sa)
        ctx.kv_offload(kv, second, 0, n2, image2, hl2, stream=sb)
        ctx.sync(sa)
        ctx.sync(sb)
        assert bool((image[size:] == 0x5A).all())
        _check_image_against_pool(image[:size], planes, shape, NB, dst, n, strides)
        _check_image_against_pool(image2, planes, shape, NB, second, n2, strides2)
        _oracle_layers(image.numpy(), planes, shape, src, n, strides, layers=(47,), restored_into=dst, n_restore=n)
        _oracle_layers(image2.numpy(), planes, shape, second, n2, strides2, layers=(12,))
        untouched = torch.ones(NB, dtype=torch.bool, device=DEV)
        untouched[torch.from_numpy(dst.astype(np.int64)).to(DEV)] = False
        assert torch.equal(_block_sums(planes, NB)[:, untouched], sums0[:, untouched])
    finally:
        ctx.destroy()
        del planes


def test_config5_weight_staging_with_concurrent_restore():
    _need(host_gb=8, device_gb=130)
    ws = wl.moe_weight_set()
    plan, span = wl.stage_plan(ws.sizes, 2 << 20)
    assert 58.9e9 < ws.total_bytes < 59.0e9
    g = wl.rng(5)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(55)
    staging = torch.empty(span, dtype=torch.uint8, device=DEV)
    for off in range(0, span, 1 << 30):
        m = min(1 << 30, span - off)
        staging[off:off + m].view(torch.int16).random_(generator=gen)
    slots = torch.zeros(span, dtype=torch.uint8, device=DEV)
    n = len(plan)
    dirty = g.uniform(size=n) < 0.01                                       # about 1 % of the chunks
    missing = (~dirty) & (g.uniform(size=n) < 0.002)
    from_host = np.nonzero(dirty | missing)[0]
    # authoritative host bytes only for the chunks that need them, packed back to back
    host_off = np.zeros(n, np.int64)
    at = 0
    for k in from_host:
        host_off[k] = at
        at += -(-plan[k][1] // 256) * 256
    host = torch.empty(max(at, 256), dtype=torch.uint8, pin_memory=True)
    host.numpy()[:] = g.integers(0, 256, size=host.numel(), dtype=np.uint8)
    arr = np.zeros(n, tb.COPY_DTYPE)
    for k, (off, nb, cid) in enumerate(plan):
        arr[k] = (0 if missing[k] else staging.data_ptr() + off,
                  host.data_ptr() + int(host_off[k]) if (dirty[k] or missing[k]) else 0,
                  slots.data_ptr() + off, nb, cid, 0)
    bitmap = np.packbits(dirty, bitorder="little")
    # the KV restore that runs next to it: one 25,000-token session
    shape, NB = wl.QWEN235, 2048
    nblk = shape.blocks_for(25_000)
    planes, kv, keep = _pool(shape, NB, 56)
    table = np.ascontiguousarray(g.permutation(NB)[:nblk].astype(np.int32))
    strides = wl.dense_strides(shape, nblk, "PF")
    image = torch.empty(nblk * shape.bytes_per_block, dtype=torch.uint8, pin_memory=True)
    for off in range(0, image.numel(), 1 << 30):                          # random fill via the device
        m = min(1 << 30, image.numel() - off)
        image[off:off + m].copy_(torch.empty(m // 8, dtype=torch.int64, device=DEV).random_(generator=gen).view(torch.uint8))
    hl = tb.host_layout(strides, image.numel())
    ctx = tb.Talaria(0)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    try:
        torch.cuda.synchronize()
        st = ctx.stage(arr, bitmap, stream=sa)
        ctx.kv_restore(kv, table, 0, nblk, image, hl, stream=sb)
        ctx.sync(sa)
        ctx.sync(sb)
        total = sum(nb for _, nb, _ in plan)
        h2d = int(sum(plan[k][1] for k in from_host))
        assert (st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks) == \
            (total - h2d, h2d, int(dirty.sum()), int(missing.sum()))
        # (b) every chunk: clean ones equal the staged bytes, dirty / missing ones the host bytes
        host_dev = host.to(DEV)
        prev = 0
        for k in list(from_host) + [n]:
            if k > prev:                                                    # a run of clean chunks
                lo, hi = plan[prev][0], plan[k - 1][0] + plan[k - 1][1]
                assert torch.equal(slots[lo:hi], staging[lo:hi]), (prev, k)
            if k < n:
                off, nb, _ = plan[k]
                assert torch.equal(slots[off:off + nb], host_dev[int(host_off[k]):int(host_off[k]) + nb]), k
            prev = k + 1
        # (a) the oracle on a window of the plan that holds clean, dirty and missing chunks
        lo_k = max(int(from_host[0]) - 3, 0)
        win = list(range(lo_k, min(lo_k + 24, n)))
        lo, hi = plan[win[0]][0], plan[win[-1]][0] + plan[win[-1]][1]
        st_np, host_np = staging[lo:hi].cpu().numpy(), host.numpy()
        o_slots = np.zeros(hi - lo, np.uint8)
        entries = [(None if missing[k] else plan[k][0] - lo, int(host_off[k]) if (dirty[k] or missing[k]) else None,
                    plan[k][0] - lo, plan[k][1], plan[k][2]) for k in win]
        orc.stage(st_np, host_np, o_slots, entries, bitmap)
        got = slots[lo:hi].cpu().numpy()
        for k in win:
            a, b = plan[k][0] - lo, plan[k][0] - lo + plan[k][1]
            assert np.array_equal(got[a:b], o_slots[a:b]), k
        _check_image_against_pool(image, planes, shape, NB, table, nblk, strides)
    finally:
        ctx.destroy()
