"""Pins for the oracle's block-table copies (Sec. 4.3: checkpoint aligned blocks
to pinned host slabs, restore into newly allocated device slots; App. C:
layer-first and page-first host layouts are two views of the same prefix)."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import workloads as wl

SHAPES = [wl.TINY, wl.KvShape(3, 1, 4, 8, elt_bytes=2), wl.KvShape(2, 3, 5, 6, elt_bytes=1, num_planes=1),
          wl.KvShape(2, 2, 2, 3, elt_bytes=4)]


def _oshape(s):
    return orc.KvShape(s.num_layers, s.num_kv_heads, s.block_tokens, s.head_dim, s.elt_bytes, s.num_planes)


def _pool(seed, shape, nb):
    g = wl.rng(300, seed)
    return [g.integers(0, 256, size=nb * shape.chunk_bytes, dtype=np.uint8)
            for _ in range(shape.num_layers * shape.num_planes)]


def _image_numpy(shape, planes, bt, order):
    """Independent route: numpy fancy indexing per plane."""
    L, P, C = shape.num_layers, shape.num_planes, shape.chunk_bytes
    g = np.stack([pl.reshape(-1, C)[bt] for pl in planes]).reshape(L, P, len(bt), C)
    if order == "PF":
        g = g.transpose(2, 0, 1, 3)
    return np.ascontiguousarray(g).reshape(-1)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("order", ["LF", "PF"])
def test_offload_elem_chunk_and_numpy_agree(shape, order):
    nb, n = 23, 9
    planes = _pool(1, shape, nb)
    bt = wl.disjoint_tables(wl.rng(301), nb, [n])[0]
    strides = wl.dense_strides(shape, n, order)
    size = n * shape.bytes_per_block
    a = np.full(size, 0xAA, np.uint8); b = np.full(size, 0x55, np.uint8)
    orc.kv_offload(_oshape(shape), planes, bt, 0, n, a, strides, form="elem")
    orc.kv_offload(_oshape(shape), planes, bt, 0, n, b, strides, form="chunk")
    want = _image_numpy(shape, planes, bt, order)
    assert np.array_equal(a, want) and np.array_equal(b, want)


def test_element_index_formula_against_4d_view():
    # the pool plane is [blocks, kv_heads, block_tokens, head_dim]; one element, one address
    shape = wl.KvShape(1, 3, 4, 5, elt_bytes=2, num_planes=1)
    nb = 6
    plane = np.arange(nb * shape.chunk_bytes // 2, dtype=np.uint16)
    view = plane.reshape(nb, 3, 4, 5)
    bt = np.array([4, 1], dtype=np.int32)
    img = np.zeros(2 * shape.chunk_bytes, np.uint8)
    orc.kv_offload(_oshape(shape), [plane.view(np.uint8)], bt, 0, 2, img, wl.dense_strides(shape, 2, "LF"), form="elem")
    got = img.view(np.uint16).reshape(2, 3, 4, 5)
    for i, b in enumerate(bt):
        for h in range(3):
            for t in range(4):
                for d in range(5):
                    assert got[i, h, t, d] == view[b, h, t, d]


@pytest.mark.parametrize("shape", SHAPES)
def test_lf_and_pf_images_are_permutations_of_each_other(shape):
    nb, n = 17, 7
    planes = _pool(2, shape, nb)
    bt = wl.disjoint_tables(wl.rng(302), nb, [n])[0]
    L, P, C = shape.num_layers, shape.num_planes, shape.chunk_bytes
    lf = np.zeros(n * shape.bytes_per_block, np.uint8); pf = np.zeros_like(lf)
    orc.kv_offload(_oshape(shape), planes, bt, 0, n, lf, wl.dense_strides(shape, n, "LF"))
    orc.kv_offload(_oshape(shape), planes, bt, 0, n, pf, wl.dense_strides(shape, n, "PF"))
    assert np.array_equal(lf.reshape(L, P, n, C).transpose(2, 0, 1, 3), pf.reshape(n, L, P, C))


@pytest.mark.parametrize("order", ["LF", "PF"])
@pytest.mark.parametrize("form", ["elem", "chunk"])
def test_round_trip_into_new_slots(order, form):
    shape, nb = wl.TINY, 64
    planes = _pool(3, shape, nb)
    before = [p.copy() for p in planes]
    g = wl.rng(303)
    bt = wl.disjoint_tables(g, nb, [19])[0]
    strides = wl.dense_strides(shape, 19, order)
    guard = 4096
    buf = np.full(19 * shape.bytes_per_block + 2 * guard, 0xC3, np.uint8)
    img = buf[guard:-guard]
    orc.kv_offload(_oshape(shape), planes, bt, 0, 19, img, strides, form=form)
    assert all(np.array_equal(a, b) for a, b in zip(planes, before))        # offload only reads the pool
    assert np.all(buf[:guard] == 0xC3) and np.all(buf[-guard:] == 0xC3)     # and stays inside the image
    bt2 = wl.disjoint_tables(g, nb, [19], exclude=bt)[0]                    # restore goes to NEW slots
    assert not set(bt.tolist()) & set(bt2.tolist())
    orc.kv_restore(_oshape(shape), planes, bt2, 0, 19, img, strides, form=form)
    C = shape.chunk_bytes
    touched = np.zeros(nb, bool); touched[bt2] = True
    for pl, old in zip(planes, before):
        now, was = pl.reshape(nb, C), old.reshape(nb, C)
        assert np.array_equal(now[bt2], was[bt])                            # every moved chunk, byte for byte
        assert np.array_equal(now[~touched], was[~touched])                 # everything else untouched


def test_restore_with_same_table_is_identity_and_identity_table_is_memcpy():
    shape, nb = wl.TINY, 32
    planes = _pool(4, shape, nb)
    before = [p.copy() for p in planes]
    bt = wl.disjoint_tables(wl.rng(304), nb, [10])[0]
    strides = wl.dense_strides(shape, 10, "PF")
    img = np.zeros(10 * shape.bytes_per_block, np.uint8)
    orc.kv_offload(_oshape(shape), planes, bt, 0, 10, img, strides)
    orc.kv_restore(_oshape(shape), planes, bt, 0, 10, img, strides)
    assert all(np.array_equal(a, b) for a, b in zip(planes, before))
    # identity table + layer-first image: each plane's first n blocks, back to back
    ident = np.arange(10, dtype=np.int32)
    lf = np.zeros_like(img)
    orc.kv_offload(_oshape(shape), planes, ident, 0, 10, lf, wl.dense_strides(shape, 10, "LF"))
    assert np.array_equal(lf, np.concatenate([p[:10 * shape.chunk_bytes] for p in planes]))


def test_sub_range_and_padded_strides():
    shape, nb = wl.KvShape(3, 2, 4, 8), 40
    planes = _pool(5, shape, nb)
    bt = wl.disjoint_tables(wl.rng(305), nb, [20])[0]
    C, L, P = shape.chunk_bytes, shape.num_layers, shape.num_planes
    first, n = 6, 9
    # padded page-first image: every chunk slot is C+32 bytes wide
    slot = C + 32
    strides = (P * slot, slot, L * P * slot)
    img = np.full(n * L * P * slot, 0x11, np.uint8)
    orc.kv_offload(_oshape(shape), planes, bt, first, n, img, strides)
    v = img.reshape(n, L, P, slot)
    for i in range(n):
        for l in range(L):
            for p in range(P):
                assert np.array_equal(v[i, l, p, :C], planes[l * P + p].reshape(nb, C)[bt[first + i]])
    assert np.all(v[..., C:] == 0x11)
    # the same blocks offloaded as a whole-table call agree on the overlap
    whole = np.zeros(20 * shape.bytes_per_block, np.uint8)
    orc.kv_offload(_oshape(shape), planes, bt, 0, 20, whole, wl.dense_strides(shape, 20, "PF"))
    assert np.array_equal(whole.reshape(20, L, P, C)[first:first + n], v[..., :C])


def test_bad_block_id_is_rejected_and_zero_blocks_is_a_no_op():
    shape, nb = wl.TINY, 8
    planes = _pool(6, shape, nb)
    img = np.zeros(2 * shape.bytes_per_block, np.uint8)
    for bad in (-1, nb):
        with pytest.raises(ValueError):
            orc.kv_offload(_oshape(shape), planes, np.array([0, bad], np.int32), 0, 2, img,
                           wl.dense_strides(shape, 2, "LF"))
    img = np.zeros(2 * shape.bytes_per_block, np.uint8)
    orc.kv_offload(_oshape(shape), planes, np.array([], np.int32), 0, 0, img, wl.dense_strides(shape, 0, "PF"))
    assert not img.any()


@pytest.mark.parametrize("shape", SHAPES)
def test_page_slabs_reduce_to_dense_page_first_and_follow_any_page_order(shape):
    nb, n = 29, 11
    planes = _pool(7, shape, nb)
    g = wl.rng(306)
    bt = wl.disjoint_tables(g, nb, [n])[0]
    slab = shape.bytes_per_block
    dense = np.zeros(n * slab, np.uint8)
    orc.kv_offload(_oshape(shape), planes, bt, 0, n, dense, wl.dense_strides(shape, n, "PF"))
    # consecutive pages = the dense page-first image
    pool = np.full(n * slab, 0x42, np.uint8)
    orc.kv_pages(_oshape(shape), planes, bt, 0, n, pool, np.arange(n) * slab, True)
    assert np.array_equal(pool, dense)
    # shuffled pages with gaps: page i sits where its offset says, everything else untouched
    order = g.permutation(2 * n)[:n]
    offs = order.astype(np.int64) * (slab + 16) + 8
    big = np.full(2 * n * (slab + 16) + 64, 0x42, np.uint8)
    orc.kv_pages(_oshape(shape), planes, bt, 0, n, big, offs, True)
    touched = np.zeros(big.size, bool)
    for i in range(n):
        assert np.array_equal(big[offs[i]:offs[i] + slab], dense[i * slab:(i + 1) * slab])
        touched[offs[i]:offs[i] + slab] = True
    assert np.all(big[~touched] == 0x42)
    # restore from the shuffled slabs into new blocks equals restore from the dense image
    bt2 = wl.disjoint_tables(g, nb, [n], exclude=bt)[0]
    a, b = [p.copy() for p in planes], [p.copy() for p in planes]
    orc.kv_pages(_oshape(shape), a, bt2, 0, n, big, offs, False)
    orc.kv_restore(_oshape(shape), b, bt2, 0, n, dense, wl.dense_strides(shape, n, "PF"))
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    with pytest.raises(ValueError):
        orc.kv_pages(_oshape(shape), planes, bt, 0, n, big, offs + big.size, True)
