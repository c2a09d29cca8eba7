"""Host-side argument validation of the library, run without a GPU and compared with brute force
and with the oracle's O(n^2) definition of a valid stage plan (Sec. 4.4)."""
import itertools

import numpy as np

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl


def test_block_table_checks():
    assert tb.check_block_table([0, 5, 7], 8, True) == tb.OK
    assert tb.check_block_table([0, 8], 8, False) == tb.ERR_BAD_BLOCK_ID
    assert tb.check_block_table([0, -1], 8, False) == tb.ERR_BAD_BLOCK_ID
    assert tb.check_block_table([3, 1, 3], 8, False) == tb.OK
    assert tb.check_block_table([3, 1, 3], 8, True) == tb.ERR_DUP_BLOCK
    assert tb.check_block_table([], 8, True) == tb.OK
    g = wl.rng(960)
    for _ in range(200):
        nb = int(g.integers(1, 200))
        t = g.integers(0, nb, size=int(g.integers(0, 40)))
        want = tb.ERR_DUP_BLOCK if np.unique(t).size != t.size else tb.OK
        assert tb.check_block_table(t, nb, True) == want


def _chunk_intervals(shape, n, strides):
    C = shape.chunk_bytes
    return sorted((l * strides[0] + p * strides[1] + i * strides[2], C)
                  for l in range(shape.num_layers) for p in range(shape.num_planes) for i in range(n))


def test_dense_layouts_report_their_contiguous_runs():
    shape, n = wl.QWEN235, 1563
    C = shape.chunk_bytes
    size = n * shape.bytes_per_block
    assert tb.check_image_layout(shape, 4096, n, wl.dense_strides(shape, n, "PF"), size) == (tb.OK, size)
    assert tb.check_image_layout(shape, 4096, n, wl.dense_strides(shape, n, "LF"), size) == (tb.OK, size)
    assert tb.check_image_layout(shape, 4096, n, wl.dense_strides(shape, n, "PF"), size - 1)[0] == tb.ERR_EXTENT
    # a padded page-first image: runs are one block's fragments
    pitch = shape.bytes_per_block + 4096
    assert tb.check_image_layout(shape, 4096, n, (2 * C, C, pitch), n * pitch) == (tb.OK, shape.bytes_per_block)
    # layer-first image of a longer session: runs are one plane's n blocks
    big = wl.dense_strides(shape, 2 * n, "LF")
    assert tb.check_image_layout(shape, 4096, n, big, 2 * size) == (tb.OK, n * C)
    assert tb.check_image_layout(shape, 4096, 0, (0, 0, 0), 0) == (tb.OK, 0)


def test_layout_verdicts_against_brute_force_on_small_shapes():
    shape = wl.KvShape(3, 1, 2, 4, elt_bytes=2, num_planes=2)          # 16-byte chunks
    C, n = shape.chunk_bytes, 3
    cands = [0, C // 2, C, 2 * C, 3 * C, 4 * C, 6 * C, 7 * C, 12 * C, 13 * C, 18 * C]
    accepted = 0
    for strides in itertools.product(cands, repeat=3):
        iv = _chunk_intervals(shape, n, strides)
        overlap = any(a[0] + a[1] > b[0] for a, b in zip(iv, iv[1:]))
        extent = iv[-1][0] + C
        rc, run = tb.check_image_layout(shape, 8, n, strides, extent)
        if overlap:
            assert rc == tb.ERR_INVALID_ARG, strides              # never accept an image whose chunks collide
        if rc == tb.OK:
            accepted += 1
            assert not overlap
            assert tb.check_image_layout(shape, 8, n, strides, extent - 1)[0] == tb.ERR_EXTENT
            # the reported run really is contiguous and aligned in image order
            starts = [a for a, _ in iv]
            k = run // C
            assert run % C == 0 and len(starts) % k == 0
            for r in range(0, len(starts), k):
                assert all(starts[r + j] == starts[r] + j * C for j in range(k))
    assert accepted > 20


def test_stage_plan_verdicts_against_the_oracle_definition():
    g = wl.rng(961)
    buf = np.zeros(1 << 16, np.uint8)
    host = np.zeros(1 << 16, np.uint8)
    base, hbase = buf.ctypes.data, host.ctypes.data
    seen = {tb.OK: 0, tb.ERR_OVERLAP: 0}
    for trial in range(400):
        n = int(g.integers(1, 7))
        plan = np.zeros(n, tb.COPY_DTYPE)
        entries = []
        dirty = g.uniform(size=n) < 0.3
        for k in range(n):
            nb = int(g.integers(0, 3000))
            so, do = int(g.integers(0, 30000)), int(g.integers(30000 if trial % 2 else 0, 60000))
            missing = g.uniform() < 0.15
            plan[k] = (0 if missing else base + so, hbase + so, base + do, nb, k, 0)
            entries.append((None if missing else so, so, do, nb, k))
        bitmap = np.packbits(dirty, bitorder="little")
        rc, st = tb.check_stage_plan(plan, bitmap)
        valid = orc.stage_validate(buf, host, buf, entries, bitmap)
        assert rc == (tb.OK if valid else tb.ERR_OVERLAP), (trial, entries)
        seen[rc] += 1
        if valid:
            ost = orc.stage(buf, host, buf.copy(), entries, bitmap)
            assert (st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks) == \
                (ost.d2d_bytes, ost.h2d_bytes, ost.dirty_chunks, ost.missing_chunks)
    assert seen[tb.OK] > 30 and seen[tb.ERR_OVERLAP] > 30
    bad = np.zeros(1, tb.COPY_DTYPE); bad[0] = (0, 0, base, 16, 0, 0)
    assert tb.check_stage_plan(bad)[0] == tb.ERR_INVALID_ARG          # missing chunk without a host copy
    bad[0] = (base, 0, 0, 16, 0, 0)
    assert tb.check_stage_plan(bad)[0] == tb.ERR_INVALID_ARG          # no destination


def test_prefix_agreement_against_the_oracle():
    # App. B "Prefix agreement": pure host arithmetic, so it is checked here without a GPU
    g = wl.rng(962)
    for _ in range(300):
        R, nb = int(g.integers(1, 9)), int(g.integers(0, 14))
        hashes = np.tile(g.integers(0, 2**63, size=nb, dtype=np.uint64), (R, 1)) if nb else np.zeros((R, 0), np.uint64)
        committed = g.integers(0, nb + 1, size=R)
        for _ in range(int(g.integers(0, 3))):
            if nb:
                hashes[int(g.integers(0, R)), int(g.integers(0, nb))] ^= np.uint64(1)
        assert tb.Talaria.prefix_agree(committed, hashes) == orc.prefix_agree(committed, hashes)
