"""The stable-address HBM layout (Sec. 4.2) and its staging surface (Sec. 4.4): host arithmetic,
no GPU.  The C implementation and the plain-Python definition in the oracle are both held to
what the paper and arithmetic fix, by brute force over byte ranges: regions never overlap, the
pool is as large as the gap allows, every address is the same before and after a switch, blocks
come lowest first and never from rows under a staging write, staged chunks sit in free tail rows
outside the next model's weights, and an allocation dirties exactly the staged chunks whose
bytes it takes (checked against the interval definition of talaria_mark_dirty).  Then the two
are compared with each other on random scenarios."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl

BASE = 0x7F0000000000          # only ever used as a number


def _models(g, n):
    out = []
    for _ in range(n):
        Cb = int(g.choice([256, 512, 4096]))
        out.append((int(g.integers(0, 60_000)), int(g.integers(0, 9_000)), int(g.integers(1, 4)), int(g.integers(1, 3)), Cb))
    return out


def _ranges_disjoint(ranges):
    r = sorted((a, a + n) for a, n in ranges if n > 0)
    return all(r[k][1] <= r[k + 1][0] for k in range(len(r) - 1))


def test_worked_example():
    # S = 1 MiB, A = 256; weights 1000 B, runtime 500 B, 2 layers x 2 planes of 256-byte rows:
    # K = 1024, R = floor(1048076 / 256) * 256 = 4094 * 256 = 1048064, NB = floor((1048064 - 1024) / 1024) = 1022
    b = tb.Bump(BASE, 1 << 20, [(1000, 500, 2, 2, 256)])
    v, planes = b.view(0)
    assert (v.weights_base, v.weights_bytes) == (BASE, 1000)
    assert (v.runtime_base - BASE, v.runtime_bytes) == (1048064, 500)
    assert (v.kv_base - BASE, v.num_blocks, v.kv_bytes) == (1024, 1022, 4 * 1022 * 256)
    assert [p - BASE for p in planes] == [1024 + k * 1022 * 256 for k in range(4)]
    o = orc.BumpLayout(1 << 20, 256, [(1000, 500, 2, 2, 256)]).view(0)
    assert (o["kv"], o["runtime"], o["num_blocks"]) == ((1024, 4 * 1022 * 256), (1048064, 500), 1022)
    with pytest.raises(tb.TalariaError) as e:                      # no room for a single block
        tb.Bump(BASE, 4096, [(2000, 1500, 2, 2, 256)])
    assert e.value.status == tb.ERR_EXTENT
    for bad in ((BASE + 8, 1 << 20, [(0, 0, 1, 1, 256)], 256), (BASE, 1 << 20, [(0, 0, 1, 1, 100)], 256),
                (BASE, 1 << 20, [(0, 0, 1, 1, 256)], 96)):
        with pytest.raises(tb.TalariaError) as e:
            tb.Bump(bad[0], bad[1], bad[2], align=bad[3])
        assert e.value.status == tb.ERR_INVALID_ARG


@pytest.mark.parametrize("seed", range(6))
def test_regions_never_overlap_and_addresses_survive_switches(seed):
    g = wl.rng(700, seed)
    S, A = int(g.integers(200_000, 400_000)) // 256 * 256, 256
    models = _models(g, 3)
    b = tb.Bump(BASE, S, models, align=A)
    o = orc.BumpLayout(S, A, models)
    first = {}
    for m in list(range(3)) * 3 + [2, 0, 1, 1, 0]:                 # activate in changing orders
        av = b.activate(m)
        v, planes = b.view(m)
        W, Rt, L, P, Cb = models[m]
        got = (v.weights_base - BASE, v.weights_bytes, v.kv_base - BASE, v.kv_bytes, v.runtime_base - BASE,
               v.runtime_bytes, v.num_blocks, tuple(p - BASE for p in planes))
        assert (av.kv_base, av.num_blocks, av.runtime_base) == (v.kv_base, v.num_blocks, v.runtime_base)
        assert first.setdefault(m, got) == got                     # the pointer check of Sec. 4.2 always passes
        NB = v.num_blocks
        regions = [(got[0], W), (got[4], Rt)] + [(p, NB * Cb) for p in got[7]]
        assert _ranges_disjoint(regions) and all(0 <= a and a + n <= S for a, n in regions)
        assert got[2] % A == 0 and got[4] % A == 0 and all(p % A == 0 for p in got[7])
        assert got[2] >= W and got[2] - W < A                      # the pool starts right above the weights
        assert got[7][-1] + NB * Cb <= got[4] < got[7][-1] + NB * Cb + L * P * Cb + A    # ... and fills the gap
        ov = o.view(m)
        assert (ov["weights"], ov["runtime"], ov["kv"], ov["num_blocks"], tuple(ov["planes"])) == \
            ((got[0], got[1]), (got[4], got[5]), (got[2], got[3]), got[6], got[7])
        assert b.free_count() == NB


def _bitmap(ids, n):
    bm = np.zeros((n + 7) // 8 or 1, np.uint8)
    for c in ids:
        bm[c >> 3] |= 1 << (c & 7)
    return bm


def _bits(bm, n):
    return {c for c in range(n) if (bm[c >> 3] >> (c & 7)) & 1}


@pytest.mark.parametrize("seed", range(8))
def test_allocation_staging_and_dirty_marking_against_brute_force_and_oracle(seed):
    g = wl.rng(701, seed)
    A = 256
    models = _models(g, 2)
    S = int(g.integers(300_000, 600_000)) // 256 * 256
    b = tb.Bump(BASE, S, models, align=A)
    o = orc.BumpLayout(S, A, models)
    cur, nxt = (0, 1) if seed % 2 == 0 else (1, 0)
    b.activate(cur); o.activate(cur)
    v, planes = b.view(cur)
    NB, Cb, LP = v.num_blocks, models[cur][4], models[cur][2] * models[cur][3]
    planes = [p - BASE for p in planes]
    live = []
    # ---- some traffic before staging: allocations come lowest first, frees make holes --------
    for _ in range(4):
        n = int(g.integers(0, max(1, NB // 6)))
        ids, _ = b.alloc_blocks(n)
        oids, _ = o.alloc_blocks(n)
        assert list(ids) == oids == sorted(set(range(NB)) - set(live))[:n]
        live += oids
        drop = [x for x in live if g.uniform() < 0.3]
        if drop:
            b.free_blocks(drop); o.free_blocks(drop)
            live = [x for x in live if x not in drop]
    with pytest.raises(tb.TalariaError):
        b.free_blocks([sorted(set(range(NB)) - set(live))[0]])      # already free
    # ---- placement of the next model's chunks --------------------------------------------------
    chunk = int(g.choice([Cb, 3 * Cb, 2 * Cb + 100, 5 * Cb]))
    W2 = models[nxt][0]
    plan, placed = b.stage_place(nxt, chunk, host_weights=0x10000000)
    oplan = o.stage_place(nxt, chunk)
    n_chunks = -(-W2 // chunk)
    assert plan.size == n_chunks == len(oplan)
    r = -(-chunk // Cb)
    lim = -(-W2 // A) * A
    got_src = [None if e["src_dev"] == 0 else int(e["src_dev"]) - BASE for e in plan]
    assert got_src == [p[0] for p in oplan] and placed == sum(p[0] is not None for p in oplan)
    assert [int(e["dst_dev"]) - BASE for e in plan] == [j * chunk for j in range(n_chunks)]
    assert [int(e["bytes"]) for e in plan] == [min(chunk, W2 - j * chunk) for j in range(n_chunks)]
    assert [int(e["src_host"]) for e in plan] == [0x10000000 + j * chunk for j in range(n_chunks)]
    assert [int(e["chunk_id"]) for e in plan] == list(range(n_chunks))
    staged_ranges = [(s, r * Cb) for s in got_src if s is not None]
    assert _ranges_disjoint(staged_ranges)
    for s in (x for x in got_src if x is not None):
        k = max(i for i in range(LP) if planes[i] <= s)
        row0 = (s - planes[k]) // Cb
        assert (s - planes[k]) % Cb == 0 and row0 + r <= NB and (NB - row0) % r == 0      # a whole tail slot of one plane
        assert all(x not in live for x in range(row0, row0 + r))                         # its rows were free
        assert s >= lim                                                                  # outside the next weights region
    if placed < n_chunks:                                            # chunks are left out only when no usable slot remains
        assert b.staging_slack(nxt, chunk) == 0
    assert b.staging_slack(nxt, chunk) == o.staging_slack(nxt, chunk)
    assert all(s is not None for s in got_src[:placed]) and all(s is None for s in got_src[placed:])
    # ---- a staging write in flight: its rows are passed over ---------------------------------------
    staged = {c for c in range(placed) if g.uniform() < 0.8}
    dirty_bm, staged_bm = _bitmap([], n_chunks), _bitmap(staged, n_chunks)
    odirty = set()
    locked = [c for c in range(placed) if g.uniform() < 0.2][:3]
    for c in locked:
        b.lock_chunk(c, True); o.locked.add(c)
    locked_rows = set()
    for c in locked:
        k = max(i for i in range(LP) if planes[i] <= got_src[c])
        row0 = (got_src[c] - planes[k]) // Cb
        locked_rows |= set(range(row0, row0 + r))
    # ---- allocations that reach into the tails: dirty marking ---------------------------------------
    for step in range(6):
        free_now = sorted(set(range(NB)) - set(live) - locked_rows)
        n = min(len(free_now), int(g.integers(0, max(2, NB // 3))))
        before = dirty_bm.copy()
        ids, nd = b.alloc_blocks(n, staged_bm, dirty_bm)
        oids, onew = o.alloc_blocks(n, staged, odirty)
        assert list(ids) == oids == free_now[:n]                     # lowest first, never a locked row
        live += oids
        # the interval definition: every row of every plane the allocation took, through talaria_mark_dirty
        want = before.copy()
        changed = 0
        for bid in oids:
            for k in range(LP):
                changed += tb.Talaria.mark_dirty(plan, BASE + planes[k] + bid * Cb, Cb, staged_bm, want)
        assert np.array_equal(dirty_bm, want) and nd == changed == len(onew)
        assert _bits(dirty_bm, n_chunks) == odirty
        if step == 2:
            for c in locked:
                b.lock_chunk(c, False); o.locked.discard(c)
            locked_rows = set()
    with pytest.raises(tb.TalariaError) as e:
        b.alloc_blocks(NB + 1)
    assert e.value.status == tb.ERR_NO_MEMORY
    # ---- the switch: addresses of the next model are what they always were ------------------------------
    v2_before, p2_before = b.view(nxt)
    b.activate(nxt); o.activate(nxt)
    v2, p2 = b.view(nxt)
    assert (v2.weights_base, v2.kv_base, v2.runtime_base, v2.num_blocks, p2) == \
        (v2_before.weights_base, v2_before.kv_base, v2_before.runtime_base, v2_before.num_blocks, p2_before)
    assert b.free_count() == v2.num_blocks
