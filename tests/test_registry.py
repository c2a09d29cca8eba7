"""The host-side page registry against its dict definition (Sec. 4.3: blocks keyed by the
cumulative prefix hash).  Needs no GPU."""
import numpy as np

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl


def test_random_operation_sequences_match_the_dict_definition():
    g = wl.rng(950)
    universe = g.integers(0, 2**63, size=4000, dtype=np.uint64) * np.uint64(2) + g.integers(0, 2, size=4000, dtype=np.uint64)
    universe[:8] = np.array([0, 1, 2**64 - 1, 2**63, 16, 32, 48, 64], dtype=np.uint64)   # awkward keys, clustered low bits
    reg, ref = tb.Registry(4), orc.Registry()
    for step in range(400):
        op = g.uniform()
        idx = g.integers(0, universe.size, size=int(g.integers(0, 60)))
        keys = universe[idx]
        if op < 0.5:
            offs = g.integers(0, 2**40, size=keys.size).astype(np.int64)
            assert reg.insert(keys, offs) == ref.insert(keys, offs)
        elif op < 0.75:
            assert reg.erase(keys) == ref.erase(keys)
        else:
            k1, o1 = reg.lookup_prefix(keys)
            k2, o2 = ref.lookup_prefix(keys)
            assert k1 == k2 and np.array_equal(o1, o2)
        assert len(reg) == len(ref)
    # every key, one by one
    for h in universe[:500]:
        k1, o1 = reg.lookup_prefix([h]); k2, o2 = ref.lookup_prefix([h])
        assert k1 == k2 and np.array_equal(o1, o2)
    reg.destroy()


def test_longest_restorable_prefix_of_a_returning_stream():
    # a stored session's chained hashes are registered; a continuation sharing 21 blocks finds 21 pages
    g = wl.rng(1)
    wl.tokens(g, 300)
    sess = wl.tokens(g, 500)
    cont = wl.continuation(g, sess, 560, 350)
    hs, hc = orc.block_hash(sess, 16, wl.HASH_SEED), orc.block_hash(cont, 16, wl.HASH_SEED)
    reg = tb.Registry()
    assert reg.insert(hs, np.arange(hs.size) * 1000) == 31
    k, offs = reg.lookup_prefix(hc)
    assert k == 21 and np.array_equal(offs, np.arange(21) * 1000)
    assert reg.insert(hs[:5], np.full(5, 7)) == 0                  # first wins
    assert np.array_equal(reg.lookup_prefix(hc)[1], np.arange(21) * 1000)
    assert reg.erase(hs[10:12]) == 2                               # an evicted page cuts the prefix there
    assert reg.lookup_prefix(hc)[0] == 10
    assert reg.lookup_prefix(orc.block_hash(cont, 16, wl.HASH_SEED + 1))[0] == 0   # another model key shares nothing
    assert reg.lookup_prefix(np.zeros(0, np.uint64))[0] == 0
