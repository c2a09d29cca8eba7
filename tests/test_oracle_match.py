"""Pins for the oracle's prefix match (App. A "Prefix reuse": longest common
prefix after tokenisation; Sec. 4.3: blocks keyed by cumulative hash; App. B
"Prefix agreement")."""
import itertools

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import workloads as wl

SEED = wl.HASH_SEED


def _lcp_numpy(a, b):
    n = min(a.size, b.size)
    ne = np.nonzero(a[:n] != b[:n])[0]
    return int(ne[0]) if ne.size else n


def test_lcp_brute_force_all_tiny_pairs():
    streams = [np.array(s, dtype=np.int32) for n in range(0, 5) for s in itertools.product((0, 1), repeat=n)]
    for a in streams:
        for b in streams:
            k = 0
            while k < min(a.size, b.size) and a[k] == b[k]:
                k += 1
            assert orc.lcp_tokens(a, b) == k == _lcp_numpy(a, b)


def test_lcp_against_numpy_on_random_streams():
    g = wl.rng(201)
    for _ in range(50):
        ta, tb = int(g.integers(0, 3000)), int(g.integers(0, 3000))
        a = wl.tokens(g, ta)
        shared = int(g.integers(0, min(ta, tb) + 1))
        b = wl.continuation(g, a, tb, shared)
        want = shared if shared < min(ta, tb) else min(ta, tb)
        assert orc.lcp_tokens(b, a) == _lcp_numpy(b, a) == want


def test_config1_constructed_answer():
    g = wl.rng(1)
    wl.tokens(g, 300)
    sess = wl.tokens(g, 500)
    cont = wl.continuation(g, sess, 560, 350)
    m, hc = orc.prefix_match(cont, sess, 16, SEED)
    assert (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree) == (350, 21, 336, 0)
    assert hc.size == 35


def test_config2_constructed_answer():
    g = wl.rng(2)
    sess = wl.tokens(g, 25_000)
    cont = wl.continuation(g, sess, 27_000, 24_000)
    m, hc = orc.prefix_match(cont, sess, 16, SEED)
    assert (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree) == (24_000, 1_500, 24_000, 0)
    assert hc.size == 1_687
    m32, _ = orc.prefix_match(cont, sess, 32, SEED)
    assert (m32.lcp_tokens, m32.matched_blocks, m32.reusable_tokens) == (24_000, 750, 24_000)


@pytest.mark.parametrize("B", [1, 3, 16, 32])
def test_special_cases(B):
    g = wl.rng(202, B)
    s = wl.tokens(g, 10 * B + B // 2)
    # identical streams
    m, _ = orc.prefix_match(s, s, B, SEED)
    assert (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree) == (s.size, 10, 10 * B, 0)
    # empty on either side
    e = np.zeros(0, dtype=np.int32)
    for a, b in ((e, s), (s, e), (e, e)):
        m, h = orc.prefix_match(a, b, B, SEED)
        assert (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree) == (0, 0, 0, 0)
        assert h.size == a.size // B
    # mismatch at token 0
    c = wl.continuation(g, s, s.size, 0)
    m, _ = orc.prefix_match(c, s, B, SEED)
    assert (m.lcp_tokens, m.matched_blocks, m.reusable_tokens) == (0, 0, 0)
    # mismatch exactly on a block boundary, one before and one after
    for split, blocks in ((4 * B, 4), (4 * B - 1, 3), (4 * B + 1, 4 if B > 1 else 5)):
        c = wl.continuation(g, s, s.size + 7, split)
        m, _ = orc.prefix_match(c, s, B, SEED)
        assert m.lcp_tokens == split
        assert m.matched_blocks == split // B == blocks
        assert m.reusable_tokens == (split // B) * B
        assert m.hash_token_disagree == 0
    # continuation shorter than the stored stream, fully contained
    c = s[: 6 * B + 1].copy()
    m, h = orc.prefix_match(c, s, B, SEED)
    assert (m.lcp_tokens, m.matched_blocks, m.reusable_tokens) == (c.size, c.size // B, (c.size // B) * B)
    assert h.size == c.size // B


def test_matched_blocks_agree_with_tokens_on_random_pairs():
    g = wl.rng(203)
    for _ in range(40):
        B = int(g.choice([1, 2, 8, 16, 32, 24]))
        ts, tc = int(g.integers(0, 2500)), int(g.integers(0, 2500))
        s = wl.tokens(g, ts)
        shared = int(g.integers(0, min(ts, tc) + 1))
        c = wl.continuation(g, s, tc, shared)
        m, hc = orc.prefix_match(c, s, B, SEED)
        lcp = _lcp_numpy(c, s)
        assert m.lcp_tokens == lcp
        assert m.matched_blocks == min(lcp // B, tc // B, ts // B)
        assert m.reusable_tokens == B * m.matched_blocks
        assert m.hash_token_disagree == 0
        assert np.array_equal(hc, orc.block_hash(c, B, SEED))


def test_stored_hashes_given_equal_derived_and_corruption_is_reported():
    g = wl.rng(204)
    s = wl.tokens(g, 1000)
    c = wl.continuation(g, s, 1200, 800)
    hs = orc.block_hash(s, 16, SEED)
    m0, h0 = orc.prefix_match(c, s, 16, SEED)
    m1, h1 = orc.prefix_match(c, s, 16, SEED, sess_hashes=hs)
    assert m0 == m1 and np.array_equal(h0, h1)
    bad = hs.copy(); bad[20] ^= np.uint64(1)
    m2, _ = orc.prefix_match(c, s, 16, SEED, sess_hashes=bad)
    assert m2.lcp_tokens == 800 and m2.matched_blocks == 20
    assert m2.reusable_tokens == 320 and m2.hash_token_disagree == 1
    # a different model key never matches stored hashes of another key
    m3, _ = orc.prefix_match(c, s, 16, SEED + 1, sess_hashes=hs)
    assert m3.matched_blocks == 0 and m3.reusable_tokens == 0 and m3.hash_token_disagree == 1


def test_prefix_agreement_brute_force():
    g = wl.rng(205)
    for _ in range(200):
        R = int(g.integers(1, 9))
        nb = int(g.integers(0, 12))
        base = g.integers(0, 2**63, size=nb, dtype=np.uint64)
        hashes = np.tile(base, (R, 1)) if nb else np.zeros((R, 0), dtype=np.uint64)
        committed = g.integers(0, nb + 1, size=R)
        if nb and g.uniform() < 0.7:
            r, k = int(g.integers(0, R)), int(g.integers(0, nb))
            hashes[r, k] ^= np.uint64(1)
        want = 0
        while want < int(committed.min()) and all(hashes[r, want] == hashes[0, want] for r in range(R)):
            want += 1
        assert orc.prefix_agree(committed, hashes) == want
    # one rank: everything it committed is agreed
    assert orc.prefix_agree([5], np.arange(8, dtype=np.uint64)[None, :]) == 5
