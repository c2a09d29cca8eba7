"""Pins for the oracle's chained block hash (reading of Sec. 4.3 "cumulative
prefix hash" / App. B "at page boundaries").  The paper prints no hash value, so
the pins are mathematical: the published SplitMix64 sequence, the closed form
of the affine chain evaluated with Python big integers, the prefix property,
exhaustive injectivity on tiny alphabets and sensitivity to every kind of edit."""
import itertools
import os

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2607_17181_b200 import workloads as wl

M64 = (1 << 64) - 1
G = 0x9E3779B97F4A7C15
P = 0xD1342543DE82EF95
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _vectors():
    out = {}
    with open(os.path.join(GOLDEN, "splitmix64_vectors.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            seed, idx, val = line.split()
            out.setdefault(int(seed), {})[int(idx)] = int(val, 0)
    return out


def test_finaliser_matches_published_splitmix64_sequence():
    for seed, vals in _vectors().items():
        state = seed
        for idx in range(max(vals) + 1):
            state = (state + G) & M64
            assert orc.mix64(state) == vals[idx], (seed, idx)


def test_zero_block_digest_is_sum_of_splitmix64_outputs():
    v = _vectors()[0]
    for B in (1, 2, 3):
        want = sum(v[j] for j in range(B)) & M64
        assert orc.block_digest(np.zeros(B, dtype=np.int32)) == want


def test_single_token_digest_is_one_generator_step():
    # token t at position 0 enters as t + G: the SplitMix64 state one step after seed t
    assert orc.block_digest(np.array([1234567], dtype=np.int32)) == _vectors()[1234567][0]


def test_negative_token_is_hashed_as_its_uint32_pattern():
    assert orc.block_digest(np.array([-1], dtype=np.int32)) == orc.mix64(0xFFFFFFFF + G)
    assert orc.block_digest(np.array([-2**31], dtype=np.int32)) == orc.mix64(0x80000000 + G)


@pytest.mark.parametrize("B", [1, 4, 16, 32, 24])
def test_chain_closed_form_with_big_integers(B):
    g = wl.rng(101, B)
    T = 11 * B + 5
    tok = wl.tokens(g, T)
    seed = wl.HASH_SEED
    got = orc.block_hash(tok, B, seed)
    assert got.size == T // B
    dig = [orc.block_digest(tok[k * B:(k + 1) * B]) for k in range(T // B)]
    for k in range(T // B):
        s = seed * pow(P, k + 1) + sum(dig[i] * pow(P, k - i) for i in range(k + 1))
        assert int(got[k]) == orc.mix64(s & M64)


def test_digest_from_first_principles_python():
    # an independent evaluation of the per-block sum with Python integers
    tok = wl.tokens(wl.rng(102), 16)
    acc = 0
    for j, t in enumerate(tok.tolist()):
        acc += orc.mix64((t + G * (j + 1)) & M64)
    assert orc.block_digest(tok) == acc & M64


def test_prefix_property_and_partial_tail_ignored():
    tok = wl.tokens(wl.rng(103), 16 * 40 + 7)
    full = orc.block_hash(tok, 16, 7)
    assert full.size == 40
    for cut in (0, 1, 15, 16, 17, 16 * 20, 16 * 40, 16 * 40 + 6):
        h = orc.block_hash(tok[:cut], 16, 7)
        assert h.size == cut // 16
        assert np.array_equal(h, full[:cut // 16])


@pytest.mark.parametrize("B,T", [(1, 6), (2, 8), (4, 8)])
def test_exhaustive_injectivity_on_tiny_alphabet(B, T):
    # over every stream on {0,1,2}: hash_k equal  <=>  first (k+1)B tokens equal
    for seed in (0, wl.HASH_SEED):
        by_hash = [dict() for _ in range(T // B)]
        by_prefix = [dict() for _ in range(T // B)]
        for s in itertools.product((0, 1, 2), repeat=T):
            h = orc.block_hash(np.array(s, dtype=np.int32), B, seed)
            for k in range(T // B):
                pre = s[:(k + 1) * B]
                assert by_hash[k].setdefault(int(h[k]), pre) == pre
                assert by_prefix[k].setdefault(pre, int(h[k])) == int(h[k])
        for k in range(T // B):
            assert len(by_hash[k]) == 3 ** ((k + 1) * B)


def test_every_edit_changes_that_hash_and_all_later_ones():
    B, nb = 16, 12
    tok = wl.tokens(wl.rng(104), B * nb)
    base = orc.block_hash(tok, B, 5)

    def changed_from(other, k):
        assert np.array_equal(other[:k], base[:k])
        assert np.all(other[k:] != base[k:])

    t = tok.copy(); t[5 * B + 3] ^= 1
    changed_from(orc.block_hash(t, B, 5), 5)
    t = tok.copy(); a, b = 4 * B + 2, 4 * B + 9
    assert t[a] != t[b]; t[a], t[b] = t[b], t[a]
    changed_from(orc.block_hash(t, B, 5), 4)               # order inside a block matters
    t = tok.copy(); blk = t[2 * B:3 * B].copy(); t[2 * B:3 * B] = t[7 * B:8 * B]; t[7 * B:8 * B] = blk
    changed_from(orc.block_hash(t, B, 5), 2)               # order of blocks matters
    changed_from(orc.block_hash(tok, B, 6), 0)             # the model key matters
    # moving one token across a block boundary
    t = tok.copy(); t[3 * B - 1], t[3 * B] = t[3 * B], t[3 * B - 1]
    changed_from(orc.block_hash(t, B, 5), 2)


def test_position_weights_never_alias_for_32bit_tokens():
    # (token, position) pairs are injective inside a block: G*dj stays farther than 2^32
    # from 0 mod 2^64 for every position gap below 4096.
    for dj in range(1, 4096):
        d = (G * dj) & M64
        assert min(d, (1 << 64) - d) > (1 << 32)


def test_finaliser_is_a_bijection_so_equal_hashes_mean_equal_chain_states():
    # The block hash is the finaliser applied to the chain state.  Its inverse exists (undo the
    # xor-shifts, multiply by the inverses of the two odd constants), so two block hashes are equal
    # exactly when the chain states are -- which lets an implementation compare states, and lets it
    # skip hashing a stored stream over the prefix where the tokens are equal.
    def unshift(z, s):
        x = z
        for _ in range(64 // s + 1):
            x = z ^ (x >> s)
        return x

    inv1, inv2 = pow(0xBF58476D1CE4E5B9, -1, 1 << 64), pow(0x94D049BB133111EB, -1, 1 << 64)

    def unmix(h):
        z = unshift(h, 31)
        z = (z * inv2) & M64
        z = unshift(z, 27)
        z = (z * inv1) & M64
        return unshift(z, 30)

    g = wl.rng(77)
    for x in [0, 1, M64, 1 << 63] + [int(v) for v in g.integers(0, 1 << 63, size=2000, dtype=np.int64)]:
        assert unmix(orc.mix64(x)) == x
    # and at the level of the chain: streams equal up to a block give equal hashes up to that block,
    # and from the first different block on the hashes differ exactly where the states do
    B, seed = 16, 0x54414C41524941
    a = wl.tokens(g, 40 * B)
    b = a.copy()
    b[17 * B + 5] ^= 1
    ha, hb = orc.block_hash(a, B, seed), orc.block_hash(b, B, seed)
    assert np.array_equal(ha[:17], hb[:17]) and not np.any(ha[17:] == hb[17:])
    sa, sb = seed, seed
    for k in range(40):
        sa = (sa * P + orc.block_digest(a[k * B:(k + 1) * B])) & M64
        sb = (sb * P + orc.block_digest(b[k * B:(k + 1) * B])) & M64
        assert (sa == sb) == (int(ha[k]) == int(hb[k]))


def test_golden_config1_hashes():
    path = os.path.join(GOLDEN, "config1_hashes.txt")
    want = [int(ln, 16) for ln in open(path).read().splitlines() if ln.strip() and not ln.startswith("#")]
    from tests.golden.make_golden import config1_streams
    sess, cont = config1_streams()
    got = np.concatenate([orc.block_hash(sess, 16, wl.HASH_SEED), orc.block_hash(cont, 16, wl.HASH_SEED)])
    assert [int(x) for x in got] == want
