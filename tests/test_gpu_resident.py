"""GPU parity: prefix match against streams that live on the device (Sec. 4.3: the instance keeps a
session's state between its calls; App. A: the new prompt is compared with what the session held).
Every record against the oracle's plain definition; the device arrays byte for byte."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl

pytestmark = pytest.mark.gpu
SEED = wl.HASH_SEED
FILL_T, FILL_H = -7, -3          # what untouched elements of the two arrays hold


class Arena:
    """The caller's side of the call: one token array and one hash array on the device, two places
    per session (the stored stream and the one the next prompt goes to), host mirrors of both."""

    def __init__(self, n_sessions, max_tokens, B, odd=0):
        self.B = B
        self.tok_stride = max_tokens + 5 + odd               # places are not 16-byte aligned on purpose
        self.hash_stride = max_tokens // B + 3
        self.d_tokens = torch.full((2 * n_sessions * self.tok_stride + 8,), FILL_T, dtype=torch.int32, device="cuda")
        self.d_hashes = torch.full((2 * n_sessions * self.hash_stride + 8,), FILL_H, dtype=torch.int64, device="cuda")
        self.m_tokens = np.full(self.d_tokens.numel(), FILL_T, np.int32)
        self.m_hashes = np.full(self.d_hashes.numel(), FILL_H, np.int64).view(np.uint64)
        self.side = [0] * n_sessions                         # which place holds the stored stream
        self.stored = [np.zeros(0, np.int32) for _ in range(n_sessions)]

    def slots(self, s, side):
        return 3 + (2 * s + side) * self.tok_stride, 1 + (2 * s + side) * self.hash_stride

    def pair(self, s, cont, derive=False):
        ct, ch = self.slots(s, self.side[s] ^ 1)
        st, sh = self.slots(s, self.side[s])
        return (cont, ct, ch, st, self.stored[s].size, -1 if derive else sh)

    def commit(self, s, cont, seed):
        ct, ch = self.slots(s, self.side[s] ^ 1)
        self.m_tokens[ct:ct + cont.size] = cont
        h = orc.block_hash(cont, self.B, seed)
        self.m_hashes[ch:ch + h.size] = h
        self.side[s] ^= 1
        self.stored[s] = cont

    def check(self):
        assert np.array_equal(self.d_tokens.cpu().numpy(), self.m_tokens)
        assert np.array_equal(self.d_hashes.cpu().numpy().view(np.uint64), self.m_hashes)


def _expect(res, q, cont, stored, B, seed):
    m, _ = orc.prefix_match(cont, stored, B, seed)
    r = res[q]
    assert (int(r["lcp_tokens"]), int(r["matched_blocks"]), int(r["reusable_tokens"]), int(r["hash_token_disagree"])) == \
        (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree), q


@pytest.mark.parametrize("B,derive", [(16, False), (16, True), (32, False), (24, False), (8, True)])
def test_sessions_over_several_turns(B, derive):
    """Three sessions, five turns, all sessions matched in one call per turn: turn 0 finds nothing
    stored, later turns match against what the previous turn left on the device."""
    g = wl.rng(1201, 2 * B + int(derive))
    ctx = tb.Talaria(0)
    try:
        n = 3
        arena = Arena(n, 9000, B, odd=B % 3)
        for turn in range(5):
            conts = []
            for s in range(n):
                prev = arena.stored[s]
                T = int(g.integers(1, 9000)) if turn else int(g.integers(0, 4000))
                shared = 0 if prev.size == 0 else int(g.integers(0, min(prev.size, T) + 1))
                if turn == 3 and s == 1:
                    shared = min(prev.size, T)              # one stream is a prefix of the other
                conts.append(wl.continuation(g, prev, T, shared) if prev.size else wl.tokens(g, T))
            res = np.zeros(n, tb.MATCH_DTYPE)
            ctx.prefix_match_resident([arena.pair(s, conts[s], derive) for s in range(n)], arena.d_tokens, arena.d_hashes,
                                      B, SEED, res)
            for s in range(n):
                _expect(res, s, conts[s], arena.stored[s], B, SEED)
                arena.commit(s, conts[s], SEED)
            arena.check()
    finally:
        ctx.destroy()


@pytest.mark.parametrize("n", [12, 160])
def test_many_sessions_in_one_call(n):
    """More pairs than travel in the kernel parameters (12) and at least one per SM (160): the batch
    kernels read the same places."""
    g = wl.rng(1202, n)
    B = 16
    ctx = tb.Talaria(0)
    try:
        arena = Arena(n, 3000, B)
        for turn in range(3):
            conts = []
            for s in range(n):
                prev = arena.stored[s]
                T = int(g.integers(0, 3000))
                conts.append(wl.continuation(g, prev, T, int(g.integers(0, min(prev.size, T) + 1))) if prev.size
                             else wl.tokens(g, T))
            res = np.zeros(n, tb.MATCH_DTYPE)
            ctx.prefix_match_resident([arena.pair(s, conts[s]) for s in range(n)], arena.d_tokens, arena.d_hashes, B, SEED, res)
            for s in range(n):
                _expect(res, s, conts[s], arena.stored[s], B, SEED)
                arena.commit(s, conts[s], SEED)
            arena.check()
    finally:
        ctx.destroy()


@pytest.mark.parametrize("case", range(24))
def test_random_sessions(case):
    """Random block size (powers of two and others), number of sessions (every kernel route), stream
    lengths including empty ones, alignment of the places, stored or derived hashes."""
    g = wl.rng(1206, case)
    B = int(g.choice([1, 3, 4, 8, 16, 24, 32, 64]))
    n = int(g.choice([1, 2, 5, 8, 9, 20, 150, 200]))
    longest = int(g.choice([200, 3000, 40000])) if n < 50 else int(g.choice([200, 3000]))
    derive = bool(g.uniform() < 0.4)
    ctx = tb.Talaria(0, host_match_bytes=2 << 20)
    try:
        arena = Arena(n, longest, B, odd=int(g.integers(0, 4)))
        for turn in range(3):
            conts = []
            for s in range(n):
                prev = arena.stored[s]
                T = int(g.integers(0, longest + 1)) if g.uniform() < 0.9 else 0
                shared = int(g.integers(0, min(prev.size, T) + 1)) if g.uniform() < 0.8 else min(prev.size, T)
                conts.append(wl.continuation(g, prev, T, shared) if prev.size else wl.tokens(g, T))
            res = np.zeros(n, tb.MATCH_DTYPE)
            ctx.prefix_match_resident([arena.pair(s, conts[s], derive) for s in range(n)], arena.d_tokens, arena.d_hashes,
                                      B, SEED, res)
            for s in range(n):
                _expect(res, s, conts[s], arena.stored[s], B, SEED)
                arena.commit(s, conts[s], SEED)
            arena.check()
    finally:
        ctx.destroy()


def test_prompts_larger_than_the_staging_go_in_several_rounds():
    g = wl.rng(1203)
    B = 16
    ctx = tb.Talaria(0, host_match_bytes=1 << 20)            # room for about 262,000 tokens per round
    try:
        n = 6
        arena = Arena(n, 120_000, B)
        for turn in range(2):
            conts = []
            for s in range(n):
                prev = arena.stored[s]
                T = int(g.integers(90_000, 120_000))
                conts.append(wl.continuation(g, prev, T, int(g.integers(0, min(prev.size, T) + 1))) if prev.size
                             else wl.tokens(g, T))
            before = ctx.get_counters().kernel_launches
            res = np.zeros(n, tb.MATCH_DTYPE)
            ctx.prefix_match_resident([arena.pair(s, conts[s]) for s in range(n)], arena.d_tokens, arena.d_hashes, B, SEED, res)
            assert ctx.get_counters().kernel_launches - before >= 2        # really several rounds
            for s in range(n):
                _expect(res, s, conts[s], arena.stored[s], B, SEED)
                arena.commit(s, conts[s], SEED)
            arena.check()
    finally:
        ctx.destroy()


def test_bad_calls_are_rejected_before_anything_moves():
    g = wl.rng(1204)
    B = 16
    ctx = tb.Talaria(0, host_match_bytes=1 << 20)
    try:
        arena = Arena(2, 2000, B)
        first = [wl.tokens(g, 1500), wl.tokens(g, 1700)]
        res = np.zeros(2, tb.MATCH_DTYPE)
        ctx.prefix_match_resident([arena.pair(s, first[s]) for s in range(2)], arena.d_tokens, arena.d_hashes, B, SEED, res)
        for s in range(2):
            arena.commit(s, first[s], SEED)
        arena.check()
        cont = [wl.continuation(g, first[s], 1800, 900) for s in range(2)]
        good = [arena.pair(s, cont[s]) for s in range(2)]
        launches = ctx.get_counters().kernel_launches

        def rejected(pairs, code, d_tokens=None, d_hashes=None):
            with pytest.raises(tb.TalariaError) as e:
                ctx.prefix_match_resident(pairs, arena.d_tokens if d_tokens is None else d_tokens,
                                          arena.d_hashes if d_hashes is None else d_hashes, B, SEED, res)
            assert e.value.status == code
            assert ctx.get_counters().kernel_launches == launches
            arena.check()

        c, ct, ch, st, n_st, sh = good[0]
        rejected([(c, st + 100, ch, st, n_st, sh), good[1]], tb.ERR_OVERLAP)               # prompt onto its own stored stream
        rejected([good[0], (cont[1], ct + 8, good[1][2], *good[1][3:])], tb.ERR_OVERLAP)    # two prompts onto each other
        rejected([(c, ct, sh, st, n_st, sh), good[1]], tb.ERR_OVERLAP)                      # hashes onto the stored hashes
        rejected([(c, arena.d_tokens.numel() - 100, ch, st, n_st, sh), good[1]], tb.ERR_EXTENT)
        rejected([(c, ct, arena.d_hashes.numel() - 3, st, n_st, sh), good[1]], tb.ERR_EXTENT)
        rejected([(c, ct, ch, st, arena.d_tokens.numel(), sh), good[1]], tb.ERR_EXTENT)
        rejected([(c, ct, ch, st, n_st, -1), good[1]], tb.ERR_INVALID_ARG)                  # one derived, one stored
        rejected([(wl.tokens(g, 300_000), ct, ch, st, n_st, sh)], tb.ERR_EXTENT)            # larger than the arena place
        # a view that claims more elements than its allocation holds
        torch.cuda.empty_cache()
        small = torch.zeros(4096, dtype=torch.int32, device="cuda")

        class Lying:
            def data_ptr(self):
                return small.data_ptr()

            def numel(self):
                return 1 << 28

        rejected([(c, 0, ch, 2048, 0, -1)], tb.ERR_EXTENT, d_tokens=Lying())
        # the good call still goes through
        ctx.prefix_match_resident(good, arena.d_tokens, arena.d_hashes, B, SEED, res)
        for s in range(2):
            _expect(res, s, cont[s], first[s], B, SEED)
            arena.commit(s, cont[s], SEED)
        arena.check()
    finally:
        ctx.destroy()


def test_prompt_larger_than_the_staging_is_refused():
    g = wl.rng(1205)
    ctx = tb.Talaria(0, host_match_bytes=1 << 20)
    try:
        d_tokens = torch.zeros(450_000, dtype=torch.int32, device="cuda")
        d_hashes = torch.zeros(40_000, dtype=torch.int64, device="cuda")
        res = np.zeros(1, tb.MATCH_DTYPE)
        with pytest.raises(tb.TalariaError) as e:
            ctx.prefix_match_resident([(wl.tokens(g, 400_000), 0, 0, 420_000, 0, -1)], d_tokens, d_hashes, 16, SEED, res)
        assert e.value.status == tb.ERR_EXTENT
        assert int(d_tokens.abs().sum()) == 0
    finally:
        ctx.destroy()
