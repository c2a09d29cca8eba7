"""GPU parity: chained block hash and prefix match through the C ABI against the
CPU oracle, bit for bit (Sec. 4.3 cumulative prefix hash; App. A prefix reuse)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl

pytestmark = pytest.mark.gpu
SEED = wl.HASH_SEED


@pytest.fixture(scope="module")
def ctx():
    c = tb.Talaria(0)
    yield c
    c.destroy()


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _hash_gpu(ctx, tok, B, seed):
    d_tok = _dev(tok) if tok.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    nb = tok.size // B
    out = torch.full((max(nb, 1) + 2,), -1, dtype=torch.int64, device="cuda")   # two canary words
    ctx.block_hash(d_tok, tok.size, B, seed, out)
    ctx.sync()
    h = out.cpu().numpy().view(np.uint64)
    assert np.all(h[nb:max(nb, 1) + 2][-2:] == np.uint64(0xFFFFFFFFFFFFFFFF))
    return h[:nb]


@pytest.mark.parametrize("B", [1, 2, 3, 4, 8, 16, 24, 32, 64, 100, 4096])
def test_block_hash_matches_oracle(ctx, B):
    g = wl.rng(501, B)
    for T in (0, 1, B - 1, B, B + 1, 5 * B + 3, 2048, 2049, 4097, 3 * 2048 + 17 * B + 5):
        if T < 0:
            continue
        tok = wl.tokens(g, T)
        for seed in (0, SEED):
            assert np.array_equal(_hash_gpu(ctx, tok, B, seed), orc.block_hash(tok, B, seed)), (B, T)


def test_block_hash_long_stream_crosses_scan_chunks(ctx):
    # 105,000 tokens at 16-token blocks: 6,562 hashes = more than three scan chunks of 2,048
    tok = wl.tokens(wl.rng(502), 105_000)
    tok[100:200] = -np.arange(1, 101, dtype=np.int32)          # negative ids hash as their bit pattern
    for B in (16, 32, 1):
        assert np.array_equal(_hash_gpu(ctx, tok, B, SEED), orc.block_hash(tok, B, SEED))


def _match_batch(ctx, pairs, B, seed, with_stored, pad_front=0):
    """pairs: list of (cont, sess).  Returns GPU results + hashes via the device entry point."""
    pad_c, pad_s = pad_front if isinstance(pad_front, tuple) else (pad_front, pad_front)
    cont = np.concatenate([np.zeros(pad_c, np.int32)] + [c for c, _ in pairs])
    sess = np.concatenate([np.zeros(pad_s, np.int32)] + [s for _, s in pairs])
    co = np.cumsum([pad_c] + [c.size for c, _ in pairs]).astype(np.int64)
    so = np.cumsum([pad_s] + [s.size for _, s in pairs]).astype(np.int64)
    stored = [orc.block_hash(s, B, seed) for _, s in pairs]
    nbc = sum(c.size // B for c, _ in pairs)
    d_cont = _dev(cont) if cont.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    d_sess = _dev(sess) if sess.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    d_stored = None
    if with_stored:
        allh = np.concatenate(stored) if stored else np.zeros(0, np.uint64)
        d_stored = _dev(allh.view(np.int64)) if allh.size else torch.zeros(1, dtype=torch.int64, device="cuda")
    d_hashes = torch.zeros(max(nbc, 1), dtype=torch.int64, device="cuda")
    d_res = torch.zeros(len(pairs) * 4, dtype=torch.int64, device="cuda")
    ctx.prefix_match(len(pairs), d_cont, co, d_sess, so, d_stored, B, seed, d_hashes, d_res)
    ctx.sync()
    res = d_res.cpu().numpy().view(tb.MATCH_DTYPE)
    return res, d_hashes.cpu().numpy().view(np.uint64)[:nbc]


def _check_batch(ctx, pairs, B, seed, with_stored, pad_front=0):
    res, hashes = _match_batch(ctx, pairs, B, seed, with_stored, pad_front)
    at = 0
    for q, (c, s) in enumerate(pairs):
        m, hc = orc.prefix_match(c, s, B, seed)
        got = res[q]
        assert (int(got["lcp_tokens"]), int(got["matched_blocks"]), int(got["reusable_tokens"]),
                int(got["hash_token_disagree"])) == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens,
                                                     m.hash_token_disagree), (q, B)
        assert np.array_equal(hashes[at:at + hc.size], hc)
        at += hc.size


@pytest.mark.parametrize("with_stored", [False, True])
def test_config1_and_config2_pairs(ctx, with_stored):
    g = wl.rng(1)
    wl.tokens(g, 300)
    s1 = wl.tokens(g, 500)
    c1 = wl.continuation(g, s1, 560, 350)
    g2 = wl.rng(2)
    s2 = wl.tokens(g2, 25_000)
    c2 = wl.continuation(g2, s2, 27_000, 24_000)
    res, _ = _match_batch(ctx, [(c1, s1), (c2, s2)], 16, SEED, with_stored)
    assert [int(res[0][k]) for k in ("lcp_tokens", "matched_blocks", "reusable_tokens")] == [350, 21, 336]
    assert [int(res[1][k]) for k in ("lcp_tokens", "matched_blocks", "reusable_tokens")] == [24_000, 1_500, 24_000]
    _check_batch(ctx, [(c1, s1), (c2, s2)], 16, SEED, with_stored)
    _check_batch(ctx, [(c2, s2)], 32, SEED, with_stored)


@pytest.mark.parametrize("B", [1, 3, 16, 32, 24, 128])
@pytest.mark.parametrize("with_stored", [False, True])
def test_ragged_batch_with_degenerate_pairs(ctx, B, with_stored):
    g = wl.rng(503, B)
    e = np.zeros(0, np.int32)
    pairs = []
    for _ in range(12):
        ts, tc = int(g.integers(0, 9000)), int(g.integers(0, 9000))
        s = wl.tokens(g, ts)
        shared = int(g.integers(0, min(ts, tc) + 1))
        pairs.append((wl.continuation(g, s, tc, shared), s))
    s = wl.tokens(g, 5 * 2048)
    pairs += [(e, s), (s, e), (e, e), (s.copy(), s),                       # empty sides, identical streams
              (wl.continuation(g, s, s.size, 0), s),                       # differ at token 0
              (wl.continuation(g, s, s.size + 9, 2048), s),                # differ exactly on a tile boundary
              (wl.continuation(g, s, 3000, 2047), s),
              (s[:4 * B + 1].copy(), s)]                                   # continuation shorter than stored
    _check_batch(ctx, pairs, B, SEED, with_stored)
    _check_batch(ctx, pairs[:5], B, 0, with_stored, pad_front=3)           # token arrays not 16-byte aligned


@pytest.mark.parametrize("with_stored", [False, True])
def test_small_batch_with_a_long_pair_uses_the_tile_and_chain_kernels(ctx, with_stored):
    # a dozen pairs, one of them longer than a single CTA should take: the two-kernel path
    g = wl.rng(511)
    pairs = []
    for ts, tc, shared in [(118_000, 120_000, 110_001)] + [(int(g.integers(0, 6000)), int(g.integers(0, 6000)), None) for _ in range(11)]:
        s = wl.tokens(g, ts)
        pairs.append((wl.continuation(g, s, tc, int(g.integers(0, min(ts, tc) + 1)) if shared is None else shared), s))
    before = ctx.get_counters().kernel_launches
    _check_batch(ctx, pairs, 16, SEED, with_stored)
    assert ctx.get_counters().kernel_launches - before == 2
    before = ctx.get_counters().kernel_launches
    _check_batch(ctx, pairs[1:], 16, SEED, with_stored, pad_front=(2, 1))      # without the long pair: one CTA per pair
    assert ctx.get_counters().kernel_launches - before == 1


def test_corrupted_stored_hash_is_reported(ctx):
    g = wl.rng(504)
    s = wl.tokens(g, 1000)
    c = wl.continuation(g, s, 1200, 800)
    hs = orc.block_hash(s, 16, SEED)
    hs[20] ^= np.uint64(1)
    d_res = torch.zeros(4, dtype=torch.int64, device="cuda")
    ctx.prefix_match(1, _dev(c), [0, c.size], _dev(s), [0, s.size], _dev(hs.view(np.int64)), 16, SEED, None, d_res)
    ctx.sync()
    r = d_res.cpu().numpy().view(tb.MATCH_DTYPE)[0]
    m, _ = orc.prefix_match(c, s, 16, SEED, sess_hashes=hs)
    assert (int(r["lcp_tokens"]), int(r["matched_blocks"]), int(r["reusable_tokens"]), int(r["hash_token_disagree"])) \
        == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree) == (800, 20, 320, 1)


def test_host_entry_point_matches_oracle(ctx):
    g = wl.rng(505)
    pairs = []
    for _ in range(6):
        ts, tc = int(g.integers(1, 40_000)), int(g.integers(1, 40_000))
        s = wl.tokens(g, ts)
        pairs.append((wl.continuation(g, s, tc, int(g.integers(0, min(ts, tc) + 1))), s))
    cont = np.concatenate([c for c, _ in pairs]); sess = np.concatenate([s for _, s in pairs])
    co = np.cumsum([0] + [c.size for c, _ in pairs]); so = np.cumsum([0] + [s.size for _, s in pairs])
    for stored in (False, True):
        hs = np.concatenate([orc.block_hash(s, 16, SEED) for _, s in pairs]) if stored else None
        out_h = np.zeros(sum(c.size // 16 for c, _ in pairs), np.uint64)
        res = np.zeros(len(pairs), tb.MATCH_DTYPE)
        ctx.prefix_match_host(len(pairs), cont, co, sess, so, hs, 16, SEED, out_h, res)
        at = 0
        for q, (c, s) in enumerate(pairs):
            m, hc = orc.prefix_match(c, s, 16, SEED)
            assert (int(res[q]["lcp_tokens"]), int(res[q]["matched_blocks"]), int(res[q]["reusable_tokens"]),
                    int(res[q]["hash_token_disagree"])) == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, 0)
            assert np.array_equal(out_h[at:at + hc.size], hc)
            at += hc.size


def test_host_entry_point_splits_batches_larger_than_its_staging():
    # 1 MiB of staging (the minimum): the batch below needs several sub-batches of whole pairs
    small = tb.Talaria(0, host_match_bytes=1 << 20)
    try:
        g = wl.rng(510)
        pairs = []
        for _ in range(40):
            ts, tc = int(g.integers(0, 20_000)), int(g.integers(0, 20_000))
            s = wl.tokens(g, ts)
            pairs.append((wl.continuation(g, s, tc, int(g.integers(0, min(ts, tc) + 1))), s))
        cont = np.concatenate([c for c, _ in pairs]); sess = np.concatenate([s for _, s in pairs])
        co = np.cumsum([0] + [c.size for c, _ in pairs]); so = np.cumsum([0] + [s.size for _, s in pairs])
        assert (cont.size + sess.size) * 4 > 3 * (1 << 20)
        for stored in (False, True):
            hs = np.concatenate([orc.block_hash(s, 16, SEED) for _, s in pairs]) if stored else None
            out_h = np.zeros(sum(c.size // 16 for c, _ in pairs), np.uint64)
            res = np.zeros(len(pairs), tb.MATCH_DTYPE)
            before = small.get_counters().kernel_launches
            small.prefix_match_host(len(pairs), cont, co, sess, so, hs, 16, SEED, out_h, res)
            assert small.get_counters().kernel_launches - before >= 3          # really several sub-batches
            at = 0
            for q, (c, s) in enumerate(pairs):
                m, hc = orc.prefix_match(c, s, 16, SEED)
                assert (int(res[q]["lcp_tokens"]), int(res[q]["matched_blocks"]), int(res[q]["reusable_tokens"]),
                        int(res[q]["hash_token_disagree"])) == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, 0)
                assert np.array_equal(out_h[at:at + hc.size], hc)
                at += hc.size
        # a single pair that cannot fit is refused; nothing is allocated to make room
        big = wl.tokens(g, 200_000)
        free_before = torch.cuda.mem_get_info()[0]
        with pytest.raises(tb.TalariaError) as e:
            small.prefix_match_host(1, big, [0, big.size], big, [0, big.size], None, 16, SEED, None, np.zeros(1, tb.MATCH_DTYPE))
        assert e.value.status == tb.ERR_EXTENT
        assert torch.cuda.mem_get_info()[0] == free_before
    finally:
        small.destroy()


def test_prefix_agree_host_arithmetic():
    g = wl.rng(506)
    for _ in range(100):
        R, nb = int(g.integers(1, 9)), int(g.integers(0, 12))
        hashes = np.tile(g.integers(0, 2**63, size=nb, dtype=np.uint64), (R, 1)) if nb else np.zeros((R, 0), np.uint64)
        committed = g.integers(0, nb + 1, size=R)
        if nb and g.uniform() < 0.7:
            hashes[int(g.integers(0, R)), int(g.integers(0, nb))] ^= np.uint64(1)
        assert tb.Talaria.prefix_agree(committed, hashes) == orc.prefix_agree(committed, hashes)


def test_bad_arguments(ctx):
    d = torch.zeros(64, dtype=torch.int32, device="cuda")
    out = torch.zeros(64, dtype=torch.int64, device="cuda")
    for args in ((d, 64, 0, 0, out), (d, -1, 16, 0, out), (None, 64, 16, 0, out)):
        with pytest.raises(tb.TalariaError) as e:
            ctx.block_hash(*args)
        assert e.value.status == tb.ERR_INVALID_ARG
    with pytest.raises(tb.TalariaError):
        ctx.prefix_match(1, d, [0, 64], d, [64, 0], None, 16, 0, None, out)    # negative length
    ctx.block_hash(d, 64, 16, 0, out)
    ctx.sync()


def test_calls_on_two_streams_share_scratch_safely(ctx):
    # the context's digest scratch is shared: calls on different streams must not overlap on the GPU
    g = wl.rng(507)
    jobs = []
    for k in range(6):
        s = wl.tokens(g, 60_000 + 1000 * k)
        c = wl.continuation(g, s, 64_000, 30_000 + 500 * k)
        jobs.append((c, s, _dev(c), _dev(s), torch.zeros(64_000 // 16, dtype=torch.int64, device="cuda"),
                     torch.zeros(4, dtype=torch.int64, device="cuda")))
    streams = [torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for rep in range(3):
        for k, (c, s, dc, ds, dh, dr) in enumerate(jobs):
            ctx.prefix_match(1, dc, [0, c.size], ds, [0, s.size], None, 16, SEED, dh, dr, stream=streams[k % 3])
    torch.cuda.synchronize()
    for c, s, dc, ds, dh, dr in jobs:
        m, hc = orc.prefix_match(c, s, 16, SEED)
        r = dr.cpu().numpy()
        assert [int(r[0]), int(r[1]), int(r[2])] == [m.lcp_tokens, m.matched_blocks, m.reusable_tokens]
        assert np.array_equal(dh.cpu().numpy().view(np.uint64), hc)


def test_thousands_of_small_pairs(ctx):
    # descriptor tables far beyond the inline path, many empty and one-token pairs
    g = wl.rng(508)
    pairs = []
    for _ in range(3000):
        ts, tc = int(g.integers(0, 300)), int(g.integers(0, 300))
        s = wl.tokens(g, ts)
        pairs.append((wl.continuation(g, s, tc, int(g.integers(0, min(ts, tc) + 1))), s))
    _check_batch(ctx, pairs, 16, SEED, False)
    _check_batch(ctx, pairs, 4, SEED, True)


def _big_batch(B, seed):
    """At least one pair per SM, so the one-CTA-per-pair kernel runs: mostly short ragged pairs,
    plus pairs built around that kernel's boundaries (chunks of 1,024 blocks, rounds of 1,024 tokens)."""
    g = wl.rng(509, seed)
    chunk = 1024 * B
    e = np.zeros(0, np.int32)
    pairs = []
    for _ in range(150):
        ts, tc = int(g.integers(0, 3000)), int(g.integers(0, 3000))
        s = wl.tokens(g, ts)
        pairs.append((wl.continuation(g, s, tc, int(g.integers(0, min(ts, tc) + 1))), s))
    long_s = wl.tokens(g, 2 * chunk + 5 * B + 3)
    for tc, shared in ((2 * chunk + 900, chunk), (2 * chunk + 900, chunk - 1), (2 * chunk + 900, chunk + 1),
                       (long_s.size, long_s.size), (long_s.size + 1, long_s.size), (chunk, chunk), (chunk, 0),
                       (chunk + 1024, 1024), (chunk + 1024, 1023), (3 * chunk, 2 * chunk + 5 * B + 3),
                       (700, 700), (chunk // 2 + 7, 5)):
        pairs.append((wl.continuation(g, long_s, tc, shared), long_s))
    short_s = wl.tokens(g, 2 * B + 1)
    pairs += [(wl.continuation(g, short_s, 2 * chunk + 17, short_s.size), short_s),   # the continuation extends a short stream
              (long_s[: 3 * B].copy(), long_s), (e, long_s), (long_s, e), (e, e), (long_s.copy(), long_s)]
    return pairs


@pytest.mark.parametrize("B", [4, 8, 16, 32])
@pytest.mark.parametrize("with_stored", [False, True])
def test_large_batch_one_cta_per_pair(ctx, B, with_stored):
    pairs = _big_batch(B, B)
    assert len(pairs) >= 148
    _check_batch(ctx, pairs, B, SEED, with_stored)
    order = wl.rng(509, 77).permutation(len(pairs))                     # long pairs anywhere in the batch
    _check_batch(ctx, [pairs[k] for k in order], B, 0, with_stored, pad_front=(1, 2))
    _check_batch(ctx, [pairs[k] for k in order[::-1]], B, SEED, with_stored, pad_front=(3, 0))


def test_large_batch_detects_a_corrupted_stored_hash_in_a_late_chunk(ctx):
    B = 16
    pairs = _big_batch(B, 5)
    q = next(k for k, (c, s) in enumerate(pairs) if c.size > 2 * 1024 * B and np.array_equal(c[: s.size], s))
    cont = np.concatenate([c for c, _ in pairs]); sess = np.concatenate([s for _, s in pairs])
    co = np.cumsum([0] + [c.size for c, _ in pairs]).astype(np.int64)
    so = np.cumsum([0] + [s.size for _, s in pairs]).astype(np.int64)
    stored = [orc.block_hash(s, B, SEED) for _, s in pairs]
    bad_block = 1024 + 700                                              # second chunk of that pair
    stored[q][bad_block] ^= np.uint64(1 << 40)
    d_res = torch.zeros(len(pairs) * 4, dtype=torch.int64, device="cuda")
    ctx.prefix_match(len(pairs), _dev(cont), co, _dev(sess), so, _dev(np.concatenate(stored).view(np.int64)), B, SEED,
                     None, d_res)
    ctx.sync()
    res = d_res.cpu().numpy().view(tb.MATCH_DTYPE)
    for k, (c, s) in enumerate(pairs):
        m, _ = orc.prefix_match(c, s, B, SEED, sess_hashes=stored[k])
        assert (int(res[k]["lcp_tokens"]), int(res[k]["matched_blocks"]), int(res[k]["reusable_tokens"]),
                int(res[k]["hash_token_disagree"])) == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens,
                                                        m.hash_token_disagree), k
    assert int(res[q]["matched_blocks"]) == bad_block and int(res[q]["hash_token_disagree"]) == 1


def test_smoke_entry_point_runs():
    # the build/smoke entry used outside pytest must stay in step with the library
    import __graft_entry__ as ge
    ge.smoke()
