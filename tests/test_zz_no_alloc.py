"""The allocation-free prefix match must give exactly what the ordinary entry point gives.

`talaria_prefix_match_static` exists for callers that cannot touch the CUDA allocator (all HBM is
owned by the serving engine's own memory manager, or the call sits in a latency-critical loop
where an allocation would stall every stream).  It keeps its scratch in a fixed array inside the
library, which every call shares and which still holds the previous call's data; so the check is
made on two different batches in a row, through the C ABI, and compares hashes and match records
bit for bit with `talaria_prefix_match` (tolerance 0, as in every other parity test here).
A second test compares it with the CPU oracle directly and checks the property in its name: the
device's free memory is the same before and after calls that follow the first one.
The file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _batch(seed, lengths, B):
    g = wl.rng(900, seed)
    pairs = []
    for ts, tc, shared in lengths:
        s = wl.tokens(g, ts)
        pairs.append((wl.continuation(g, s, tc, min(shared, ts, tc)), s))
    cont = np.concatenate([c for c, _ in pairs])
    sess = np.concatenate([s for _, s in pairs])
    co = np.cumsum([0] + [c.size for c, _ in pairs]).astype(np.int64)
    so = np.cumsum([0] + [s.size for _, s in pairs]).astype(np.int64)
    nbc = sum(c.size // B for c, _ in pairs)
    nbs = sum(s.size // B for _, s in pairs)
    return torch.from_numpy(cont).cuda(), co, torch.from_numpy(sess).cuda(), so, nbc, nbs, len(pairs)


def _run_both(ctx, batch, B, with_stored):
    d_cont, co, d_sess, so, nbc, nbs, n = batch
    stored = None
    if with_stored:
        stored = torch.zeros(max(nbs, 1), dtype=torch.int64, device="cuda")
        for q in range(n):                      # the registry's stored hashes, pair by pair
            ts = int(so[q + 1] - so[q])
            off = sum(int(so[r + 1] - so[r]) // B for r in range(q))
            if ts // B:
                ctx.block_hash(d_sess[int(so[q]):], ts, B, wl.HASH_SEED, stored[off:])
    out = []
    for which in ("context", "static"):
        hashes = torch.full((max(nbc, 1),), -1, dtype=torch.int64, device="cuda")
        res = torch.full((n * 4,), -1, dtype=torch.int64, device="cuda")
        if which == "context":
            ctx.prefix_match(n, d_cont, co, d_sess, so, stored, B, wl.HASH_SEED, hashes, res)
        else:
            tb.Talaria.prefix_match_static(n, d_cont, co, d_sess, so, stored, B, wl.HASH_SEED, hashes, res)
        torch.cuda.synchronize()
        out.append((hashes.cpu().numpy(), res.cpu().numpy()))
    return out


def test_static_scratch_entry_point_matches_the_context_one_on_two_calls_in_a_row():
    torch.cuda.set_device(0)
    ctx = tb.Talaria(0)
    try:
        first = _batch(1, [(25_000, 27_000, 24_000), (500, 560, 350), (0, 40, 0), (7000, 33, 33)], 16)
        second = _batch(2, [(9000, 3000, 2047), (4097, 4097, 4097), (100, 0, 0)], 32)
        third = _batch(3, [(5000, 6000, 4500)], 24)                   # general block size path
        for batch, B in ((first, 16), (second, 32), (third, 24), (first, 16)):
            for with_stored in (False, True):
                (h_ctx, r_ctx), (h_st, r_st) = _run_both(ctx, batch, B, with_stored)
                assert np.array_equal(h_ctx, h_st)
                assert np.array_equal(r_ctx, r_st)
                assert r_ctx[0] >= 0                                  # results were really written
    finally:
        ctx.destroy()


def test_static_entry_point_matches_the_oracle_and_allocates_nothing():
    torch.cuda.set_device(0)
    g = wl.rng(901)
    B = 16
    cases = [(25_000, 27_000, 24_000), (500, 560, 350), (7000, 33, 33), (4097, 9000, 4096)]
    bufs = []
    for ts, tc, shared in cases:                                     # every buffer exists before the measured calls
        s = wl.tokens(g, ts)
        c = wl.continuation(g, s, tc, shared)
        bufs.append((c, s, torch.from_numpy(c).cuda(), torch.from_numpy(s).cuda(),
                     torch.from_numpy(orc.block_hash(s, B, wl.HASH_SEED).view(np.int64).copy()).cuda(),
                     torch.full((max(tc // B, 1),), -1, dtype=torch.int64, device="cuda"),
                     torch.full((4,), -1, dtype=torch.int64, device="cuda")))
    c, s, dc, ds, dst, dh, dr = bufs[0]
    tb.Talaria.prefix_match_static(1, dc, [0, c.size], ds, [0, s.size], None, B, wl.HASH_SEED, dh, dr)   # first call: address lookup
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for c, s, dc, ds, dst, dh, dr in bufs:
        for stored in (None, dst):
            dh.fill_(-1); dr.fill_(-1)
            tb.Talaria.prefix_match_static(1, dc, [0, c.size], ds, [0, s.size], stored, B, wl.HASH_SEED, dh, dr)
            torch.cuda.synchronize()
            m, hc = orc.prefix_match(c, s, B, wl.HASH_SEED)
            r = dr.cpu().numpy().view(tb.MATCH_DTYPE)[0]
            assert (int(r["lcp_tokens"]), int(r["matched_blocks"]), int(r["reusable_tokens"]), int(r["hash_token_disagree"])) \
                == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, m.hash_token_disagree)
            assert np.array_equal(dh.cpu().numpy().view(np.uint64)[: hc.size], hc)
    assert torch.cuda.mem_get_info()[0] == free_before               # nothing was allocated or freed on the device


def test_static_entry_point_accepts_the_documented_limit_case():
    # one pair of two 1,000,000-token streams at B = 16: 2 x 62,500 digests + 489 tiles <= 131,072 words
    torch.cuda.set_device(0)
    g = wl.rng(902)
    T, B = 1_000_000, 16
    s = wl.tokens(g, T)
    c = wl.continuation(g, s, T, 777_777)
    dc, ds = torch.from_numpy(c).cuda(), torch.from_numpy(s).cuda()
    dh = torch.zeros(T // B, dtype=torch.int64, device="cuda")
    dr = torch.zeros(4, dtype=torch.int64, device="cuda")
    tb.Talaria.prefix_match_static(1, dc, [0, T], ds, [0, T], None, B, wl.HASH_SEED, dh, dr)
    torch.cuda.synchronize()
    m, hc = orc.prefix_match(c, s, B, wl.HASH_SEED)
    r = dr.cpu().numpy().view(tb.MATCH_DTYPE)[0]
    assert (int(r["lcp_tokens"]), int(r["matched_blocks"]), int(r["reusable_tokens"])) == \
        (m.lcp_tokens, m.matched_blocks, m.reusable_tokens) == (777_777, 777_777 // B, 777_777 // B * B)
    assert np.array_equal(dh.cpu().numpy().view(np.uint64), hc)
    with pytest.raises(tb.TalariaError) as e:                         # a little more no longer fits
        big = np.array([0, 1_050_000], dtype=np.int64)
        tb.Talaria.prefix_match_static(1, dc, big, ds, big, None, B, wl.HASH_SEED, None, dr)
    assert e.value.status == tb.ERR_EXTENT


def test_static_entry_point_rejects_sizes_beyond_its_fixed_scratch():
    torch.cuda.set_device(0)
    d = torch.zeros(64, dtype=torch.int32, device="cuda")
    res = torch.zeros(64, dtype=torch.int64, device="cuda")
    offs9 = np.arange(10, dtype=np.int64)
    with pytest.raises(tb.TalariaError) as e:                         # more than 8 pairs
        tb.Talaria.prefix_match_static(9, d, offs9, d, offs9, None, 16, 0, None, res)
    assert e.value.status == tb.ERR_EXTENT
    big = np.array([0, 3_000_000], dtype=np.int64)                    # 3M tokens at B=1: 6M words needed
    with pytest.raises(tb.TalariaError) as e:                         # rejected before any launch or access
        tb.Talaria.prefix_match_static(1, d, big, d, big, None, 1, 0, None, res)
    assert e.value.status == tb.ERR_EXTENT
    with pytest.raises(tb.TalariaError) as e:
        tb.Talaria.prefix_match_static(1, d, [0, 64], d, [0, 64], None, 0, 0, None, res)
    assert e.value.status == tb.ERR_INVALID_ARG
    tb.Talaria.prefix_match_static(1, d, [0, 64], d, [0, 64], None, 16, 0, None, res)
    torch.cuda.synchronize()
    assert res.cpu().numpy().view(tb.MATCH_DTYPE)[0]["lcp_tokens"] == 64
