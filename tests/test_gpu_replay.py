"""GPU parity for the session-replay mix: 30 sessions with lognormal depth and prompt length,
97 % high-reuse continuations, a pool capped at the block count of a 60 GB Qwen3-235B pool, LRU
eviction, checkpoints of newly aligned blocks after every call (or whole-session copies at
eviction) and restore on return.  Every byte-moving step the driver logs is
replayed on the CPU oracle over a host mirror of the pool; pool, host images, match records and
hashes must agree exactly.  The KV shape is cut to 2 layers x 2 heads x 64 (16 KiB per block) so
the mirror stays small; block counts, tables and the schedule are those of the full shape.
Sec. 4.3 (checkpoint, restore into new slots, memory pressure), App. A (prefix reuse)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from paper_2607_17181_b200.replay import ReplayDriver
from tests.gpu_util import ReplayMirror as Mirror

pytestmark = pytest.mark.gpu


def _content(sid, k, nbytes):
    g = np.random.Generator(np.random.Philox(key=[wl.BASE_SEED + 4, (sid << 16) | k]))
    return g.integers(0, 256, size=nbytes, dtype=np.uint8)


def _groups(schedule, size):
    out, cur = [], []
    for c in schedule:
        if len(cur) == size or any(x.session == c.session for x in cur):
            out.append(cur)
            cur = []
        cur.append(c)
    if cur:
        out.append(cur)
    return out


@pytest.mark.parametrize("order,host_budget_frac,checkpoint,resident",
                         [("PF", 0.35, "eviction", False), ("LF", 10.0, "eviction", False),
                          ("PF", 10.0, "incremental", False), ("LF", 10.0, "incremental", True),
                          ("PF", 0.9, "incremental", True)])
def test_session_replay_mix_matches_oracle_mirror(order, host_budget_frac, checkpoint, resident):
    shape = wl.KvShape(2, 2, 16, 64)
    full = wl.QWEN235
    pool_blocks = int(60e9) // full.bytes_per_block                       # 19,479 blocks, as at the full shape
    assert pool_blocks == 19_479
    schedule = wl.session_replay()[:160]
    g = wl.rng(4, 1)
    planes_np = [g.integers(0, 256, size=pool_blocks * shape.chunk_bytes, dtype=np.uint8)
                 for _ in range(shape.num_layers * shape.num_planes)]
    d_planes = [torch.from_numpy(p).cuda() for p in planes_np]
    mirror = Mirror(shape, [p.copy() for p in planes_np], order)
    kv, keep = tb.kv_layout(shape, [t.data_ptr() for t in d_planes], pool_blocks)
    total_kv = sum(shape.blocks_for(c.prompt_tokens) for c in schedule[:30]) * shape.bytes_per_block
    ctx = tb.Talaria(0, bounce_bytes=8 << 20, dma_min_bytes=4 << 20)      # both variants get exercised
    log = []
    drv = ReplayDriver(ctx, shape, kv, pool_blocks, int(total_kv * host_budget_frac), wl.HASH_SEED, _content,
                       lambda n: torch.empty(n, dtype=torch.uint8, pin_memory=True),
                       lambda a: torch.from_numpy(a).cuda(), order=order, log=log, checkpoint=checkpoint,
                       resident=(30, 131_072) if resident else None)
    streams, tg = {}, wl.rng(4, 2)
    try:
        for gi, group in enumerate(_groups(schedule, 4)):
            calls = []
            for c in group:
                prev = streams.get(c.session)
                toks = wl.tokens(tg, c.prompt_tokens) if prev is None else \
                    wl.continuation(tg, prev, c.prompt_tokens, min(c.shared_tokens, prev.size))
                calls.append((c.session, c.index, toks))
            before = {sid: streams.get(sid, np.zeros(0, np.int32)) for sid, _, _ in calls}
            log.clear()
            drv.run_group(calls)
            for entry in log:
                mirror.apply(entry, calls, before, _content)
            for sid, _, toks in calls:
                streams[sid] = toks
            if gi % 8 == 7:
                mirror.check_host_images(drv)
        mirror.check_host_images(drv)
        for d, m in zip(d_planes, mirror.planes):
            assert np.array_equal(d.cpu().numpy(), m)
        # block ownership stays consistent: no block is owned twice or both owned and free
        owned = np.concatenate([s.table for s in drv.sessions.values() if s.where == "device"])
        assert owned.size == np.unique(owned).size
        assert not set(owned.tolist()) & set(drv.free)
        assert owned.size + len(drv.free) == pool_blocks
        st = drv.stats
        assert st.calls == len(schedule) and st.evictions > 0
        assert st.device_hits + st.host_restores + st.recomputes == st.calls
        if host_budget_frac >= 1:
            assert st.host_restores > 0 and st.capacity_misses == 0
        if checkpoint == "eviction" and host_budget_frac < 1:
            assert st.capacity_misses > 0 and st.host_restores > 0
        if checkpoint == "incremental":
            # the barrier at eviction found most of the session on the host already
            assert st.checkpoint_bytes > 0
            assert st.evict_bytes_already_on_host > 10 * st.evict_bytes_copied
    finally:
        ctx.destroy()
