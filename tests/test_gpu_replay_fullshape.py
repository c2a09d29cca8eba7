"""GPU parity for the session-replay mix at the REAL KV shape (94 layers x 4 KV heads x 128, bf16,
16-token blocks) with the 19,479-block (60 GB) pool: the first calls of the schedule, enough to
force evictions, capacity pressure and restores.  The whole pool cannot be mirrored on the host
in seconds, so the test checks
  (a) three sampled layers (first, middle, last) of every checkpoint image, every restore and the
      final pool against the CPU oracle over a host mirror of just those layers;
  (b) every match record and every hash against the oracle;
  (c) for ALL layers, with torch indexing on the device as an independent routine: every
      checkpoint image equals the pool blocks its table names, and after every restore the new
      blocks equal the host images they came from.
Sec. 4.1 / 4.3 (checkpoint at call finish, restore into new slots, memory pressure), App. A, App. B."""
import numpy as np
import pytest
import torch

from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from paper_2607_17181_b200.replay import ReplayDriver
from tests.gpu_util import PinnedArena, ReplayMirror

pytestmark = pytest.mark.gpu

N_CALLS = 36
LAYERS = (0, 47, 93)


def _need(host_gb, device_gb):
    import psutil
    torch.cuda.empty_cache()
    free_dev = torch.cuda.mem_get_info()[0]
    avail = psutil.virtual_memory().available
    if avail < host_gb * 1.15e9:
        pytest.skip(f"needs {host_gb:.0f} GB of free host memory, the box has {avail / 1e9:.0f} GB available")
    if free_dev < device_gb * 1.02e9:
        pytest.skip(f"needs {device_gb:.0f} GB of free device memory, the GPU has {free_dev / 1e9:.0f} GB free")


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


def test_session_replay_at_the_full_kv_shape():
    shape = wl.QWEN235
    C, LP = shape.chunk_bytes, shape.num_layers * shape.num_planes
    pool_blocks = int(60e9) // shape.bytes_per_block
    assert pool_blocks == 19_479
    schedule = wl.session_replay()[:N_CALLS]
    max_blocks = max(shape.blocks_for(c.prompt_tokens) for c in schedule)
    host_budget = 72e9
    _need(host_gb=host_budget / 1e9 + 6, device_gb=60 + 2 * max_blocks * shape.bytes_per_block / 1e9 + 8)

    planes = [torch.zeros(pool_blocks * C, dtype=torch.uint8, device="cuda") for _ in range(LP)]
    kv, keep = tb.kv_layout(shape, [t.data_ptr() for t in planes], pool_blocks)
    lp_idx = [l * shape.num_planes + p for l in LAYERS for p in range(shape.num_planes)]
    small = wl.KvShape(len(LAYERS), shape.num_kv_heads, shape.block_tokens, shape.head_dim)
    mirror = ReplayMirror(small, [np.zeros(pool_blocks * C, np.uint8) for _ in lp_idx], "PF")
    arena = PinnedArena(int(host_budget) + (1 << 30))
    scratch = torch.empty(max_blocks * shape.bytes_per_block, dtype=torch.uint8, device="cuda")
    sampled = {}                                             # (sid, call) -> the sampled layers of that call's new KV

    def content(sid, k, nbytes):
        gen = torch.Generator(device="cuda")
        gen.manual_seed((sid << 16) | k)
        v = scratch[:nbytes]
        v.view(torch.int64).random_(generator=gen)
        m = nbytes // shape.bytes_per_block
        sampled[(sid, k)] = v.view(m, LP, C)[:, lp_idx, :].contiguous().cpu().numpy().reshape(-1)
        return v

    def all_layers_equal(image, table_slice):
        """image: pinned [n, L*P, C] page-first; every chunk must equal the pool block its table entry names."""
        n = table_slice.size
        d_img = image.cuda(non_blocking=True).view(n, LP, C)
        idx = torch.from_numpy(table_slice.astype(np.int64)).cuda()
        return all(bool(torch.equal(planes[lp].view(pool_blocks, C)[idx], d_img[:, lp])) for lp in range(LP))

    ctx = tb.Talaria(0)
    log = []
    drv = ReplayDriver(ctx, shape, kv, pool_blocks, int(host_budget), wl.HASH_SEED, content, arena.alloc, lambda a: a,
                       order="PF", log=log, free_pinned=arena.release, checkpoint="incremental", resident=(30, 131_072))
    streams, tg = {}, wl.rng(4, 2)
    checked_ckpt = checked_restore = 0
    try:
        for group in _groups(schedule, 4):
            calls = []
            for c in group:
                prev = streams.get(c.session)
                toks = wl.tokens(tg, c.prompt_tokens) if prev is None else \
                    wl.continuation(tg, prev, c.prompt_tokens, min(c.shared_tokens, prev.size))
                calls.append((c.session, c.index, toks))
            before = {sid: streams.get(sid, np.zeros(0, np.int32)) for sid, _, _ in calls}
            log.clear()
            drv.run_group(calls)
            drv.drain()
            for entry in log:
                mirror.apply(entry, calls, before, lambda sid, k, nbytes: sampled.pop((sid, k)))
                if entry[0] == "restore":
                    _, sid, table = entry
                    for e in drv.sessions[sid].extents:      # (c) restored blocks == the host images, all layers
                        if e.first >= table.size:             # a checkpoint this same call added afterwards
                            continue
                        m = min(e.n, table.size - e.first)
                        assert all_layers_equal(e.image[: m * shape.bytes_per_block], table[e.first:e.first + m]), sid
                        checked_restore += 1
            # (a) sampled layers and (c) all layers of every checkpoint written by this group
            for entry in log:
                if entry[0] != "checkpoint":
                    continue
                _, sid, first, ids = entry
                s = drv.sessions[sid]
                ext = [e for e in s.extents if e.first == first]
                if not ext:                                   # cut back again within the same group
                    continue
                e = ext[0]
                want = [m for m in mirror.ext[sid] if m[0] == first][0][3]
                got = e.image.view(e.cap, LP, C)[:, lp_idx, :].contiguous().numpy().reshape(-1)
                assert np.array_equal(got, want), (sid, first)
                if s.where == "device":                       # the blocks are still in the pool: compare all layers
                    assert all_layers_equal(e.image[: e.n * shape.bytes_per_block], s.table[first:first + e.n]), (sid, first)
                    checked_ckpt += 1
            for sid, _, toks in calls:
                streams[sid] = toks
        for k, lp in enumerate(lp_idx):                       # final pool, sampled layers, against the oracle mirror
            assert np.array_equal(planes[lp].cpu().numpy(), mirror.planes[k]), lp
        st = drv.stats
        assert st.calls == N_CALLS and st.evictions >= 3 and st.host_restores >= 1
        assert checked_ckpt >= N_CALLS // 2 and checked_restore >= 1
        # under host pressure some checkpoints are skipped, but most evicted bytes were on the host already
        assert st.evict_bytes_already_on_host > 3 * st.evict_bytes_copied
    finally:
        ctx.destroy()
