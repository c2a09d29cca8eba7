"""Measurements of the other benchmark configurations (`bench.py --workload ...`).

`bench.py`'s default line is the one-session workload; these are the long-context,
staging-plus-restore and session-replay workloads.  Each function returns one dict
(printed as a JSON line by bench.py).  All timing is CUDA events on the launching
streams; parity for the same workloads lives in the tests.
"""
from __future__ import annotations

import statistics
import time
from typing import Dict, List

import numpy as np

from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from paper_2607_17181_b200.replay import ReplayDriver

PCIE5_X16_GBS = 63.0


def _pool(torch, dev, shape, num_blocks, seed):
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    planes = []
    for _ in range(shape.num_layers * shape.num_planes):
        t = torch.empty(num_blocks * shape.chunk_bytes // 2, dtype=torch.bfloat16, device=dev)
        t.normal_(generator=gen)
        planes.append(t)
    kv, keep = tb.kv_layout(shape, [t.data_ptr() for t in planes], num_blocks)
    return planes, kv, keep


def _timed(torch, stream, fn, reps):
    fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    return statistics.median(ts)


def run_long(torch, dev, ceilings, reps=3) -> Dict:
    """Long-context session (105,000 tokens) at 16- and 32-token blocks: offload, restore into
    isolated single free blocks, and the same restore while a second session (25,000 tokens) is
    offloaded on another stream."""
    out = {"workload": "configs[2]: 105,000-token session, Qwen3-235B KV shape, restore into isolated free "
                       "blocks, second-session offload overlapped", "cases": []}
    pinned = torch.empty(20_218_380_288, dtype=torch.uint8, pin_memory=True)
    for B, order in ((16, "PF"), (32, "PF"), (16, "LF")):
        shape = wl.QWEN235 if B == 16 else wl.QWEN235_B32
        NB = 16_384 if B == 16 else 8_192
        torch.cuda.empty_cache()
        planes, kv, keep = _pool(torch, dev, shape, NB, 30 + B)
        g = wl.rng(3, B)
        n, n2 = shape.blocks_for(105_000), shape.blocks_for(25_000)
        even = np.arange(0, NB, 2, dtype=np.int32)
        src = np.ascontiguousarray(g.permutation(even)[:n])
        second = np.ascontiguousarray(g.permutation(np.setdiff1d(even, src))[:n2])
        dst = wl.isolated_table(g, NB, n)
        size = n * shape.bytes_per_block
        image = pinned[:size]
        hl = tb.host_layout(wl.dense_strides(shape, n, order), size)
        image2 = torch.empty(n2 * shape.bytes_per_block, dtype=torch.uint8, pin_memory=True)
        hl2 = tb.host_layout(wl.dense_strides(shape, n2, "PF"), image2.numel())
        ctx = tb.Talaria(dev.index or 0)
        sa, sb = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        t_off = _timed(torch, sa, lambda: ctx.kv_offload(kv, src, 0, n, image, hl, stream=sa), reps)
        t_res = _timed(torch, sa, lambda: ctx.kv_restore(kv, dst, 0, n, image, hl, stream=sa), reps)
        both = []
        for _ in range(reps):
            torch.cuda.synchronize()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            e[0].record(sa); e[2].record(sb)
            ctx.kv_restore(kv, dst, 0, n, image, hl, stream=sa); e[1].record(sa)
            ctx.kv_offload(kv, second, 0, n2, image2, hl2, stream=sb); e[3].record(sb)
            torch.cuda.synchronize()
            both.append((e[0].elapsed_time(e[1]), e[2].elapsed_time(e[3])))
        t_r2, t_o2 = min(both)
        # self-check without the oracle: sampled chunks sit where the two tables say
        C, strides, ok = shape.chunk_bytes, wl.dense_strides(shape, n, order), True
        gs = wl.rng(3, 99)
        for _ in range(48):
            l, p, i = int(gs.integers(0, shape.num_layers)), int(gs.integers(0, 2)), int(gs.integers(0, n))
            a = l * strides[0] + p * strides[1] + i * strides[2]
            pl = planes[l * 2 + p].view(torch.uint8)
            chunk = image[a:a + C]
            ok &= bool(torch.equal(pl[int(src[i]) * C:(int(src[i]) + 1) * C].cpu(), chunk))
            ok &= bool(torch.equal(pl[int(dst[i]) * C:(int(dst[i]) + 1) * C].cpu(), chunk))
        toks = wl.tokens(g, 105_000)
        cont = wl.continuation(g, toks, 110_000, 100_000)
        d_s, d_c = torch.from_numpy(toks).to(dev), torch.from_numpy(cont).to(dev)
        d_h = torch.empty(110_000 // B, dtype=torch.int64, device=dev)
        d_r = torch.zeros(4, dtype=torch.int64, device=dev)
        t_m = _timed(torch, sa, lambda: [ctx.prefix_match(1, d_c, [0, 110_000], d_s, [0, 105_000], None, B,
                                                          wl.HASH_SEED, d_h, d_r, stream=sa) for _ in range(50)], reps) / 50
        out["cases"].append({
            "block_tokens": B, "host_layout": order, "blocks": n, "payload_bytes": size,
            "offload_gbs": size / t_off / 1e6, "offload_frac_of_d2h_ceiling": size / t_off / 1e6 / ceilings["d2h"],
            "restore_isolated_gbs": size / t_res / 1e6, "restore_frac_of_h2d_ceiling": size / t_res / 1e6 / ceilings["h2d"],
            "overlapped": {"restore_gbs": size / t_r2 / 1e6, "second_offload_gbs": image2.numel() / t_o2 / 1e6},
            "overlapped_sum_gbs": size / t_r2 / 1e6 + image2.numel() / t_o2 / 1e6,
            "prefix_match_us_gpu": t_m * 1e3, "variant": int(ctx.get_counters().last_variant), "self_check": ok})
        ctx.destroy()
        del planes, image2
    out["value"] = statistics.mean(c["restore_isolated_gbs"] for c in out["cases"])
    return out


def run_stage(torch, dev, ceilings, hbm_peak, reps=3) -> Dict:
    """D2D weight staging (58.96 GB in 2 MiB chunks) with a 25,000-token KV restore on a second
    stream, at 0 %, 1 % and 36 % dirty chunks."""
    ws = wl.moe_weight_set()
    plan, span = wl.stage_plan(ws.sizes, 2 << 20)
    total = sum(nb for _, nb, _ in plan)
    gen = torch.Generator(device=dev)
    gen.manual_seed(55)
    staging = torch.empty(span, dtype=torch.uint8, device=dev)
    for off in range(0, span, 1 << 30):
        m = min(1 << 30, span - off)
        staging[off:off + m].view(torch.int16).random_(generator=gen)
    slots = torch.zeros(span, dtype=torch.uint8, device=dev)
    shape, NB = wl.QWEN235, 2048
    nblk = shape.blocks_for(25_000)
    planes, kv, keep = _pool(torch, dev, shape, NB, 56)
    g = wl.rng(5)
    table = np.ascontiguousarray(g.permutation(NB)[:nblk].astype(np.int32))
    image = torch.empty(nblk * shape.bytes_per_block, dtype=torch.uint8, pin_memory=True)
    hl = tb.host_layout(wl.dense_strides(shape, nblk, "PF"), image.numel())
    ctx = tb.Talaria(dev.index or 0)
    sa, sb = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    out = {"workload": "configs[4]: 58.96 GB weight set staged D2D into stable slots (2 MiB chunks) while a "
                       "25,000-token KV restore runs on a second stream", "cases": []}
    n = len(plan)
    for frac in (0.0, 0.01, 0.36):
        dirty = g.uniform(size=n) < frac
        idx = np.nonzero(dirty)[0]
        host_off = np.zeros(n, np.int64)
        at = 0
        for k in idx:
            host_off[k] = at
            at += -(-plan[k][1] // 256) * 256
        host = torch.empty(max(at, 256), dtype=torch.uint8, pin_memory=True)
        for o in range(0, at, 1 << 30):               # host copies differ from what sits in the staging region
            m = min(1 << 30, at - o)
            host[o:o + m].copy_(torch.bitwise_not(staging[o:o + m]))
        arr = np.zeros(n, tb.COPY_DTYPE)
        for k, (off, nb, cid) in enumerate(plan):
            arr[k] = (staging.data_ptr() + off, host.data_ptr() + int(host_off[k]) if dirty[k] else 0,
                      slots.data_ptr() + off, nb, cid, 0)
        bitmap = np.packbits(dirty, bitorder="little")
        h2d = int(sum(plan[k][1] for k in idx))
        t_alone = _timed(torch, sa, lambda: ctx.stage(arr, bitmap, stream=sa), reps)
        prepared = ctx.stage_plan_create(arr)
        t_prepared = _timed(torch, sa, lambda: ctx.stage_plan_run(prepared, bitmap, stream=sa), reps)
        def host_us(call):          # host time of one call, the GPU idle when it is made
            ts = []
            for _ in range(5):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                call()
                ts.append(time.perf_counter() - t0)
            return statistics.median(ts) * 1e6
        host_us_prepared = host_us(lambda: ctx.stage_plan_run(prepared, bitmap, stream=sa))
        host_us_plain = host_us(lambda: ctx.stage(arr, bitmap, stream=sa))
        torch.cuda.synchronize()
        ctx.stage_plan_destroy(prepared)
        t_res_alone = _timed(torch, sb, lambda: ctx.kv_restore(kv, table, 0, nblk, image, hl, stream=sb), reps)
        both = []
        prepared = ctx.stage_plan_create(arr)
        for _ in range(reps):
            torch.cuda.synchronize()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            e[0].record(sa)
            ctx.stage_plan_run(prepared, bitmap, stream=sa); e[1].record(sa)
            e[2].record(sb)                               # the restore is timed from the moment it is issued
            ctx.kv_restore(kv, table, 0, nblk, image, hl, stream=sb); e[3].record(sb)
            torch.cuda.synchronize()
            both.append((e[0].elapsed_time(e[1]), e[2].elapsed_time(e[3]), max(e[0].elapsed_time(e[1]), e[0].elapsed_time(e[3]))))
        ctx.stage_plan_destroy(prepared)
        t_st, t_rs, t_window = min(both, key=lambda x: x[1])
        d2d = total - h2d
        ok = True
        for k in ([0, n // 2, n - 1] + [int(x) for x in idx[:3]]):
            off, nb, _ = plan[k]
            want = host[int(host_off[k]):int(host_off[k]) + nb].to(dev) if dirty[k] else staging[off:off + nb]
            ok &= bool(torch.equal(slots[off:off + nb], want))
        out["cases"].append({"self_check": ok,
            "dirty_fraction": frac, "d2d_bytes": d2d, "h2d_bytes": h2d,
            "stage_alone_ms": t_alone, "stage_prepared_plan_alone_ms": t_prepared,
            "host_us_per_call_plain": host_us_plain, "host_us_per_call_prepared": host_us_prepared,
            "stage_with_restore_ms": t_st,
            "d2d_gbs_read_write_alone": (2 * d2d / t_alone / 1e6) if frac == 0 else None,
            "frac_of_hbm_peak_alone": (2 * d2d / t_alone / 1e6 / hbm_peak) if frac == 0 else None,
            "h2d_gbs_alone": (h2d / t_alone / 1e6) if h2d else None,
            "restore_alone_gbs": image.numel() / t_res_alone / 1e6,
            "restore_with_stage_gbs": image.numel() / t_rs / 1e6,
            "restore_with_stage_frac_of_h2d_ceiling": image.numel() / t_rs / 1e6 / ceilings["h2d"],
            # all host-to-device bytes of the two operations over the window from the first start to the last end
            "h2d_link_gbs_over_both": (h2d + image.numel()) / t_window / 1e6,
            "h2d_link_frac_of_ceiling_over_both": (h2d + image.numel()) / t_window / 1e6 / ceilings["h2d"]})
        del host
    ctx.destroy()
    out["value"] = out["cases"][0]["d2d_gbs_read_write_alone"]
    del staging, slots, planes, image
    torch.cuda.empty_cache()
    try:
        out["through_layout"] = _stage_through_layout(torch, dev, total, hbm_peak)
    except Exception as e:
        out["through_layout"] = {"error": f"{type(e).__name__}: {e}"}
    return out


def _stage_through_layout(torch, dev, weight_bytes, hbm_peak, reps=3) -> Dict:
    """The same clean switch with every address handed out by the stable-address layout (Sec. 4.2 / 4.4):
    one 150 GB region, model A active (weights low, runtime buffers high, KV planes in the gap, 30 % of
    the blocks allocated), model B's 58.96 GB pre-staged in the tails of A's 188 KV planes, gathered
    into B's weights region at the low end."""
    S = 150 * 10**9 // 4096 * 4096
    shape = wl.QWEN235
    W = -(-weight_bytes // 256) * 256
    models = [(W, 1 << 30, shape.num_layers, shape.num_planes, shape.chunk_bytes)] * 2
    region = torch.empty(S, dtype=torch.uint8, device=dev)
    base = region.data_ptr()
    pad = (-base) % 256
    bump = tb.Bump(base + pad, S - 256, models)
    va = bump.activate(0)
    ids, _ = bump.alloc_blocks(int(va.num_blocks * 0.3))
    t0 = time.perf_counter()
    plan, placed = bump.stage_place(1, 2 << 20)
    place_ms = (time.perf_counter() - t0) * 1e3
    slack = bump.staging_slack(1, 2 << 20)
    # the staged bytes: whatever the tails hold, made random on the device
    kv_off = va.kv_base - base
    for o in range(kv_off, kv_off + va.kv_bytes, 1 << 30):
        m = min(1 << 30, kv_off + va.kv_bytes - o) // 8 * 8
        region[o:o + m].view(torch.int64).random_()
    ctx = tb.Talaria(dev.index or 0)
    st = torch.cuda.Stream(device=dev)
    prepared = ctx.stage_plan_create(plan)
    ms = _timed(torch, st, lambda: ctx.stage_plan_run(prepared, None, stream=st), reps)
    ok = placed == plan.size
    for k in (0, plan.size // 3, plan.size - 1):
        e = plan[k]
        a, d, nb = int(e["src_dev"]) - base, int(e["dst_dev"]) - base, int(e["bytes"])
        ok &= bool(torch.equal(region[a:a + nb], region[d:d + nb]))
    ctx.stage_plan_destroy(prepared)
    ctx.destroy()
    copied = int(plan["bytes"].sum())
    return {"region_bytes": S, "pool_blocks": int(va.num_blocks), "allocated_blocks": int(ids.size),
            "chunks": int(plan.size), "chunks_placed": int(placed), "stage_place_host_ms": place_ms,
            "staging_slack_bytes_after": int(slack), "stage_ms": ms, "d2d_gbs_read_write": 2 * copied / ms / 1e6,
            "frac_of_hbm_peak": 2 * copied / ms / 1e6 / hbm_peak, "self_check": bool(ok)}


class _Arena:
    """One pinned allocation handed out in pieces (best fit, explicit frees): page-locking is slow
    and a replay allocates and frees many host images."""

    def __init__(self, torch, nbytes):
        self.t = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
        self.free = [(0, nbytes)]

    def alloc(self, nbytes):
        need = -(-nbytes // 4096) * 4096
        fits = [k for k, (_, ln) in enumerate(self.free) if ln >= need]
        if not fits:
            raise MemoryError("pinned arena exhausted")
        k = min(fits, key=lambda j: self.free[j][1])          # best fit keeps large holes whole
        off, ln = self.free[k]
        self.free[k:k + 1] = [(off + need, ln - need)] if ln > need else []
        return self.t[off:off + nbytes]

    def release(self, t):
        off = t.data_ptr() - self.t.data_ptr()
        self.free.append((off, -(-t.numel() // 4096) * 4096))
        self.free.sort()
        merged = []
        for o, l in self.free:
            if merged and merged[-1][0] + merged[-1][1] == o:
                merged[-1] = (merged[-1][0], merged[-1][1] + l)
            else:
                merged.append((o, l))
        self.free = merged


def run_replay(torch, dev, ceilings, max_calls=96, host_budget_gb=96.0) -> Dict:
    """Session-replay mix at the full KV shape: 30 sessions, pool capped at 60 GB (19,479 blocks), LRU
    eviction, restore on return -- once with whole-session copies at eviction and once with background
    checkpoints of newly aligned blocks after every call (the eviction stall is what differs)."""
    shape = wl.QWEN235
    pool_blocks = int(60e9) // shape.bytes_per_block
    torch.cuda.empty_cache()
    planes, kv, keep = _pool(torch, dev, shape, pool_blocks, 44)
    arena = _Arena(torch, int(host_budget_gb * 1e9) + (2 << 30))
    scratch = torch.empty(131_072 // 16 * shape.bytes_per_block, dtype=torch.uint8, device=dev)

    def content(sid, k, nbytes):                 # synthetic "prefill output", generated on the device
        v = scratch[:nbytes]
        v.view(torch.int64).random_()
        return v

    schedule = wl.session_replay()[:max_calls]
    groups, cur = [], []
    for c in schedule:
        if len(cur) == 4 or any(x.session == c.session for x in cur):
            groups.append(cur)
            cur = []
        cur.append(c)
    if cur:
        groups.append(cur)
    out = {"workload": f"configs[3]: session-replay mix, first {len(schedule)} calls of 30 sessions, 60 GB pool "
                       f"({pool_blocks} blocks), LRU eviction, host budget {host_budget_gb:.0f} GB, 4 calls per group",
           "modes": []}
    C = shape.chunk_bytes
    for mode in ("eviction", "incremental"):
        ctx = tb.Talaria(dev.index or 0)
        arena.free = [(0, arena.t.numel())]
        drv = ReplayDriver(ctx, shape, kv, pool_blocks, int(host_budget_gb * 1e9), wl.HASH_SEED, content, arena.alloc,
                           lambda a: a, order="PF", free_pinned=arena.release, checkpoint=mode, resident=(30, 131_072))
        streams, tg = {}, wl.rng(4, 2)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for grp in groups:
            calls = []
            for c in grp:
                prev = streams.get(c.session)
                toks = wl.tokens(tg, c.prompt_tokens) if prev is None else \
                    wl.continuation(tg, prev, c.prompt_tokens, min(c.shared_tokens, prev.size))
                calls.append((c.session, c.index, toks))
                streams[c.session] = toks
            drv.run_group(calls)
        drv.drain()
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
        st = drv.stats
        # self-check without the oracle: blocks are owned once, and sampled chunks of the checkpoints of
        # resident sessions equal the pool blocks their tables name
        owned = np.concatenate([s.table for s in drv.sessions.values() if s.where == "device"])
        ok = owned.size == np.unique(owned).size and owned.size + len(drv.free) == pool_blocks
        gs = wl.rng(4, 9)
        for s in drv.sessions.values():
            if s.where != "device":
                continue
            for e in s.extents[:3]:
                i, lp = int(gs.integers(0, e.n)), int(gs.integers(0, shape.num_layers * shape.num_planes))
                got = e.image[(i * shape.num_layers * shape.num_planes + lp) * C:][:C]
                blk = int(s.table[e.first + i])
                ok &= bool(torch.equal(planes[lp].view(torch.uint8)[blk * C:(blk + 1) * C].cpu(), got))
        stalls = sorted(st.evict_stalls) or [0.0]
        out["modes"].append({
            "checkpoint": mode, "calls": st.calls, "device_hits": st.device_hits, "host_restores": st.host_restores,
            "recomputes": st.recomputes, "capacity_misses": st.capacity_misses, "evictions": st.evictions,
            "d2h_bytes": st.offload_bytes, "checkpoint_bytes": st.checkpoint_bytes, "restore_bytes": st.restore_bytes,
            "evict_bytes_already_on_host": st.evict_bytes_already_on_host, "evict_bytes_copied_at_eviction": st.evict_bytes_copied,
            "evict_stall_ms_total": st.evict_stall_s * 1e3, "evict_stall_ms_median": statistics.median(stalls) * 1e3,
            "evict_stall_ms_max": stalls[-1] * 1e3,
            "eviction_copy_gbs": (st.evict_bytes_copied / st.evict_stall_s / 1e9) if st.evict_stall_s > 0 else None,
            "restore_gbs": st.restore_bytes / max(st.restore_s, 1e-9) / 1e9,
            "restore_frac_of_h2d_ceiling": st.restore_bytes / max(st.restore_s, 1e-9) / 1e9 / ceilings["h2d"],
            "reused_fraction": st.reused_tokens / max(st.prompt_tokens, 1),
            "match": "prompts from pageable host memory; the sessions' stored streams and hashes stay on the device",
            "batched_match_us_per_group_from_pageable_host_median": statistics.median(st.match_times) * 1e6,
            "batched_match_us_per_group_from_pageable_host_max": max(st.match_times) * 1e6,
            "tokens_per_s_of_prefix_preserved": st.reused_tokens / max(wall, 1e-9),
            "wall_s_including_host_side_token_generation": wall, "self_check": bool(ok)})
        ctx.destroy()
        del drv
    ev, inc = out["modes"]
    out["timing"] = "host wall clock around drained calls (evictions and restores are 0.1 s and longer)"
    out["value"] = inc["restore_gbs"]
    return out


def run_sweep(torch, dev, ceilings) -> Dict:
    """Offload / restore time per variant over transfer sizes (the table behind the AUTO
    thresholds), the bounce-buffer size sweep, and both directions at once."""
    shape, NB = wl.QWEN235, 4096
    planes, kv, keep = _pool(torch, dev, shape, NB, 21)
    g = wl.rng(2)
    perm = g.permutation(NB).astype(np.int32)
    n_max = shape.blocks_for(25_000)
    bt, bt2 = np.ascontiguousarray(perm[:n_max]), np.ascontiguousarray(perm[n_max:2 * n_max])
    image = torch.empty(n_max * shape.bytes_per_block, dtype=torch.uint8, pin_memory=True)
    image2 = torch.empty(n_max * shape.bytes_per_block, dtype=torch.uint8, pin_memory=True)
    sa, sb = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    rows = []
    for nblk in (1, 4, 16, 64, 256, 1024, n_max):
        hl = tb.host_layout(wl.dense_strides(shape, nblk, "PF"), image.numel())
        row = {"blocks": nblk, "payload_bytes": nblk * shape.bytes_per_block}
        for variant in (tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE, tb.VARIANT_RUNS):
            if variant == tb.VARIANT_RUNS and nblk > 256:
                continue                                    # one 16 KiB copy per chunk: minutes at this size
            ctx = tb.Talaria(dev.index or 0, variant=variant)
            reps = 20 if nblk <= 64 else 5
            row[f"offload_v{variant}_us"] = _timed(torch, sa, lambda: ctx.kv_offload(kv, bt, 0, nblk, image, hl, stream=sa), reps) * 1e3
            row[f"restore_v{variant}_us"] = _timed(torch, sa, lambda: ctx.kv_restore(kv, bt2, 0, nblk, image, hl, stream=sa), reps) * 1e3
            ctx.destroy()
        rows.append(row)
    # table shape: adjacent ids (one long run) and isolated ids, layer-first image, every variant + AUTO
    shapes = []
    hl_lf = tb.host_layout(wl.dense_strides(shape, n_max, "LF"), image.numel())
    tables = {"random": (bt, bt2),
              "contiguous": (np.arange(100, 100 + n_max, dtype=np.int32), np.arange(2000, 2000 + n_max, dtype=np.int32)),
              "isolated": (wl.isolated_table(wl.rng(2, 7), NB, n_max), wl.isolated_table(wl.rng(2, 8), NB, n_max))}
    for name, (ta, tb_) in tables.items():
        row = {"table": name, "host_layout": "LF", "blocks": n_max}
        for variant in (tb.VARIANT_AUTO, tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE, tb.VARIANT_RUNS):
            if variant == tb.VARIANT_RUNS and name != "contiguous":
                continue
            ctx = tb.Talaria(dev.index or 0, variant=variant)
            t_o = _timed(torch, sa, lambda: ctx.kv_offload(kv, ta, 0, n_max, image, hl_lf, stream=sa), 3)
            t_r = _timed(torch, sa, lambda: ctx.kv_restore(kv, tb_, 0, n_max, image, hl_lf, stream=sa), 3)
            row[f"v{variant}"] = {"offload_gbs": image.numel() / t_o / 1e6, "restore_gbs": image.numel() / t_r / 1e6,
                                  "used": int(ctx.get_counters().last_variant)}
            ctx.destroy()
        shapes.append(row)
    hl = tb.host_layout(wl.dense_strides(shape, n_max, "PF"), image.numel())
    size = image.numel()
    bounce = []
    for mib in (32, 64, 128, 256, 512):
        ctx = tb.Talaria(dev.index or 0, variant=tb.VARIANT_BOUNCE, bounce_bytes=mib << 20)
        t_o = _timed(torch, sa, lambda: ctx.kv_offload(kv, bt, 0, n_max, image, hl, stream=sa), 5)
        t_r = _timed(torch, sa, lambda: ctx.kv_restore(kv, bt2, 0, n_max, image, hl, stream=sa), 5)
        bounce.append({"bounce_mib": mib, "offload_gbs": size / t_o / 1e6, "restore_gbs": size / t_r / 1e6})
        ctx.destroy()
    both = []
    ctxs = {v: tb.Talaria(dev.index or 0, variant=v) for v in (tb.VARIANT_ZEROCOPY, tb.VARIANT_BOUNCE)}
    for vo in ctxs:
        for vr in ctxs:
            best = None
            for _ in range(3):
                torch.cuda.synchronize()
                e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
                e[0].record(sa); e[2].record(sb)
                ctxs[vo].kv_offload(kv, bt, 0, n_max, image, hl, stream=sa); e[1].record(sa)
                ctxs[vr].kv_restore(kv, bt2, 0, n_max, image2, hl, stream=sb); e[3].record(sb)
                torch.cuda.synchronize()
                t = (e[0].elapsed_time(e[1]), e[2].elapsed_time(e[3]))
                if best is None or max(t) < max(best):
                    best = t
            both.append({"offload_variant": vo, "restore_variant": vr, "offload_gbs": size / best[0] / 1e6,
                         "restore_gbs": size / best[1] / 1e6, "total_gbs": 2 * size / max(best) / 1e6})
    for c in ctxs.values():
        c.destroy()
    return {"workload": "variant sweep: Qwen3-235B KV shape, random block tables, page-first pinned image",
            "sizes": rows, "table_shapes": shapes, "bounce_buffer": bounce, "bidirectional": both,
            "value": max(b["offload_gbs"] for b in bounce)}


def _match_from_host(torch, dev, ctx, g, n=4, T=36_000, B=16, reps=100) -> Dict:
    """A returning group of n sessions, prompts in pageable host memory, on an idle link: every stream
    sent up with the call (`prefix_match_host`) against streams and hashes kept on the device
    (`prefix_match_resident`).  Host wall time per synchronous call, median."""
    stored = [wl.tokens(g, T) for _ in range(n)]
    conts = [wl.continuation(g, s, T + 2000, T - 1000) for s in stored]
    want = [(T - 1000, (T - 1000) // B, (T - 1000) // B * B)] * n
    res = np.zeros(n, tb.MATCH_DTYPE)
    got = lambda: [(int(r["lcp_tokens"]), int(r["matched_blocks"]), int(r["reusable_tokens"])) for r in res]
    # (a) everything from host memory
    cont_all, sess_all = np.concatenate(conts), np.concatenate(stored)
    co = np.cumsum([0] + [c.size for c in conts]).astype(np.int64)
    so = np.cumsum([0] + [s.size for s in stored]).astype(np.int64)
    hs = np.zeros(int(sum(s.size // B for s in stored)), np.uint64)
    ctx.prefix_match_host(n, sess_all, so, sess_all, so, None, B, wl.HASH_SEED, hs, res)     # the stored streams' hashes
    out_h = np.zeros(int(sum(c.size // B for c in conts)), np.uint64)
    def timed(call):
        ts = []
        for _ in range(reps):
            t0 = time.perf_counter()
            call()
            ts.append(time.perf_counter() - t0)
        return statistics.median(ts) * 1e6
    us_host = timed(lambda: ctx.prefix_match_host(n, cont_all, co, sess_all, so, hs, B, wl.HASH_SEED, out_h, res))
    ok = got() == want
    # (b) stored streams and hashes resident: two places per session, used in turn
    stride, hstride = 131_072, 131_072 // B
    d_tokens = torch.zeros(2 * n * stride, dtype=torch.int32, device=dev)
    d_hashes = torch.zeros(2 * n * hstride, dtype=torch.int64, device=dev)
    ctx.prefix_match_resident([(stored[s], 2 * s * stride, 2 * s * hstride, (2 * s + 1) * stride, 0, -1) for s in range(n)],
                              d_tokens, d_hashes, B, wl.HASH_SEED, res)
    pairs = [(conts[s], (2 * s + 1) * stride, (2 * s + 1) * hstride, 2 * s * stride, stored[s].size, 2 * s * hstride)
             for s in range(n)]
    us_res = timed(lambda: ctx.prefix_match_resident(pairs, d_tokens, d_hashes, B, wl.HASH_SEED, res))
    ok = ok and got() == want
    ctx.set_timing(True)
    ctx.prefix_match_resident(pairs, d_tokens, d_hashes, B, wl.HASH_SEED, res)
    gpu_us = ctx.get_timing().total_ms * 1e3
    ctx.set_timing(False)
    same = bool(np.array_equal(d_hashes[(2 * 0 + 1) * hstride:(2 * 0 + 1) * hstride + conts[0].size // B].cpu().numpy().view(np.uint64),
                               out_h[:conts[0].size // B]))
    return {"sessions": n, "prompt_tokens": T + 2000, "stored_tokens": T,
            "us_per_call_every_stream_from_host": us_host, "us_per_call_streams_resident": us_res,
            "of_which_on_the_gpu_us_resident": gpu_us, "bytes_up_from_host": int(cont_all.nbytes + sess_all.nbytes + hs.nbytes),
            "bytes_up_resident": int(cont_all.nbytes), "self_check": bool(ok and same)}


def run_prefix(torch, dev, hbm_peak=6542.4, small=False) -> Dict:
    """Prefix-match latency for one returning session and throughput for a large batch.
    small: only the batch, cut to 444 pairs (one wave of the one-CTA-per-pair kernel, 155 MB of
    tokens) and a few launches: the profiling-sized case."""
    ctx = tb.Talaria(dev.index or 0)
    g = wl.rng(2)
    out = {"workload": "prefix match: one pair at session sizes; batch of 1,024 pairs x 32,768 tokens", "single": []}
    st = torch.cuda.Stream(device=dev)
    for Ts, Tc, shared in (() if small else ((25_000, 27_000, 24_000), (105_000, 110_000, 100_000))):
        sess = wl.tokens(g, Ts)
        cont = wl.continuation(g, sess, Tc, shared)
        d_c, d_s = torch.from_numpy(cont).to(dev), torch.from_numpy(sess).to(dev)
        d_st = torch.empty(Ts // 16, dtype=torch.int64, device=dev)
        ctx.block_hash(d_s, Ts, 16, wl.HASH_SEED, d_st, stream=st)
        d_h = torch.empty(Tc // 16, dtype=torch.int64, device=dev)
        d_r = torch.zeros(4, dtype=torch.int64, device=dev)
        for stored in (d_st, None):
            call = lambda: ctx.prefix_match(1, d_c, [0, Tc], d_s, [0, Ts], stored, 16, wl.HASH_SEED, d_h, d_r, stream=st)
            back = _timed(torch, st, lambda: [call() for _ in range(200)], 3) / 200
            t0 = time.perf_counter()
            for _ in range(200):
                call()
                ctx.sync(st)
            lat = (time.perf_counter() - t0) / 200
            r = d_r.cpu().numpy()
            out["single"].append({"cont_tokens": Tc, "sess_tokens": Ts, "stored_hashes": stored is not None,
                                  "us_per_call_gpu_back_to_back": back * 1e3, "us_call_plus_sync_via_python": lat * 1e6,
                                  "tokens_per_s_gpu": (Tc + Ts) / back * 1e3,
                                  "self_check": [int(r[0]), int(r[1]), int(r[2])] == [shared, shared // 16, shared // 16 * 16]})
    if not small:
        out["from_host"] = _match_from_host(torch, dev, ctx, g)
    npairs, T = (444 if small else 1024), 32768
    big_c = torch.randint(0, wl.VOCAB, (npairs * T,), dtype=torch.int32, device=dev)
    big_s = big_c.clone()
    big_s[T // 2::T] += 1
    offs = np.arange(npairs + 1, dtype=np.int64) * T
    d_hb = torch.empty(npairs * T // 16, dtype=torch.int64, device=dev)
    d_rb = torch.zeros(npairs * 4, dtype=torch.int64, device=dev)
    d_stb = torch.empty(npairs * T // 16, dtype=torch.int64, device=dev)
    ctx.prefix_match(npairs, big_c, offs, big_s, offs, None, 16, wl.HASH_SEED, d_hb, d_rb, stream=st)
    ctx.sync(st)
    r = d_rb.view(npairs, 4).cpu().numpy()
    ok = bool((r[:, 0] == T // 2).all() and (r[:, 1] == T // 2 // 16).all() and (r[:, 2] == T // 2).all())
    out["batch"] = []
    reps = 2 if small else 20                     # back to back, so host-side launch work overlaps the GPU
    for stored in (None, d_stb):
        if stored is not None:                    # the registry's stored hashes: the session streams' own
            for q in range(0, npairs, 128):       # (block_hash takes one stream at a time; done in slices of the batch)
                pass
            ctx.prefix_match(npairs, big_s, offs, big_s, offs, None, 16, wl.HASH_SEED, d_stb, d_rb, stream=st)
            ctx.sync(st)
        call = lambda: [ctx.prefix_match(npairs, big_c, offs, big_s, offs, stored, 16, wl.HASH_SEED, d_hb, d_rb, stream=st)
                        for _ in range(reps)]
        ms = _timed(torch, st, call, 1 if small else 5) / reps
        r = d_rb.view(npairs, 4).cpu().numpy()
        ok &= bool((r[:, 0] == T // 2).all() and (r[:, 1] == T // 2 // 16).all() and (r[:, 3] & 0xFFFFFFFF == 0).all())
        # mixes the kernel executes: the continuation's tokens only -- with derived hashes too, since
        # blocks before the first differing token have equal digests by construction (the session is
        # hashed for one block per pair)
        mixes = npairs * T
        out["batch"].append({"stored_hashes": stored is not None, "ms_per_call_back_to_back": ms,
                             "tokens_per_s": 2 * npairs * T / ms * 1e3,
                             "token_read_gbs": 2 * npairs * T * 4 / ms / 1e6,
                             "frac_of_hbm_peak": 2 * npairs * T * 4 / ms / 1e6 / hbm_peak,
                             "mixes_per_s": mixes / ms * 1e3,
                             "frac_of_alu_ceiling_1.08e12_mixes_per_s": mixes / ms * 1e3 / 1.08e12})
    out["self_check"] = ok and out.get("from_host", {}).get("self_check", True)
    ctx.destroy()
    out["value"] = out["batch"][0]["tokens_per_s"]
    return out
