#!/usr/bin/env python
"""Benchmark of the KV-substrate hot path on B200 (one process per GPU).

The timed step is one pass of the whole path for one Qwen3-235B-shaped session
(94 layers, 4 KV heads, head_dim 128, bf16, 16-token blocks, 25,000-token prefix):

    stream A: KV offload of the session's 1,563 scattered blocks to pinned host
    stream B: D2D staging of a ~59 GB weight set into stable slots   (concurrent; the plan was
              validated and uploaded once, before the timed region: talaria_stage_plan_run)
    drain both (switch barrier)
    prefix match of the 27,000-token continuation (24,000 shared) + result read-back
    KV restore of the matched 1,500 blocks into a different free-block permutation

`value` is host-link payload GB/s (offload + restore bytes) over the whole step.
Prints ONE JSON line on rank 0.  After the timed steps the same run measures the other
configurations and adds them to that line: "configs2" (105,000-token session, 16- and 32-token
blocks, restore into isolated blocks, overlapped second offload), "configs3" (session-replay mix
under a 60 GB pool, whole-session eviction vs background checkpoints), "configs4" (59 GB staged
switch at 0 / 1 / 36 % dirty chunks, with and without a concurrent restore) and "prefix" (one pair
at session sizes, batch of 1,024 x 32,768 tokens).  `--workload X` prints one of them alone;
`--workload session` only the timed step.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_17181_b200 import workloads as wl  # noqa: E402

METRIC = "KV restore/offload GB/s (frac of host-link peak); gather/stage GB/s vs HBM peak"
UNIT = "GB/s host-link payload (offload+restore) over the whole step"
PCIE5_X16_GBS = 63.0          # 32 GT/s x 16 lanes x 128/130 / 8, per direction
POOL_BLOCKS = 4096
PREFIX_TOKENS, CONT_TOKENS, SHARED_TOKENS = 25_000, 27_000, 24_000
STAGE_CHUNK = 2 << 20
STAGE_FRACTION = 1.0
# DRAM bytes per algorithmic byte of stage_copy_kernel, from an ncu capture of the profiling-sized
# case (--scale small): (dram__bytes_read.sum + dram__bytes_write.sum) / (2 x payload)
STAGE_TRAFFIC_RATIO = 0.987


def apply_scale(scale: str):
    """'small' is the same step on a workload that fits an ncu capture: 1,024-block pool,
    4,096-token session, the first 1/32 of the staging plan (about 5 GB on the device)."""
    global POOL_BLOCKS, PREFIX_TOKENS, CONT_TOKENS, SHARED_TOKENS, STAGE_FRACTION
    if scale == "small":
        POOL_BLOCKS, PREFIX_TOKENS, CONT_TOKENS, SHARED_TOKENS, STAGE_FRACTION = 1024, 4096, 4608, 4000, 1 / 32


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f), "measured"
    except Exception:
        return {"hbm_gbs": 6650.0}, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.proc = gpu_index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------- CPU arm


def oracle_step_factory(layers: int, stage_fraction: float):
    """A bounded sample of the same workload for the CPU oracle: the first
    `layers` of the 94 layers for the block-table copies, the full token streams
    for the match, and the first `stage_fraction` of the staging plan."""
    from oracle import oracle as orc
    shape = wl.KvShape(layers, 4, 16, 128)
    g = wl.rng(2)
    sess = wl.tokens(g, PREFIX_TOKENS)
    cont = wl.continuation(g, sess, CONT_TOKENS, SHARED_TOKENS)
    perm = g.permutation(POOL_BLOCKS).astype(np.int32)
    n = shape.blocks_for(PREFIX_TOKENS)
    bt, bt2 = np.ascontiguousarray(perm[:n]), np.ascontiguousarray(perm[n:2 * n])
    one = wl.bf16_normal_bytes(g, POOL_BLOCKS * shape.chunk_bytes)
    planes = [one.copy() for _ in range(shape.num_layers * shape.num_planes)]
    strides = wl.dense_strides(shape, n, "PF")
    image = np.zeros(n * shape.bytes_per_block, np.uint8)
    oshape = orc.KvShape(layers, 4, 16, 128)
    ws = wl.moe_weight_set()
    plan, _ = wl.stage_plan(ws.sizes, STAGE_CHUNK)
    plan = plan[: max(1, int(len(plan) * stage_fraction))]
    span = plan[-1][0] + plan[-1][1]
    staging = np.frombuffer(np.random.default_rng(0).bytes(1 << 20), np.uint8)
    staging = np.resize(staging, span)
    slots = np.zeros(span, np.uint8)
    entries = [(off, None, off, nb, cid) for off, nb, cid in plan]
    stored = orc.block_hash(sess, 16, wl.HASH_SEED)

    def step():
        orc.kv_offload(oshape, planes, bt, 0, n, image, strides)
        orc.stage(staging, None, slots, entries, None)
        m, _ = orc.prefix_match(cont, sess, 16, wl.HASH_SEED, sess_hashes=stored)
        nr = m.reusable_tokens // 16
        orc.kv_restore(oshape, planes, bt2, 0, nr, image, strides)
        return (n + nr) * shape.bytes_per_block

    sample = (f"{layers} of 94 layers of the same session (offload {n} + restore 1500 blocks) and the same "
              f"fraction ({stage_fraction:.3f}) of the staging plan, full 27k/25k-token match; single thread")
    return step, sample


# the CPU arm samples the KV layers and the staging plan with ONE fraction
ORACLE_LAYERS = 12
ORACLE_FRACTION = ORACLE_LAYERS / 94


def time_oracle(steps: int, warmup: int, layers: int = ORACLE_LAYERS, stage_fraction: float = ORACLE_FRACTION):
    step, sample = oracle_step_factory(layers, stage_fraction)
    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    moved = 0
    for _ in range(steps):
        moved += step()
    dt = time.perf_counter() - t0
    return moved / dt / 1e9, dt / steps * 1e3, sample


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    gbs, ms, sample = time_oracle(args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": "configs[1]: Qwen3-235B-shaped KV, one 25,000-token session (bounded CPU sample)"},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------- GPU arm


def link_ceiling(torch, dev, nbytes=1 << 30, reps=6):
    """Pinned cudaMemcpyAsync ceilings (GB/s): H2D, D2H, best of `reps`."""
    h = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    d = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    best = {}
    for name, (dst, src) in {"h2d": (d, h), "d2h": (h, d)}.items():
        t = 1e9
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); dst.copy_(src, non_blocking=True); e1.record(); e1.synchronize()
            t = min(t, e0.elapsed_time(e1))
        best[name] = nbytes / t / 1e6
    del h, d
    return best


def _release_memory(torch):
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    try:
        torch._C._host_emptyCache()              # pinned blocks cached by torch
    except Exception:
        pass


def run_leg(name, torch, dev, ceilings, hbm_peak, small=False):
    """One of the other configurations; returns its dict (or the error that stopped it)."""
    import bench_configs as bc
    units = {
        "long": "GB/s restore into isolated blocks (mean over cases)",
        "stage": "GB/s read+write of the D2D staging kernel, all chunks clean, alone",
        "replay": "GB/s restore of returning sessions (background-checkpoint mode)",
        "prefix": "tokens/s, batch of 1,024 pairs x 32,768 tokens, session hashes derived",
        "sweep": "GB/s best bounce-variant offload of the 25,000-token session",
    }
    t0 = time.perf_counter()
    try:
        if name == "long":
            res = bc.run_long(torch, dev, ceilings)
        elif name == "stage":
            res = bc.run_stage(torch, dev, ceilings, hbm_peak)
        elif name == "replay":
            res = bc.run_replay(torch, dev, ceilings)
        elif name == "prefix":
            res = bc.run_prefix(torch, dev, hbm_peak, small=small)
        else:
            res = bc.run_sweep(torch, dev, ceilings)
        res["unit"] = units[name]
    except Exception as e:                        # a leg that cannot run here (memory) must not lose the line
        res = {"error": f"{type(e).__name__}: {e}"}
    res["seconds"] = time.perf_counter() - t0
    _release_memory(torch)
    return res


def run_other_workload(args):
    """One of configs[2..4] / prefix / sweep as a line of its own."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ceilings = link_ceiling(torch, dev)
    peaks, kind = measured_peaks()
    sampler = ClockSampler(local)
    sampler.start()
    res = run_leg(args.workload, torch, dev, ceilings, float(peaks["hbm_gbs"]), small=args.scale == "small")
    clocks = sampler.stop()
    line = {"metric": METRIC, "value": res.pop("value", None), "unit": res.pop("unit", None), "n_gpus": 1,
            "higher_is_better": True, "dtype": "u8", "data": "synthetic", "vs_baseline": None,
            "config": {"workload": res.pop("workload", args.workload)},
            "ceilings": {"h2d_gbs": ceilings["h2d"], "d2h_gbs": ceilings["d2h"], "hbm_gbs": peaks["hbm_gbs"],
                         "hbm_kind": kind, "nominal_pcie5_x16_gbs": PCIE5_X16_GBS}, "clocks": clocks}
    line.update(res)
    print(json.dumps(line))


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2607_17181_b200 import binding as tb
    from paper_2607_17181_b200.replicas import job_totals

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    tb.lib()                                        # fails loudly if the CUDA library was not built

    shape = wl.QWEN235
    C = shape.chunk_bytes
    g = wl.rng(2)
    sess = wl.tokens(g, PREFIX_TOKENS)
    cont = wl.continuation(g, sess, CONT_TOKENS, SHARED_TOKENS)
    perm = g.permutation(POOL_BLOCKS).astype(np.int32)
    n = shape.blocks_for(PREFIX_TOKENS)
    bt, bt2 = np.ascontiguousarray(perm[:n]), np.ascontiguousarray(perm[n:2 * n])

    # ---- device state (untimed) ------------------------------------------
    gen = torch.Generator(device=dev); gen.manual_seed(wl.BASE_SEED + 2)
    planes = []
    for _ in range(shape.num_layers * shape.num_planes):
        t = torch.empty(POOL_BLOCKS * C // 2, dtype=torch.bfloat16, device=dev)
        t.normal_(generator=gen)
        planes.append(t)
    kv, _keep = tb.kv_layout(shape, [t.data_ptr() for t in planes], POOL_BLOCKS)
    strides = wl.dense_strides(shape, n, "PF")
    image = torch.empty(n * shape.bytes_per_block, dtype=torch.uint8, pin_memory=True)
    hl = tb.host_layout(strides, image.numel())

    ws = wl.moe_weight_set()
    plan, span = wl.stage_plan(ws.sizes, STAGE_CHUNK)
    if STAGE_FRACTION < 1.0:
        plan = plan[: max(1, int(len(plan) * STAGE_FRACTION))]
        span = plan[-1][0] + plan[-1][1]
    if args.no_stage:
        plan, span = [], 0
    staging = torch.empty(max(span, 16), dtype=torch.uint8, device=dev)
    slots = torch.zeros(max(span, 16), dtype=torch.uint8, device=dev)
    for off in range(0, span, 1 << 30):
        m = min(1 << 30, span - off)
        staging[off:off + m].view(torch.int16)[: m // 2].random_(generator=gen)
    plan_arr = np.zeros(len(plan), tb.COPY_DTYPE)
    for k, (off, nb, cid) in enumerate(plan):
        plan_arr[k] = (staging.data_ptr() + off, 0, slots.data_ptr() + off, nb, cid, 0)
    stage_bytes = int(sum(nb for _, nb, _ in plan))

    d_cont = torch.from_numpy(cont).to(dev)
    d_sess = torch.from_numpy(sess).to(dev)
    ctx = tb.Talaria(local, variant=args.variant, pack_ctas=args.pack_ctas)
    # the model's gather plan is known long before the switch: validate and upload it once
    prepared = ctx.stage_plan_create(plan_arr) if len(plan_arr) else None
    d_stored = torch.empty(PREFIX_TOKENS // 16, dtype=torch.int64, device=dev)
    ctx.block_hash(d_sess, PREFIX_TOKENS, 16, wl.HASH_SEED, d_stored)     # the registry's stored hashes
    d_hashes = torch.empty(CONT_TOKENS // 16, dtype=torch.int64, device=dev)
    d_res = torch.zeros(4, dtype=torch.int64, device=dev)
    h_res = torch.zeros(4, dtype=torch.int64, pin_memory=True)
    h_cont = torch.from_numpy(cont).pin_memory()
    h_sess = torch.from_numpy(sess).pin_memory()
    h_stored = d_stored.cpu().pin_memory()
    h_hashes = torch.empty(CONT_TOKENS // 16, dtype=torch.int64, pin_memory=True)
    h_match = np.zeros(1, tb.MATCH_DTYPE)
    co, so = np.array([0, CONT_TOKENS], np.int64), np.array([0, PREFIX_TOKENS], np.int64)
    sa, sb = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ceilings = link_ceiling(torch, dev)

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    marks = []                                   # per step: dict of (start, end) event pairs

    def step(e2e: bool, record: bool):
        m = {k: (ev(), ev()) for k in ("offload", "stage", "match", "restore")} if record else None
        if record: m["offload"][0].record(sa)
        ctx.kv_offload(kv, bt, 0, n, image.data_ptr(), hl, stream=sa)
        if record: m["offload"][1].record(sa)
        if len(plan_arr):
            if record: m["stage"][0].record(sb)
            ctx.stage_plan_run(prepared, None, stream=sb)
            if record: m["stage"][1].record(sb)
        ctx.sync(sa); ctx.sync(sb)                                   # switch barrier: drain D2H and D2D
        if record: m["match"][0].record(sa)
        if e2e:
            ctx.prefix_match_host(1, h_cont.numpy(), co, h_sess.numpy(), so, h_stored.numpy().view(np.uint64), 16,
                                  wl.HASH_SEED, h_hashes.numpy().view(np.uint64), h_match, stream=sa)
            reusable = int(h_match[0]["reusable_tokens"])
        else:
            # the result record is written by the kernel straight into pinned host memory
            ctx.prefix_match(1, d_cont, co, d_sess, so, d_stored, 16, wl.HASH_SEED, d_hashes, h_res, stream=sa)
            ctx.sync(sa)
            reusable = int(h_res[2])
        if record: m["match"][1].record(sa)
        nr = reusable // 16
        if record: m["restore"][0].record(sa)
        ctx.kv_restore(kv, bt2, 0, nr, image.data_ptr(), hl, stream=sa)
        if record: m["restore"][1].record(sa)
        ctx.sync(sa)
        if record: marks.append(m)
        return nr

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_ms = []

    def timed(e2e: bool):
        for _ in range(args.warmup):
            step(e2e, False)
        marks.clear()
        ctx.reset_counters()
        barrier()
        e0, e1 = ev(), ev()
        e0.record()
        nr = 0
        bounds = [e0]
        for _ in range(args.steps):
            nr = step(e2e, True)
            bounds.append(ev())
            bounds[-1].record()
        e1.record()
        barrier()
        step_ms[:] = [a.elapsed_time(b) for a, b in zip(bounds[:-1], bounds[1:])]
        ms, _ = job_totals(e0.elapsed_time(e1), 0.0, dist if world > 1 else None, dev)
        return ms / args.steps, nr, ctx.get_counters()

    sampler = ClockSampler(local)
    sampler.start()
    ms_step, nr, counters = timed(False)
    clocks = sampler.stop()
    step_stats = {"mean": ms_step, "median": statistics.median(step_ms), "min": min(step_ms), "max": max(step_ms),
                  "note": "per-step times from CUDA events on the default stream between steps (each step ends drained)"}
    phase = {k: statistics.mean(m[k][0].elapsed_time(m[k][1]) for m in marks)
             for k in ("offload", "stage", "match", "restore") if not (k == "stage" and not len(plan_arr))}
    variant_used = int(counters.last_variant)
    ms_e2e, _, _ = timed(True)

    # ---- in-HBM block gather / scatter of the same session (outside the step; the metric's
    # "gather GB/s vs HBM peak"): image in device memory, read + write bytes = 2 x payload
    d_image = torch.empty(n * shape.bytes_per_block, dtype=torch.uint8, device=dev)
    gather_ms = {}
    for name, fn in (("gather", lambda: ctx.kv_gather(kv, bt, 0, n, d_image, hl)),
                     ("scatter", lambda: ctx.kv_scatter(kv, bt2, 0, n, d_image, hl))):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        g0, g1 = ev(), ev()
        g0.record()
        for _ in range(5):
            fn()
        g1.record()
        torch.cuda.synchronize()
        gather_ms[name] = g0.elapsed_time(g1) / 5
    del d_image
    # the dominant kernel once more, alone on the GPU (context for the in-step figure)
    stage_alone_ms = None
    if len(plan_arr):
        for _ in range(2):
            ctx.stage_plan_run(prepared, None)
        torch.cuda.synchronize()
        g0, g1 = ev(), ev()
        g0.record()
        for _ in range(5):
            ctx.stage_plan_run(prepared, None)
        g1.record()
        torch.cuda.synchronize()
        stage_alone_ms = g0.elapsed_time(g1) / 5

    # prefix match of this session on the GPU alone: events around 100 back-to-back calls
    for _ in range(3):
        ctx.prefix_match(1, d_cont, co, d_sess, so, d_stored, 16, wl.HASH_SEED, d_hashes, d_res, stream=sa)
    ctx.sync(sa)
    g0, g1 = ev(), ev()
    g0.record(sa)
    for _ in range(100):
        ctx.prefix_match(1, d_cont, co, d_sess, so, d_stored, 16, wl.HASH_SEED, d_hashes, d_res, stream=sa)
    g1.record(sa)
    ctx.sync(sa)
    match_gpu_us = g0.elapsed_time(g1) * 10.0

    off_bytes, res_bytes = n * shape.bytes_per_block, nr * shape.bytes_per_block
    link_bytes = off_bytes + res_bytes
    value = world * link_bytes / (ms_step * 1e6)
    e2e_value = world * link_bytes / (ms_e2e * 1e6)

    # ---- self-check of the state the timed steps left behind (no oracle here: the
    # parity tests own that).  Sampled chunks must sit where the tables say, the match
    # must return the answer the generator constructed, staged samples must have landed.
    check = None
    if rank == 0 and not args.no_verify:
        check = True
        gs = wl.rng(2, 99)
        img_dev_view = image        # pinned host tensor
        for _ in range(64):
            l, p, i = int(gs.integers(0, shape.num_layers)), int(gs.integers(0, 2)), int(gs.integers(0, n))
            a = l * strides[0] + p * strides[1] + i * strides[2]
            chunk = img_dev_view[a:a + C]
            pl = planes[l * 2 + p].view(torch.uint8)
            check &= bool(torch.equal(pl[int(bt[i]) * C:(int(bt[i]) + 1) * C].cpu(), chunk))
            if i < nr:
                check &= bool(torch.equal(pl[int(bt2[i]) * C:(int(bt2[i]) + 1) * C].cpu(), chunk))
        r = h_res.numpy()
        check &= [int(r[0]), int(r[1]), int(r[2]), int(r[3]) & 0xFFFFFFFF] == [SHARED_TOKENS, SHARED_TOKENS // 16, SHARED_TOKENS // 16 * 16, 0]
        if len(plan_arr):
            for off, nb, _ in (plan[0], plan[len(plan) // 2], plan[-1]):
                check &= bool(torch.equal(slots[off:off + nb], staging[off:off + nb]))

    # ---- the other configurations, in the same run (rank 0 of a 1-GPU run; replicas only time the step)
    legs = {}
    if world == 1 and args.workload == "all" and args.scale == "full":
        peaks0, _ = measured_peaks()
        ctx.stage_plan_destroy(prepared) if prepared is not None else None
        ctx.destroy()
        del planes, staging, slots, image, kv, _keep
        _release_memory(torch)
        for key, name in (("prefix", "prefix"), ("configs2", "long"), ("configs4", "stage"), ("configs3", "replay")):
            legs[key] = run_leg(name, torch, dev, ceilings, float(peaks0["hbm_gbs"]))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peaks_kind = measured_peaks()
    hbm_peak = float(peaks["hbm_gbs"])
    off_gbs, res_gbs = off_bytes / (phase["offload"] * 1e6), res_bytes / (phase["restore"] * 1e6)
    link_ach = link_bytes / ((phase["offload"] + phase["restore"]) * 1e6)
    link_peak = link_bytes / (res_bytes / ceilings["h2d"] + off_bytes / ceilings["d2h"])
    host_link = {
        "bound": "host_link", "op": "kv_offload + kv_restore (variant %d)" % variant_used,
        "achieved": link_ach, "peak": link_peak, "unit": "GB/s", "frac": link_ach / link_peak,
        "peak_kind": "pinned cudaMemcpyAsync, 1 GiB, best of 6, measured in this run",
        "offload_gbs": off_gbs, "restore_gbs": res_gbs, "ceiling_d2h_gbs": ceilings["d2h"],
        "ceiling_h2d_gbs": ceilings["h2d"], "offload_frac": off_gbs / ceilings["d2h"],
        "restore_frac": res_gbs / ceilings["h2d"], "nominal_pcie5_x16_gbs": PCIE5_X16_GBS,
        "frac_of_nominal": link_ach / PCIE5_X16_GBS,
    }
    roofline = None
    if len(plan_arr):
        ach = 2 * stage_bytes / (phase["stage"] * 1e6)
        roofline = {"bound": "hbm", "kernel": "stage_copy_kernel", "achieved": ach, "peak": hbm_peak,
                    "unit": "GB/s", "frac": ach / hbm_peak,
                    "peak_kind": f"hbm_gbs of {peaks_kind} (MEASURED_PEAKS.json copy bandwidth)",
                    "frac_of_nominal_8tbs": ach / 8000.0, "algorithmic_bytes": 2 * stage_bytes,
                    "traffic": (STAGE_TRAFFIC_RATIO * 2 * stage_bytes) if STAGE_TRAFFIC_RATIO else None,
                    "launch_ms": phase["stage"], "alone_ms": stage_alone_ms,
                    "alone_achieved": 2 * stage_bytes / (stage_alone_ms * 1e6),
                    "alone_frac": 2 * stage_bytes / (stage_alone_ms * 1e6) / hbm_peak,
                    "note": "dominant kernel by GPU time; timed inside the step, where it shares the GPU "
                            "with the concurrent offload's packing kernels and DMA"}

    cpu = None
    if not args.no_cpu_baseline:
        gbs, cms, sample = time_oracle(1, 1)
        cpu = {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample, "ms_per_step": cms}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": ("configs[1]: " if args.scale == "full" else "profiling-sized cut of configs[1]: ") +
                               "Qwen3-235B-shaped KV (94 layers x 4 KV heads x 128, bf16, 16-token blocks), one "
                               f"{PREFIX_TOKENS:,}-token session: offload {n:,} blocks || stage {stage_bytes / 1e9:.2f} GB "
                               f"D2D, match {CONT_TOKENS:,}-token continuation, restore {nr:,} matched blocks",
                   "pool_blocks": POOL_BLOCKS, "host_layout": "page-first", "stage_chunk_bytes": STAGE_CHUNK,
                   "stage_bytes": stage_bytes, "variant": variant_used, "replicas": world, "scale": args.scale,
                   "l2": "every op streams inputs far larger than the 126 MB L2 (4.8 GB / 59 GB)"},
        "ms_per_step_stats": step_stats, "phases_ms": phase, "self_check": check,
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": res_bytes + (CONT_TOKENS + PREFIX_TOKENS) * 4 + (PREFIX_TOKENS // 16) * 8 + (n + nr) * 4,
                "d2h_bytes_per_step": off_bytes + 32 + (CONT_TOKENS // 16) * 8},
        "gpu_launches": int(counters.kernel_launches), "copy_engine_copies": int(counters.memcpy_calls),
        "roofline": roofline, "host_link": host_link,
        "hbm_gather": {"bound": "hbm", "kernel": "kv_copy_vec_kernel (talaria_kv_gather / talaria_kv_scatter)",
                       "gather_gbs": 2 * off_bytes / (gather_ms["gather"] * 1e6),
                       "scatter_gbs": 2 * off_bytes / (gather_ms["scatter"] * 1e6), "peak": hbm_peak, "unit": "GB/s",
                       "frac": 2 * off_bytes / (gather_ms["gather"] * 1e6) / hbm_peak,
                       "algorithmic_bytes": 2 * off_bytes, "timed": "alone, after the timed steps, 5 launches"},
        "cpu_baseline": cpu, "clocks": clocks,
        "prefix_match": {"us_per_call_gpu": match_gpu_us,
                         "tokens_per_s_gpu": (CONT_TOKENS + PREFIX_TOKENS) / (match_gpu_us * 1e-6),
                         "timed": "CUDA events around 100 back-to-back calls on one stream, stored hashes supplied",
                         "us_in_step_incl_marshalling_result_copy_and_sync": phase["match"] * 1e3},
    }
    line.update(legs)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", type=int, default=0, help="0 auto, 1 zero-copy, 2 bounce+DMA, 3 per-run DMA")
    ap.add_argument("--scale", default="full", choices=["full", "small"], help="small = profiling-sized workload")
    ap.add_argument("--workload", default="all", choices=["all", "session", "long", "stage", "replay", "sweep", "prefix"],
                    help="all = the timed configs[1] step plus configs[2..4] and the prefix lines as extra keys of the "
                         "one JSON line; session = the timed step only; long / replay / stage = configs[2] / [3] / [4] "
                         "alone; sweep = variant / size table; prefix = match latency and batch throughput")
    ap.add_argument("--pack-ctas", type=int, default=0, help="grid of the bounce variant's pack kernels (0 = library default)")
    ap.add_argument("--no-stage", action="store_true")
    ap.add_argument("--no-verify", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    apply_scale(args.scale)
    if args.impl == "reference":
        run_reference(args)
    elif args.workload not in ("all", "session"):
        run_other_workload(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
