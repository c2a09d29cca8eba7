"""Session-replay driver: the eviction policy around the library calls.

The library moves bytes; which session is evicted, when a prefix is restored and
where new blocks come from is the caller's policy (the paper's instance-local
cache, Sec. 4.1 / 4.3).  This driver plays a schedule of calls from many agent
sessions against one paged KV pool of fixed capacity:

  * every group of calls is prefix-matched in one batched call against the
    sessions' stored streams (App. A) -- `talaria_prefix_match_host`;
  * a returning session whose KV is still in the pool keeps the matched blocks and
    frees the rest; one whose KV was moved to the host gets new blocks and the
    matched prefix is restored into them (Sec. 4.3) -- `talaria_kv_restore_batch`;
  * when the pool cannot hold a call, whole sessions are evicted in LRU order
    (ties: lower session id) to pinned host images -- `talaria_kv_offload_batch`;
    when the host budget is exhausted the oldest host images are dropped and the
    next call of that session recomputes everything ("host-cache capacity miss");
  * the KV of the unmatched tail is "computed": synthetic bytes are scattered
    into the new blocks -- `talaria_kv_scatter`.

Every byte-moving step is appended to `log` so a test can replay the same steps on
the CPU oracle; this module itself never imports the oracle.
"""
from __future__ import annotations

import heapq
import time
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import binding as tb
from . import workloads as wl


@dataclass
class SessionState:
    sid: int
    tokens: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))
    hashes: np.ndarray = field(default_factory=lambda: np.zeros(0, np.uint64))
    table: Optional[np.ndarray] = None        # block ids while resident in the pool
    where: str = "none"                       # "device" | "host" | "none"
    image: object = None                      # pinned host tensor while where == "host"
    image_blocks: int = 0
    last_use: int = -1


@dataclass
class ReplayStats:
    calls: int = 0
    device_hits: int = 0
    host_restores: int = 0
    recomputes: int = 0
    capacity_misses: int = 0
    evictions: int = 0
    offload_bytes: int = 0
    restore_bytes: int = 0
    reused_tokens: int = 0
    prompt_tokens: int = 0
    offload_s: float = 0.0        # host wall time of the batched calls, drained
    restore_s: float = 0.0
    match_s: float = 0.0
    match_calls: int = 0
    match_times: List[float] = field(default_factory=list)


class ReplayDriver:
    def __init__(self, ctx: tb.Talaria, shape: wl.KvShape, kv, pool_blocks: int, host_budget_bytes: int,
                 seed: int, content: Callable[[int, int, int], np.ndarray], alloc_pinned: Callable[[int], object],
                 to_device: Callable[[np.ndarray], object], order: str = "PF", log: Optional[list] = None,
                 free_pinned: Optional[Callable[[object], None]] = None):
        """content(session, call_index, nbytes) -> uint8 array: the synthetic KV of a call's new blocks.
        alloc_pinned(nbytes) -> pinned host tensor; free_pinned(tensor) gives it back (optional);
        to_device(array) -> device tensor (memory plumbing)."""
        self.ctx, self.shape, self.kv = ctx, shape, kv
        self.pool_blocks, self.host_budget = pool_blocks, host_budget_bytes
        self.seed, self.order = seed, order
        self.content, self.alloc_pinned, self.to_device = content, alloc_pinned, to_device
        self.free_pinned = free_pinned
        self.free: List[int] = list(range(pool_blocks))      # min-heap: low addresses are reused first
        heapq.heapify(self.free)
        self.sessions: Dict[int, SessionState] = {}
        self.host_bytes = 0
        self.clock = 0
        self.stats = ReplayStats()
        self.log = log if log is not None else []

    # ------------------------------------------------------------ allocation
    def _alloc(self, n: int) -> np.ndarray:
        return np.array([heapq.heappop(self.free) for _ in range(n)], dtype=np.int32)

    def _release(self, ids: Sequence[int]):
        for b in ids:
            heapq.heappush(self.free, int(b))

    def _drop_host(self, s: SessionState):
        self.host_bytes -= s.image_blocks * self.shape.bytes_per_block
        if self.free_pinned is not None and s.image is not None:
            self.free_pinned(s.image)
        s.image, s.image_blocks, s.where = None, 0, "none"

    def _make_room(self, need: int, busy: set):
        """Evict whole sessions, least recently used first, until `need` blocks are free."""
        if len(self.free) >= need:
            return
        victims = sorted((s for s in self.sessions.values() if s.where == "device" and s.sid not in busy),
                         key=lambda s: (s.last_use, s.sid))
        xfers, chosen, freed = [], [], len(self.free)
        for s in victims:
            if freed >= need:
                break
            n = len(s.table)
            nbytes = n * self.shape.bytes_per_block
            # host budget: drop the oldest host images first; if it still does not fit, the KV is lost
            while self.host_bytes + nbytes > self.host_budget:
                old = sorted((h for h in self.sessions.values() if h.where == "host" and h.sid not in busy),
                             key=lambda h: (h.last_use, h.sid))
                if not old:
                    break
                self._drop_host(old[0])
                self.log.append(("drop_host", old[0].sid))
            if self.host_bytes + nbytes <= self.host_budget:
                s.image = self.alloc_pinned(nbytes)
                s.image_blocks = n
                hl = tb.host_layout(wl.dense_strides(self.shape, n, self.order), nbytes)
                xfers.append((s.table.copy(), 0, n, s.image, hl))
                self.host_bytes += nbytes
            chosen.append(s)
            freed += n
        if freed < need:
            raise RuntimeError("pool too small for this call even after evicting every other session")
        if xfers:
            t0 = time.perf_counter()
            self.ctx.kv_offload_batch(self.kv, xfers)
            self.ctx.sync()                                   # drain before the blocks are reused (App. B)
            self.stats.offload_s += time.perf_counter() - t0
            self.stats.offload_bytes += sum(x[2] for x in xfers) * self.shape.bytes_per_block
        for s in chosen:
            kept = s.image is not None
            self.log.append(("offload" if kept else "evict_lost", s.sid, s.table.copy()))
            self._release(s.table)
            s.table = None
            s.where = "host" if kept else "none"
            self.stats.evictions += 1

    # ------------------------------------------------------------------ calls
    def run_group(self, calls: Sequence[Tuple[int, int, np.ndarray]]):
        """calls: (session id, call index, prompt tokens); distinct sessions.  Returns the match records."""
        B = self.shape.block_tokens
        self.clock += 1
        busy = {sid for sid, _, _ in calls}
        for sid, _, _ in calls:
            self.sessions.setdefault(sid, SessionState(sid))
        # ---- one batched match for the whole group -------------------------
        conts = [t for _, _, t in calls]
        sesss = [self.sessions[sid].tokens for sid, _, _ in calls]
        co = np.cumsum([0] + [c.size for c in conts]).astype(np.int64)
        so = np.cumsum([0] + [s.size for s in sesss]).astype(np.int64)
        cont_all = np.concatenate(conts) if co[-1] else np.zeros(1, np.int32)
        sess_all = np.concatenate(sesss) if so[-1] else np.zeros(1, np.int32)
        stored = np.concatenate([self.sessions[sid].hashes[: s.size // B] for (sid, _, _), s in zip(calls, sesss)])
        stored = stored if stored.size else np.zeros(1, np.uint64)
        out_h = np.zeros(max(int(sum(c.size // B for c in conts)), 1), np.uint64)
        res = np.zeros(len(calls), tb.MATCH_DTYPE)
        t0 = time.perf_counter()
        self.ctx.prefix_match_host(len(calls), cont_all, co, sess_all, so, stored, B, self.seed, out_h, res)
        self.stats.match_s += time.perf_counter() - t0
        self.stats.match_times.append(time.perf_counter() - t0)
        self.stats.match_calls += 1
        self.log.append(("match", [(sid, k) for sid, k, _ in calls], res.copy(), out_h.copy()))
        # ---- residency decisions, allocation ----------------------------------
        restores, plans, at = [], [], 0
        for q, (sid, k, toks) in enumerate(calls):
            s = self.sessions[sid]
            need = self.shape.blocks_for(toks.size)
            nbc = toks.size // B
            reuse = int(res[q]["reusable_tokens"]) // B
            if s.where == "device":
                reuse = min(reuse, len(s.table))
                keep, drop = s.table[:reuse].copy(), s.table[reuse:]
                self._release(drop)
                s.table = keep
                self._make_room(need - reuse, busy)
                new = self._alloc(need - reuse)
                table = np.concatenate([keep, new]).astype(np.int32)
                self.stats.device_hits += 1
            elif s.where == "host":
                reuse = min(reuse, s.image_blocks)
                self._make_room(need, busy)
                table = self._alloc(need)
                if reuse:
                    n_img = s.image_blocks
                    hl = tb.host_layout(wl.dense_strides(self.shape, n_img, self.order), n_img * self.shape.bytes_per_block)
                    restores.append((table.copy(), 0, reuse, s.image, hl, sid, n_img))
                self.stats.host_restores += 1
            else:
                if s.last_use >= 0:
                    self.stats.capacity_misses += 1
                reuse = 0
                self._make_room(need, busy)
                table = self._alloc(need)
                self.stats.recomputes += 1
            plans.append((s, k, toks, table, reuse, out_h[at:at + nbc].copy()))
            at += nbc
            self.stats.calls += 1
            self.stats.prompt_tokens += toks.size
            self.stats.reused_tokens += reuse * B
        # ---- restore the matched prefixes of all returning sessions in one call ----
        if restores:
            t0 = time.perf_counter()
            self.ctx.kv_restore_batch(self.kv, [r[:5] for r in restores])
            self.ctx.sync()
            self.stats.restore_s += time.perf_counter() - t0
            self.stats.restore_bytes += sum(r[2] for r in restores) * self.shape.bytes_per_block
            for table, _, reuse, _, _, sid, n_img in restores:
                self.log.append(("restore", sid, table[:reuse].copy(), n_img))
        for s, k, toks, table, reuse, hashes in plans:
            if s.where == "host":
                self._drop_host(s)
            # ---- "prefill" of the unmatched tail: synthetic KV scattered into the new blocks ----
            m = len(table) - reuse
            if m:
                img = self.content(s.sid, k, m * self.shape.bytes_per_block)
                d_img = self.to_device(img)
                il = tb.host_layout(wl.dense_strides(self.shape, m, "PF"), m * self.shape.bytes_per_block)
                self.ctx.kv_scatter(self.kv, table, reuse, m, d_img, il)
                self.ctx.sync()
                self.log.append(("fill", s.sid, k, table[reuse:].copy()))
            s.table, s.where = table, "device"
            s.tokens, s.hashes, s.last_use = toks, hashes, self.clock
        return res
