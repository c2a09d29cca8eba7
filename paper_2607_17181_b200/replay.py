"""Session-replay driver: the residency policy around the library calls.

The library moves bytes; which session is evicted, when a prefix is restored and
where new blocks come from is the caller's policy (the paper's instance-local
cache, Sec. 4.1 / 4.3).  This driver plays a schedule of calls from many agent
sessions against one paged KV pool of fixed capacity:

  * every group of calls is prefix-matched in one batched call against the
    sessions' stored streams (App. A) -- `talaria_prefix_match_host`;
  * when a call finishes, its newly aligned (full) blocks are checkpointed to pinned
    host memory on a checkpoint stream, asynchronously, one extent per call
    (Sec. 4.1 / 4.3: checkpoint when a request finishes) -- `talaria_kv_offload`
    with a `first_block / n_blocks` sub-range;
  * a returning session whose KV is still in the pool keeps the matched blocks and
    frees the rest (checkpoint extents beyond the match are cut back); one whose KV
    lives only on the host gets new blocks and the matched prefix is restored into
    them, extent by extent (Sec. 4.3) -- `talaria_kv_restore_batch`; the restored
    blocks need no new checkpoint;
  * when the pool cannot hold a call, whole sessions are evicted in LRU order
    (ties: lower session id).  Eviction drains the victim's checkpoint event and
    copies only what is not on the host yet -- normally the partial tail block
    (App. B: the barrier usually waits only for the final tail blocks);
    when the host budget is exhausted the oldest host-only sessions are dropped and
    their next call recomputes everything ("host-cache capacity miss");
  * the KV of the unmatched tail is "computed": synthetic bytes are scattered
    into the new blocks -- `talaria_kv_scatter`.

`checkpoint="eviction"` is the simpler policy with no background checkpoints: the
whole session is copied when it is evicted.

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
class Extent:
    """Blocks [first, first + n) of a session, checkpointed in one call, as a dense host image."""
    first: int
    n: int
    image: object                 # pinned host tensor of n * bytes_per_block
    hl: object                    # its layout
    cap: int                      # blocks the image was sized for (n may be cut back later)


@dataclass
class SessionState:
    sid: int
    tokens: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))
    hashes: np.ndarray = field(default_factory=lambda: np.zeros(0, np.uint64))
    table: Optional[np.ndarray] = None        # block ids while resident in the pool
    where: str = "none"                       # "device" | "host" | "none"
    extents: List[Extent] = field(default_factory=list)
    event: object = None                      # end of the last checkpoint copy (torch.cuda.Event) or None
    last_use: int = -1

    @property
    def host_blocks(self) -> int:
        return self.extents[-1].first + self.extents[-1].n if self.extents else 0


@dataclass
class ReplayStats:
    calls: int = 0
    device_hits: int = 0
    host_restores: int = 0
    recomputes: int = 0
    capacity_misses: int = 0
    evictions: int = 0
    offload_bytes: int = 0        # all device-to-host KV bytes (checkpoints and evictions)
    restore_bytes: int = 0
    checkpoint_bytes: int = 0     # of which background checkpoints
    checkpoints_skipped: int = 0  # no host budget at checkpoint time
    evict_bytes_already_on_host: int = 0
    evict_bytes_copied: int = 0
    evict_stall_s: float = 0.0    # host time an eviction blocked: drain of the checkpoint event + tail copy
    evict_stalls: List[float] = field(default_factory=list)
    reused_tokens: int = 0
    prompt_tokens: int = 0
    offload_s: float = 0.0        # host wall time of the synchronous transfer calls, drained
    restore_s: float = 0.0
    match_s: float = 0.0
    match_calls: int = 0
    match_times: List[float] = field(default_factory=list)


class ReplayDriver:
    def __init__(self, ctx: tb.Talaria, shape: wl.KvShape, kv, pool_blocks: int, host_budget_bytes: int,
                 seed: int, content: Callable[[int, int, int], np.ndarray], alloc_pinned: Callable[[int], object],
                 to_device: Callable[[np.ndarray], object], order: str = "PF", log: Optional[list] = None,
                 free_pinned: Optional[Callable[[object], None]] = None, checkpoint: str = "incremental",
                 max_extent_blocks: int = 512, resident: Optional[Tuple[int, int]] = None):
        """content(session, call_index, nbytes) -> uint8 array: the synthetic KV of a call's new blocks.
        alloc_pinned(nbytes) -> pinned host tensor; free_pinned(tensor) gives it back (optional);
        to_device(array) -> device tensor (memory plumbing).
        checkpoint: "incremental" (after every call, asynchronously) or "eviction" (whole session when evicted).
        max_extent_blocks: a checkpoint is cut into host images of at most this many blocks, so the
        pinned allocator is never asked for one multi-gigabyte piece.
        resident: (sessions, longest prompt) -- keep every session's stream and block hashes on the device
        (two places per session, used in turn) and match with `talaria_prefix_match_resident`: only the new
        prompt crosses the host link.  None: every stream goes up from host memory with each match."""
        import torch
        assert checkpoint in ("incremental", "eviction")
        self.ctx, self.shape, self.kv = ctx, shape, kv
        self.pool_blocks, self.host_budget = pool_blocks, host_budget_bytes
        self.seed, self.order, self.checkpoint = seed, order, checkpoint
        self.max_extent_blocks = max(1, max_extent_blocks)
        self.content, self.alloc_pinned, self.to_device = content, alloc_pinned, to_device
        self.free_pinned = free_pinned
        self.free: List[int] = list(range(pool_blocks))      # min-heap: low addresses are reused first
        heapq.heapify(self.free)
        self.sessions: Dict[int, SessionState] = {}
        self.host_bytes = 0
        self.clock = 0
        self.stats = ReplayStats()
        self.log = log if log is not None else []
        self._torch = torch
        self.ckpt_stream = torch.cuda.Stream()
        self.resident = resident
        if resident is not None:
            n, longest = resident
            self.tok_stride, self.hash_stride = longest, longest // shape.block_tokens + 1
            self.d_tokens = torch.zeros(2 * n * self.tok_stride, dtype=torch.int32, device="cuda")
            self.d_hashes = torch.zeros(2 * n * self.hash_stride, dtype=torch.int64, device="cuda")
            self.place: Dict[int, List[int]] = {}            # session -> [index in the arrays, side holding its stream]

    # ------------------------------------------------------------ allocation
    def _alloc(self, n: int) -> np.ndarray:
        return np.array([heapq.heappop(self.free) for _ in range(n)], dtype=np.int32)

    def _release(self, ids: Sequence[int]):
        for b in ids:
            heapq.heappush(self.free, int(b))

    # ------------------------------------------------------------- host side
    def _extent_bytes(self, e: Extent) -> int:
        return e.cap * self.shape.bytes_per_block

    def _free_extent(self, e: Extent):
        self.host_bytes -= self._extent_bytes(e)
        if self.free_pinned is not None:
            self.free_pinned(e.image)

    def _drop_host(self, s: SessionState):
        """Forget everything the host holds of this session."""
        if s.event is not None:
            s.event.synchronize()                 # a copy into these images may still be running
            s.event = None
        for e in s.extents:
            self._free_extent(e)
        s.extents = []
        if s.where == "host":
            s.where = "none"

    def _truncate_host(self, s: SessionState, keep: int):
        """Keep only the checkpoints of blocks [0, keep): the rest describes KV that is being replaced."""
        if s.host_blocks <= keep:
            return
        if s.event is not None:
            s.event.synchronize()
            s.event = None
        kept = []
        for e in s.extents:
            if e.first >= keep:
                self._free_extent(e)
            else:
                e.n = min(e.n, keep - e.first)
                kept.append(e)
        s.extents = kept
        self.log.append(("truncate", s.sid, keep))

    def _host_room(self, nbytes: int, busy: set) -> bool:
        """Make room in the host budget by dropping the oldest host-only sessions."""
        while self.host_bytes + nbytes > self.host_budget:
            old = sorted((h for h in self.sessions.values() if h.where == "host" and h.sid not in busy),
                         key=lambda h: (h.last_use, h.sid))
            if not old:
                return False
            self._drop_host(old[0])
            self.log.append(("drop_host", old[0].sid))
        return True

    def _offload_range(self, s: SessionState, first: int, n: int, busy: set, stream=None) -> int:
        """Copy blocks [first, first + n) of a resident session to new host extents of bounded size.
        Returns the number of blocks that found room on the host (a prefix of the range)."""
        done = 0
        while done < n:
            m = min(self.max_extent_blocks, n - done)
            nbytes = m * self.shape.bytes_per_block
            if not self._host_room(nbytes, busy | {s.sid}):
                break
            try:
                image = self.alloc_pinned(nbytes)
            except MemoryError:                       # the pinned allocator is fragmented: same as no room
                break
            hl = tb.host_layout(wl.dense_strides(self.shape, m, self.order), nbytes)
            e = Extent(first + done, m, image, hl, m)
            self.host_bytes += nbytes
            s.extents.append(e)
            self.ctx.kv_offload(self.kv, s.table, e.first, m, e.image, e.hl, stream=stream)
            self.stats.offload_bytes += nbytes
            self.log.append(("checkpoint", s.sid, e.first, s.table[e.first:e.first + m].copy()))
            done += m
        return done

    def _checkpoint(self, s: SessionState, busy: set, fill_done):
        """Asynchronously checkpoint the session's newly aligned (full) blocks."""
        full = s.tokens.size // self.shape.block_tokens
        first = s.host_blocks
        n = full - first
        if n <= 0:
            return
        self.ckpt_stream.wait_event(fill_done)
        done = self._offload_range(s, first, n, busy, stream=self.ckpt_stream)
        if done < n:
            self.stats.checkpoints_skipped += 1
        if done:
            s.event = self._torch.cuda.Event()
            s.event.record(self.ckpt_stream)
            self.stats.checkpoint_bytes += done * self.shape.bytes_per_block

    # --------------------------------------------------------------- eviction
    def _make_room(self, need: int, busy: set):
        """Evict whole sessions, least recently used first, until `need` blocks are free."""
        if len(self.free) >= need:
            return
        victims = sorted((s for s in self.sessions.values() if s.where == "device" and s.sid not in busy),
                         key=lambda s: (s.last_use, s.sid))
        freed = len(self.free)
        for s in victims:
            if freed >= need:
                break
            t0 = time.perf_counter()
            n_all = len(s.table)
            first = s.host_blocks
            rest = n_all - first                                  # not on the host yet (normally the tail block)
            kept = True
            if rest > 0:
                done = self._offload_range(s, first, rest, busy)
                self.stats.evict_bytes_copied += done * self.shape.bytes_per_block
                kept = done == rest                               # no host room: this session's KV is lost
            # switch barrier for this session: its checkpoint copies and the tail copy are done
            if s.event is not None:
                s.event.synchronize()
                s.event = None
            self.ctx.sync()
            dt = time.perf_counter() - t0
            self.stats.evict_stall_s += dt
            self.stats.evict_stalls.append(dt)
            self.stats.offload_s += dt
            self.stats.evict_bytes_already_on_host += first * self.shape.bytes_per_block
            if not kept:
                self._drop_host(s)
            self.log.append(("evict" if kept else "evict_lost", s.sid, s.table.copy()))
            self._release(s.table)
            s.table = None
            s.where = "host" if kept else "none"
            self.stats.evictions += 1
            freed += n_all
        if freed < need:
            raise RuntimeError("pool too small for this call even after evicting every other session")

    # ------------------------------------------------------------------ calls
    def run_group(self, calls: Sequence[Tuple[int, int, np.ndarray]]):
        """calls: (session id, call index, prompt tokens); distinct sessions.  Returns the match records."""
        torch = self._torch
        B = self.shape.block_tokens
        self.clock += 1
        busy = {sid for sid, _, _ in calls}
        for sid, _, _ in calls:
            self.sessions.setdefault(sid, SessionState(sid))
        # ---- one batched match for the whole group -------------------------
        conts = [t for _, _, t in calls]
        res = np.zeros(len(calls), tb.MATCH_DTYPE)
        if self.resident is not None:
            pairs, outs = [], []
            for sid, _, toks in calls:
                pl = self.place.setdefault(sid, [len(self.place), 0])
                assert pl[0] < self.resident[0] and toks.size <= self.tok_stride
                here, there = 2 * pl[0] + pl[1], 2 * pl[0] + (pl[1] ^ 1)
                pairs.append((toks, there * self.tok_stride, there * self.hash_stride, here * self.tok_stride,
                              self.sessions[sid].tokens.size, here * self.hash_stride))
                outs.append((there * self.hash_stride, toks.size // B))
                pl[1] ^= 1                                    # the prompt becomes the stored stream
            t0 = time.perf_counter()
            self.ctx.prefix_match_resident(pairs, self.d_tokens, self.d_hashes, B, self.seed, res)
            dt = time.perf_counter() - t0
            got = [self.d_hashes[o:o + n].cpu().numpy().view(np.uint64) for o, n in outs]      # host copies, for the log
            out_h = np.concatenate(got) if got else np.zeros(0, np.uint64)
            out_h = out_h if out_h.size else np.zeros(1, np.uint64)
        else:
            sesss = [self.sessions[sid].tokens for sid, _, _ in calls]
            co = np.cumsum([0] + [c.size for c in conts]).astype(np.int64)
            so = np.cumsum([0] + [s.size for s in sesss]).astype(np.int64)
            cont_all = np.concatenate(conts) if co[-1] else np.zeros(1, np.int32)
            sess_all = np.concatenate(sesss) if so[-1] else np.zeros(1, np.int32)
            stored = np.concatenate([self.sessions[sid].hashes[: s.size // B] for (sid, _, _), s in zip(calls, sesss)])
            stored = stored if stored.size else np.zeros(1, np.uint64)
            out_h = np.zeros(max(int(sum(c.size // B for c in conts)), 1), np.uint64)
            t0 = time.perf_counter()
            self.ctx.prefix_match_host(len(calls), cont_all, co, sess_all, so, stored, B, self.seed, out_h, res)
            dt = time.perf_counter() - t0
        self.stats.match_s += dt
        self.stats.match_times.append(dt)
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
                self._truncate_host(s, reuse)
                if s.event is not None:
                    # blocks that are about to be rewritten may still be read by a checkpoint copy
                    torch.cuda.current_stream().wait_event(s.event)
                keep, drop = s.table[:reuse].copy(), s.table[reuse:]
                self._release(drop)
                s.table = keep
                self._make_room(need - reuse, busy)
                new = self._alloc(need - reuse)
                table = np.concatenate([keep, new]).astype(np.int32)
                self.stats.device_hits += 1
            elif s.where == "host":
                reuse = min(reuse, s.host_blocks)
                self._truncate_host(s, reuse)
                self._make_room(need, busy)
                table = self._alloc(need)
                if reuse:
                    for e in s.extents:
                        restores.append((table.copy(), e.first, e.n, e.image, e.hl))
                    self.log.append(("restore", sid, table[:reuse].copy()))
                    self.stats.restore_bytes += reuse * self.shape.bytes_per_block
                self.stats.host_restores += 1
            else:
                if s.last_use >= 0:
                    self.stats.capacity_misses += 1
                reuse = 0
                self._truncate_host(s, 0)
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
            self.ctx.kv_restore_batch(self.kv, restores)
            self.ctx.sync()
            self.stats.restore_s += time.perf_counter() - t0
        filled = []
        for s, k, toks, table, reuse, hashes in plans:
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
            filled.append(s)
        # ---- the call has finished: checkpoint its newly aligned blocks in the background ----
        if self.checkpoint == "incremental":
            fill_done = torch.cuda.Event()
            fill_done.record()
            for s in filled:
                self._checkpoint(s, busy, fill_done)
        return res

    def drain(self):
        """Wait for every outstanding checkpoint copy (switch barrier, App. B)."""
        self.ckpt_stream.synchronize()
        for s in self.sessions.values():
            s.event = None
