"""ctypes front end of the CPU oracle (``talaria_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It never touches CUDA, never imports the CUDA
package, and the CUDA package never imports it.

Every function takes and returns numpy arrays (host memory).  The arithmetic
lives in the C file; this module only marshals arguments -- except for the two
pieces of host bookkeeping at the end (page registry, stable-address layout),
whose definitions are written out directly with dicts, sets and loops.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "talaria_oracle.c")
_LIB = os.path.join(_HERE, "libtalaria_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, no threads)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _KvLayout(C.Structure):
    _fields_ = [
        ("num_layers", C.c_int32), ("num_kv_heads", C.c_int32), ("block_tokens", C.c_int32),
        ("head_dim", C.c_int32), ("elt_bytes", C.c_int32), ("num_planes", C.c_int32),
        ("num_blocks", C.c_int64), ("plane_base", C.POINTER(C.c_void_p)),
    ]


class _HostLayout(C.Structure):
    _fields_ = [("stride_layer", C.c_int64), ("stride_plane", C.c_int64),
                ("stride_block", C.c_int64), ("capacity_bytes", C.c_int64)]


class _Match(C.Structure):
    _fields_ = [("lcp_tokens", C.c_int64), ("matched_blocks", C.c_int64),
                ("reusable_tokens", C.c_int64), ("hash_token_disagree", C.c_int32),
                ("pad_", C.c_int32)]


class _Copy(C.Structure):
    _fields_ = [("src_dev", C.c_void_p), ("src_host", C.c_void_p), ("dst_dev", C.c_void_p),
                ("bytes", C.c_int64), ("chunk_id", C.c_int32), ("pad_", C.c_int32)]


class _StageStats(C.Structure):
    _fields_ = [("d2d_bytes", C.c_int64), ("h2d_bytes", C.c_int64),
                ("dirty_chunks", C.c_int64), ("missing_chunks", C.c_int64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_mix64.restype = C.c_uint64
        _lib.orc_mix64.argtypes = [C.c_uint64]
        _lib.orc_block_digest.restype = C.c_uint64
        _lib.orc_block_digest.argtypes = [C.c_void_p, C.c_int32]
        _lib.orc_block_hash.restype = C.c_int64
        _lib.orc_block_hash.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_void_p]
        _lib.orc_lcp_tokens.restype = C.c_int64
        _lib.orc_lcp_tokens.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64]
        _lib.orc_prefix_match.restype = C.c_int32
        _lib.orc_prefix_match.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p,
                                          C.c_int32, C.c_uint64, C.c_void_p, C.c_void_p,
                                          C.POINTER(_Match)]
        _lib.orc_prefix_agree.restype = C.c_int64
        _lib.orc_prefix_agree.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int64]
        for name in ("orc_kv_offload_elem", "orc_kv_offload_chunk",
                     "orc_kv_restore_elem", "orc_kv_restore_chunk"):
            f = getattr(_lib, name)
            f.restype = C.c_int32
            f.argtypes = [C.POINTER(_KvLayout), C.c_void_p, C.c_int64, C.c_int64, C.c_void_p,
                          C.POINTER(_HostLayout)]
        _lib.orc_kv_pages.restype = C.c_int32
        _lib.orc_kv_pages.argtypes = [C.POINTER(_KvLayout), C.c_void_p, C.c_int64, C.c_int64, C.c_void_p,
                                      C.c_int64, C.c_void_p, C.c_int32]
        _lib.orc_stage.restype = C.c_int32
        _lib.orc_stage.argtypes = [C.POINTER(_Copy), C.c_int64, C.c_void_p, C.POINTER(_StageStats)]
        _lib.orc_prestage.restype = C.c_int32
        _lib.orc_prestage.argtypes = [C.POINTER(_Copy), C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.POINTER(_StageStats)]
        _lib.orc_mark_dirty.restype = C.c_int64
        _lib.orc_mark_dirty.argtypes = [C.POINTER(_Copy), C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        _lib.orc_stage_validate.restype = C.c_int32
        _lib.orc_stage_validate.argtypes = [C.POINTER(_Copy), C.c_int64, C.c_void_p]
    return _lib


def _i32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


# ----------------------------------------------------------------- hashing


def mix64(z: int) -> int:
    return int(lib().orc_mix64(C.c_uint64(z & 0xFFFFFFFFFFFFFFFF)))


def block_digest(tokens) -> int:
    t = _i32(tokens)
    return int(lib().orc_block_digest(_ptr(t), t.size))


def block_hash(tokens, block_tokens: int, seed: int) -> np.ndarray:
    t = _i32(tokens)
    out = np.zeros(max(t.size // block_tokens, 0), dtype=np.uint64)
    n = lib().orc_block_hash(_ptr(t), t.size, block_tokens, C.c_uint64(seed), _ptr(out))
    assert n == out.size
    return out


def lcp_tokens(a, b) -> int:
    a = _i32(a)
    b = _i32(b)
    return int(lib().orc_lcp_tokens(_ptr(a), a.size, _ptr(b), b.size))


@dataclass
class Match:
    lcp_tokens: int
    matched_blocks: int
    reusable_tokens: int
    hash_token_disagree: int


def prefix_match(cont, sess, block_tokens: int, seed: int,
                 sess_hashes: Optional[np.ndarray] = None) -> Tuple[Match, np.ndarray]:
    cont = _i32(cont)
    sess = _i32(sess)
    nbc, nbs = cont.size // block_tokens, sess.size // block_tokens
    out = np.zeros(nbc, dtype=np.uint64)
    scratch = np.zeros(nbc + nbs + 1, dtype=np.uint64)
    sh = None
    if sess_hashes is not None:
        sh = np.ascontiguousarray(sess_hashes, dtype=np.uint64)
        assert sh.size >= nbs
    r = _Match()
    rc = lib().orc_prefix_match(_ptr(cont), cont.size, _ptr(sess), sess.size, _ptr(sh),
                                block_tokens, C.c_uint64(seed), _ptr(out), _ptr(scratch),
                                C.byref(r))
    assert rc == 0
    return Match(r.lcp_tokens, r.matched_blocks, r.reusable_tokens, r.hash_token_disagree), out


def prefix_agree(committed_blocks: Sequence[int], hashes: np.ndarray) -> int:
    cb = np.ascontiguousarray(committed_blocks, dtype=np.int64)
    h = np.ascontiguousarray(hashes, dtype=np.uint64)
    assert h.ndim == 2 and h.shape[0] == cb.size
    return int(lib().orc_prefix_agree(cb.size, _ptr(cb), _ptr(h), h.shape[1]))


# ------------------------------------------------------------ block tables


@dataclass
class KvShape:
    num_layers: int
    num_kv_heads: int
    block_tokens: int
    head_dim: int
    elt_bytes: int = 2
    num_planes: int = 2

    @property
    def chunk_bytes(self) -> int:
        return self.num_kv_heads * self.block_tokens * self.head_dim * self.elt_bytes


def host_strides(shape: KvShape, n_blocks: int, order: str) -> Tuple[int, int, int]:
    """(stride_layer, stride_plane, stride_block) in bytes of a dense host image
    of n_blocks logical blocks.  'LF' = layer, plane, block (App. C layer-first);
    'PF' = block, layer, plane (App. C page-first)."""
    c = shape.chunk_bytes
    if order == "LF":
        return shape.num_planes * n_blocks * c, n_blocks * c, c
    if order == "PF":
        return shape.num_planes * c, c, shape.num_layers * shape.num_planes * c
    raise ValueError(order)


def _kv_args(shape: KvShape, planes: List[np.ndarray], strides, host: np.ndarray):
    num_blocks = planes[0].size // shape.chunk_bytes
    assert len(planes) == shape.num_layers * shape.num_planes
    for p in planes:
        assert p.dtype == np.uint8 and p.flags.c_contiguous and p.size == num_blocks * shape.chunk_bytes
    arr = (C.c_void_p * len(planes))(*[p.ctypes.data for p in planes])
    kv = _KvLayout(shape.num_layers, shape.num_kv_heads, shape.block_tokens, shape.head_dim,
                   shape.elt_bytes, shape.num_planes, num_blocks,
                   C.cast(arr, C.POINTER(C.c_void_p)))
    hl = _HostLayout(strides[0], strides[1], strides[2], host.size)
    return kv, hl, arr


def _check_extent(shape: KvShape, strides, n: int, host: np.ndarray):
    if n <= 0:
        return
    last = ((shape.num_layers - 1) * strides[0] + (shape.num_planes - 1) * strides[1]
            + (n - 1) * strides[2] + shape.chunk_bytes)
    assert last <= host.size, "host image too small"


def _kv_call(name, shape, planes, block_table, first, n, host, strides):
    assert host.dtype == np.uint8 and host.flags.c_contiguous
    bt = _i32(block_table)
    assert 0 <= first and first + n <= bt.size
    _check_extent(shape, strides, n, host)
    kv, hl, keep = _kv_args(shape, planes, strides, host)
    rc = getattr(lib(), name)(C.byref(kv), _ptr(bt), first, n, host.ctypes.data, C.byref(hl))
    del keep
    if rc != 0:
        raise ValueError(f"{name}: rc={rc}")


def kv_offload(shape, planes, block_table, first, n, host, strides, form="chunk"):
    """host[l,p,i] <- pool_{l,p}[bt[first+i]] for i<n.  planes: list of uint8
    arrays, one per (layer, plane), each num_blocks*chunk_bytes long."""
    _kv_call(f"orc_kv_offload_{form}", shape, planes, block_table, first, n, host, strides)


def kv_restore(shape, planes, block_table, first, n, host, strides, form="chunk"):
    """pool_{l,p}[bt[first+i]] <- host[l,p,i] for i<n (planes are written)."""
    _kv_call(f"orc_kv_restore_{form}", shape, planes, block_table, first, n, host, strides)


def kv_pages(shape, planes, block_table, first, n, host_pool: np.ndarray, page_offsets, to_host: bool):
    """One page-first slab per logical block at host_pool[page_offsets[i]:]: offload when
    to_host, else restore (planes are written)."""
    bt = _i32(block_table)
    po = np.ascontiguousarray(page_offsets, dtype=np.int64)
    assert po.size >= n and 0 <= first and first + n <= bt.size
    assert host_pool.dtype == np.uint8 and host_pool.flags.c_contiguous
    kv, _hl, keep = _kv_args(shape, planes, (0, 0, 0), host_pool)
    rc = lib().orc_kv_pages(C.byref(kv), _ptr(bt), first, n, host_pool.ctypes.data, host_pool.size, _ptr(po),
                            1 if to_host else 0)
    del keep
    if rc != 0:
        raise ValueError(f"orc_kv_pages: rc={rc}")


# ------------------------------------------------------------------ stage


@dataclass
class StageStats:
    d2d_bytes: int
    h2d_bytes: int
    dirty_chunks: int
    missing_chunks: int


def _plan_array(staging: np.ndarray, hostcopy: Optional[np.ndarray], slots: np.ndarray, plan):
    """plan: sequence of (src_off or None, host_off or None, dst_off, nbytes, chunk_id);
    offsets are byte offsets into the staging / hostcopy / slots uint8 arrays."""
    arr = (_Copy * max(len(plan), 1))()
    for k, (so, ho, do, nb, cid) in enumerate(plan):
        arr[k].src_dev = None if so is None else staging.ctypes.data + so
        arr[k].src_host = None if (ho is None or hostcopy is None) else hostcopy.ctypes.data + ho
        arr[k].dst_dev = slots.ctypes.data + do
        arr[k].bytes = nb
        arr[k].chunk_id = cid
    return arr


def stage(staging: np.ndarray, hostcopy: Optional[np.ndarray], slots: np.ndarray, plan,
          dirty_bitmap: Optional[np.ndarray]) -> StageStats:
    arr = _plan_array(staging, hostcopy, slots, plan)
    bm = None if dirty_bitmap is None else np.ascontiguousarray(dirty_bitmap, dtype=np.uint8)
    st = _StageStats()
    rc = lib().orc_stage(arr, len(plan), _ptr(bm), C.byref(st))
    if rc != 0:
        raise ValueError(f"orc_stage rc={rc}")
    return StageStats(st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks)


def stage_validate(staging, hostcopy, slots, plan, dirty_bitmap) -> bool:
    arr = _plan_array(staging, hostcopy, slots, plan)
    bm = None if dirty_bitmap is None else np.ascontiguousarray(dirty_bitmap, dtype=np.uint8)
    return bool(lib().orc_stage_validate(arr, len(plan), _ptr(bm)))


def prestage(staging: np.ndarray, hostcopy: np.ndarray, plan, blocked: Optional[np.ndarray],
             staged: np.ndarray, dirty: np.ndarray) -> StageStats:
    """plan: (staging_off, host_off, dst_off(unused), nbytes, chunk_id); staging is written;
    staged / dirty bitmaps (uint8, LSB-first) are updated in place."""
    arr = _plan_array(staging, hostcopy, staging, plan)
    bl = None if blocked is None else np.ascontiguousarray(blocked, dtype=np.uint8)
    st = _StageStats()
    rc = lib().orc_prestage(arr, len(plan), _ptr(bl), _ptr(staged), _ptr(dirty), C.byref(st))
    if rc != 0:
        raise ValueError(f"orc_prestage rc={rc}")
    return StageStats(st.d2d_bytes, st.h2d_bytes, st.dirty_chunks, st.missing_chunks)


def mark_dirty(staging: np.ndarray, plan, alloc_off: int, alloc_bytes: int, staged: Optional[np.ndarray],
               dirty: np.ndarray) -> int:
    arr = _plan_array(staging, None, staging, plan)
    return int(lib().orc_mark_dirty(arr, len(plan), staging.ctypes.data + alloc_off, alloc_bytes,
                                    _ptr(staged), _ptr(dirty)))


# ---------------------------------------------------------------- registry


class Registry:
    """Plain-dict definition of the page registry (Sec. 4.3: blocks keyed by cumulative
    prefix hash): first insert wins, lookup_prefix counts the leading hashes present."""

    def __init__(self):
        self.d = {}

    def insert(self, hashes, page_offsets) -> int:
        new = 0
        for h, o in zip(hashes, page_offsets):
            if int(h) not in self.d:
                self.d[int(h)] = int(o)
                new += 1
        return new

    def lookup_prefix(self, hashes):
        out = []
        for h in hashes:
            if int(h) not in self.d:
                break
            out.append(self.d[int(h)])
        return len(out), np.array(out, dtype=np.int64)

    def erase(self, hashes) -> int:
        gone = 0
        for h in hashes:
            if self.d.pop(int(h), None) is not None:
                gone += 1
        return gone

    def __len__(self):
        return len(self.d)


# ------------------------------------------------------- stable-address layout


class BumpLayout:
    """Plain definition of the stable-address HBM layout (Sec. 4.2) and its staging surface
    (Sec. 4.4), written out with Python sets and loops; offsets are relative to the region base.

    Layout of a model (weights up from the low end, runtime buffers anchored high, the gap is
    the KV pool of LP planes x NB rows of C bytes):
        weights [0, W);  runtime [R, R + Rt) with R = floor((S - Rt) / A) * A;
        K = ceil(W / A) * A;  NB = floor((R - K) / (LP * C));  plane k = [K + k*NB*C, +NB*C).
    Block ids are allocated lowest first, skipping rows under an active staging write; an
    allocated id is a row of every plane and dirties each staged chunk that owns that row.
    Staging for model `nxt`: chunk j takes the next usable tail slot, slots enumerated tail
    slot by tail slot across planes; slot t of a plane = rows [NB-(t+1)r, NB-t*r) with
    r = ceil(chunk / C); usable = all rows free and unlocked, and no byte below ceil(W_nxt/A)*A."""

    def __init__(self, region_bytes: int, align: int, models):
        """models: list of (weight_bytes, runtime_bytes, num_layers, num_planes, chunk_bytes)."""
        self.S, self.A, self.models = region_bytes, align, [tuple(m) for m in models]
        self.active = None

    def view(self, m: int):
        W, Rt, L, P, Cb = self.models[m]
        A = self.A
        K = -(-W // A) * A
        R = (self.S - Rt) // A * A
        NB = (R - K) // (L * P * Cb) if R >= K else 0
        if NB < 1:
            raise ValueError("region too small for this model")
        return {"weights": (0, W), "runtime": (R, Rt), "kv": (K, L * P * NB * Cb), "num_blocks": NB,
                "planes": [K + k * NB * Cb for k in range(L * P)]}

    def activate(self, m: int):
        self.active = m
        self.NB = self.view(m)["num_blocks"]
        self.free = set(range(self.NB))
        self.chunks = []            # per chunk: None or (plane, row0)
        self.locked = set()
        self.r = 0

    def _locked_rows(self):
        rows = set()
        for c in self.locked:
            if self.chunks[c] is not None:
                rows.update(range(self.chunks[c][1], self.chunks[c][1] + self.r))
        return rows

    def alloc_blocks(self, n: int, staged=None, dirty=None):
        """Returns (ids, newly dirtied chunk ids).  staged / dirty: Python sets of chunk ids."""
        avail = sorted(self.free - self._locked_rows())
        if len(avail) < n:
            raise MemoryError("not enough free blocks")
        ids = avail[:n]
        newly = []
        for b in ids:
            self.free.discard(b)
            for c, place in enumerate(self.chunks):
                if place is None or dirty is None:
                    continue
                if place[1] <= b < place[1] + self.r and (staged is None or c in staged) and c not in dirty:
                    dirty.add(c)
                    newly.append(c)
        return ids, newly

    def free_blocks(self, ids):
        ids = list(ids)
        if len(set(ids)) != len(ids) or any(b < 0 or b >= self.NB or b in self.free for b in ids):
            raise ValueError("bad id in free_blocks")
        self.free.update(ids)

    def _usable_slots(self, nxt: int, chunk_bytes: int, taken=()):
        W2 = self.models[nxt][0]
        lim = -(-W2 // self.A) * self.A
        _, _, L, P, Cb = self.models[self.active]
        planes = self.view(self.active)["planes"]
        r = -(-chunk_bytes // Cb)
        blocked = self._locked_rows()
        out = []
        for t in range(self.NB // r):
            row0 = self.NB - (t + 1) * r
            rows = range(row0, row0 + r)
            for k in range(L * P):
                if (k, row0) in taken:
                    continue
                if planes[k] + row0 * Cb < lim:
                    continue
                if all(x in self.free and x not in blocked for x in rows):
                    out.append((k, row0))
        return out, r

    def stage_place(self, nxt: int, chunk_bytes: int):
        """Returns the plan: per chunk (staging offset or None, weights offset, nbytes)."""
        W2 = self.models[nxt][0]
        n_chunks = -(-W2 // chunk_bytes)
        self.chunks, self.locked = [], set()
        slots, self.r = self._usable_slots(nxt, chunk_bytes)
        planes = self.view(self.active)["planes"]
        Cb = self.models[self.active][4]
        plan = []
        for j in range(n_chunks):
            place = slots[j] if j < len(slots) else None
            self.chunks.append(place)
            nbytes = min(chunk_bytes, W2 - j * chunk_bytes)
            plan.append((None if place is None else planes[place[0]] + place[1] * Cb, j * chunk_bytes, nbytes))
        return plan

    def staging_slack(self, nxt: int, chunk_bytes: int) -> int:
        Cb = self.models[self.active][4]
        same = self.r == -(-chunk_bytes // Cb)
        taken = {p for p in self.chunks if p is not None} if same else set()
        saved = self.r
        slots, _ = self._usable_slots(nxt, chunk_bytes, taken)
        self.r = saved
        return len(slots) * chunk_bytes
