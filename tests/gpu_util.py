"""Helpers for the GPU parity tests: device pools and pinned images with canary
guard bands (torch is used for device / pinned memory only)."""
import numpy as np
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl

GUARD = 4096
CANARY = 0xA5


def oshape(s):
    return orc.KvShape(s.num_layers, s.num_kv_heads, s.block_tokens, s.head_dim, s.elt_bytes, s.num_planes)


class GuardedDevice:
    """A device byte buffer with canary bands before and after the payload."""

    def __init__(self, nbytes, fill=None, align_off=0):
        self.n = nbytes
        self.t = torch.full((nbytes + 2 * GUARD + 64,), CANARY, dtype=torch.uint8, device="cuda")
        base = self.t.data_ptr()
        self.off = GUARD + ((-(base + GUARD)) % 256) % 256 + align_off
        if fill is not None:
            self.write(fill)

    @property
    def ptr(self):
        return self.t.data_ptr() + self.off

    def view(self):
        return self.t[self.off:self.off + self.n]

    def write(self, arr):
        self.view().copy_(torch.from_numpy(np.ascontiguousarray(arr).view(np.uint8).reshape(-1)))

    def read(self):
        return self.view().cpu().numpy()

    def guards_ok(self):
        h = self.t.cpu().numpy()
        return bool(np.all(h[:self.off] == CANARY) and np.all(h[self.off + self.n:] == CANARY))


class GuardedPinned:
    """A pinned host byte buffer with canary bands."""

    def __init__(self, nbytes, fill=0):
        self.n = nbytes
        self.t = torch.empty(nbytes + 2 * GUARD, dtype=torch.uint8, pin_memory=True)
        self.np_all = self.t.numpy()
        self.np_all[:] = CANARY
        self.np = self.np_all[GUARD:GUARD + nbytes]
        self.np[:] = fill

    @property
    def ptr(self):
        return self.t.data_ptr() + GUARD

    def guards_ok(self):
        return bool(np.all(self.np_all[:GUARD] == CANARY) and np.all(self.np_all[GUARD + self.n:] == CANARY))


class DevicePool:
    """Paged KV pool on the device: one guarded buffer per (layer, plane)."""

    def __init__(self, shape, planes_np):
        self.shape = shape
        self.num_blocks = planes_np[0].size // shape.chunk_bytes
        self.bufs = [GuardedDevice(p.size, p) for p in planes_np]
        self.kv, self._keep = tb.kv_layout(shape, [b.ptr for b in self.bufs], self.num_blocks)

    def read(self):
        return [b.read() for b in self.bufs]

    def guards_ok(self):
        return all(b.guards_ok() for b in self.bufs)


class ReplayMirror:
    """The oracle's copy of the driver's state: pool planes and, per session, checkpoint extents."""

    def __init__(self, shape, planes, order):
        self.shape, self.oshape = shape, orc.KvShape(shape.num_layers, shape.num_kv_heads, shape.block_tokens, shape.head_dim)
        self.planes, self.order = planes, order
        self.ext = {}                                   # sid -> list of [first, n, cap, image]

    def apply(self, entry, calls, before, content):
        shape, op = self.shape, entry[0]
        if op == "match":
            _, ids, got, hashes = entry
            at = 0
            for q, (sid, k) in enumerate(ids):
                m, hc = orc.prefix_match(calls[q][2], before[sid], shape.block_tokens, wl.HASH_SEED)
                assert (int(got[q]["lcp_tokens"]), int(got[q]["matched_blocks"]), int(got[q]["reusable_tokens"]),
                        int(got[q]["hash_token_disagree"])) == (m.lcp_tokens, m.matched_blocks, m.reusable_tokens, 0)
                assert np.array_equal(hashes[at:at + hc.size], hc)
                at += hc.size
        elif op == "checkpoint":
            _, sid, first, ids = entry
            img = np.zeros(ids.size * shape.bytes_per_block, np.uint8)
            orc.kv_offload(self.oshape, self.planes, ids, 0, ids.size, img, wl.dense_strides(shape, ids.size, self.order))
            exts = self.ext.setdefault(sid, [])
            assert first == (exts[-1][0] + exts[-1][1] if exts else 0)          # extents are appended in order
            exts.append([first, ids.size, ids.size, img])
        elif op == "truncate":
            _, sid, keep = entry
            self.ext[sid] = [[f, min(n, keep - f), cap, img] for f, n, cap, img in self.ext.get(sid, []) if f < keep]
        elif op in ("drop_host", "evict_lost"):
            self.ext.pop(entry[1], None)
        elif op == "evict":
            pass
        elif op == "restore":
            _, sid, table = entry
            covered = 0
            for f, n, cap, img in self.ext[sid]:
                orc.kv_restore(self.oshape, self.planes, table, f, n, img, wl.dense_strides(shape, cap, self.order))
                covered += n
            assert covered == table.size
        elif op == "fill":
            _, sid, k, ids = entry
            img = content(sid, k, ids.size * shape.bytes_per_block)
            orc.kv_restore(self.oshape, self.planes, ids, 0, ids.size, img, wl.dense_strides(shape, ids.size, "PF"))
        else:
            raise AssertionError(op)

    def check_host_images(self, drv):
        drv.drain()
        for sid, s in drv.sessions.items():
            mine = self.ext.get(sid, [])
            assert [(e.first, e.n, e.cap) for e in s.extents] == [(f, n, cap) for f, n, cap, _ in mine], sid
            for e, (_, _, _, img) in zip(s.extents, mine):
                assert np.array_equal(e.image.numpy(), img), sid


class PinnedArena:
    """One pinned allocation handed out in pieces (best fit, explicit frees): page-locking is slow,
    and a replay allocates and frees many host images."""

    def __init__(self, nbytes):
        self.t = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
        self.free = [(0, nbytes)]

    def alloc(self, nbytes):
        need = -(-nbytes // 4096) * 4096
        fits = [k for k, (_, ln) in enumerate(self.free) if ln >= need]
        if not fits:
            raise MemoryError("pinned arena exhausted")
        k = min(fits, key=lambda j: self.free[j][1])
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
