"""Helpers for the GPU parity tests: device pools and pinned images with canary
guard bands (torch is used for device / pinned memory only)."""
import numpy as np
import torch

from oracle import oracle as orc
from paper_2607_17181_b200 import binding as tb

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
