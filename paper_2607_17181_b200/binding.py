"""Thin ctypes binding of libtalaria (argument marshalling only).

Every method has the name of the C entry point it calls (``include/talaria.h``)
and passes raw pointers: device memory comes from ``tensor.data_ptr()`` of torch
tensors, host memory from pinned torch tensors or numpy arrays.  Nothing is
computed here and there is no fallback: if the CUDA library is missing the
import of :func:`lib` fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB_PATH = os.path.join(_HERE, "libtalaria.so")
SOURCES = ["ctx.cu", "kv_copy.cu", "prefix.cu", "prefix_pair.cu", "stage.cu", "registry.cu", "bump.cu"]
HEADERS = ["internal.h", "prefix_common.cuh"]

OK = 0
ERR_INVALID_ARG, ERR_BAD_BLOCK_ID, ERR_DUP_BLOCK, ERR_HOST_NOT_PINNED = -1, -2, -3, -4
ERR_EXTENT, ERR_OVERLAP, ERR_CUDA, ERR_NO_MEMORY = -5, -6, -7, -9
VARIANT_AUTO, VARIANT_ZEROCOPY, VARIANT_BOUNCE, VARIANT_RUNS = 0, 1, 2, 3


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the CUDA sources for sm_100a into libtalaria.so (in-tree)."""
    srcs = [os.path.join(_CSRC, s) for s in SOURCES]
    deps = srcs + [os.path.join(_CSRC, h) for h in HEADERS] + [os.path.join(_INCLUDE, "talaria.h")]
    if not force and os.path.exists(LIB_PATH) and all(
            os.path.getmtime(LIB_PATH) >= os.path.getmtime(d) for d in deps):
        return LIB_PATH
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", _INCLUDE, "-I", _CSRC, "-o", tmp] + srcs
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


class Config(C.Structure):
    _fields_ = [("bounce_bytes", C.c_int64), ("dma_min_bytes", C.c_int64), ("variant", C.c_int32),
                ("validate", C.c_int32), ("zc_ctas", C.c_int32), ("pack_ctas", C.c_int32),
                ("host_match_bytes", C.c_int64), ("reload_ctas", C.c_int32), ("reserved", C.c_int32)]


class KvLayout(C.Structure):
    _fields_ = [("num_layers", C.c_int32), ("num_kv_heads", C.c_int32), ("block_tokens", C.c_int32),
                ("head_dim", C.c_int32), ("elt_bytes", C.c_int32), ("num_planes", C.c_int32),
                ("num_blocks", C.c_int64), ("plane_base", C.POINTER(C.c_void_p))]


class HostLayout(C.Structure):
    _fields_ = [("stride_layer", C.c_int64), ("stride_plane", C.c_int64), ("stride_block", C.c_int64),
                ("capacity_bytes", C.c_int64)]


class Match(C.Structure):
    _fields_ = [("lcp_tokens", C.c_int64), ("matched_blocks", C.c_int64), ("reusable_tokens", C.c_int64),
                ("hash_token_disagree", C.c_int32), ("reserved", C.c_int32)]


MATCH_DTYPE = np.dtype([("lcp_tokens", "<i8"), ("matched_blocks", "<i8"), ("reusable_tokens", "<i8"),
                        ("hash_token_disagree", "<i4"), ("reserved", "<i4")])


class Copy(C.Structure):
    _fields_ = [("src_dev", C.c_void_p), ("src_host", C.c_void_p), ("dst_dev", C.c_void_p),
                ("bytes", C.c_int64), ("chunk_id", C.c_int32), ("reserved", C.c_int32)]


COPY_DTYPE = np.dtype([("src_dev", "<u8"), ("src_host", "<u8"), ("dst_dev", "<u8"), ("bytes", "<i8"),
                       ("chunk_id", "<i4"), ("reserved", "<i4")])


class StageStats(C.Structure):
    _fields_ = [("d2d_bytes", C.c_int64), ("h2d_bytes", C.c_int64), ("dirty_chunks", C.c_int64),
                ("missing_chunks", C.c_int64)]


class Counters(C.Structure):
    _fields_ = [("kernel_launches", C.c_int64), ("memcpy_calls", C.c_int64), ("payload_bytes", C.c_int64),
                ("last_variant", C.c_int32), ("reserved", C.c_int32)]


class ModelDesc(C.Structure):
    _fields_ = [("weight_bytes", C.c_int64), ("runtime_bytes", C.c_int64), ("num_layers", C.c_int32),
                ("num_planes", C.c_int32), ("chunk_bytes", C.c_int64)]


class BumpView(C.Structure):
    _fields_ = [("weights_base", C.c_void_p), ("weights_bytes", C.c_int64), ("kv_base", C.c_void_p),
                ("kv_bytes", C.c_int64), ("runtime_base", C.c_void_p), ("runtime_bytes", C.c_int64),
                ("num_blocks", C.c_int64)]


class Timing(C.Structure):
    _fields_ = [("total_ms", C.c_float), ("d2d_ms", C.c_float), ("h2d_ms", C.c_float), ("d2h_ms", C.c_float),
                ("op", C.c_int32), ("reserved", C.c_int32)]


class ResidentPair(C.Structure):
    _fields_ = [("h_cont_tokens", C.c_void_p), ("cont_tokens", C.c_int64), ("cont_slot", C.c_int64),
                ("cont_hash_slot", C.c_int64), ("sess_slot", C.c_int64), ("sess_tokens", C.c_int64),
                ("sess_hash_slot", C.c_int64)]


class KvXfer(C.Structure):
    _fields_ = [("block_table", C.c_void_p), ("first_block", C.c_int64), ("n_blocks", C.c_int64),
                ("host", C.c_void_p), ("hl", HostLayout)]


_P = C.c_void_p
_SIGNATURES = {
    "talaria_create": (C.c_int32, [C.POINTER(_P), C.c_int32, C.POINTER(Config)]),
    "talaria_destroy": (C.c_int32, [_P]),
    "talaria_host_register": (C.c_int32, [_P, _P, C.c_size_t]),
    "talaria_host_unregister": (C.c_int32, [_P, _P]),
    "talaria_block_hash": (C.c_int32, [_P, _P, C.c_int64, C.c_int32, C.c_uint64, _P, _P]),
    "talaria_prefix_match": (C.c_int32, [_P, C.c_int32, _P, _P, _P, _P, _P, C.c_int32, C.c_uint64, _P, _P, _P]),
    "talaria_prefix_match_host": (C.c_int32, [_P, C.c_int32, _P, _P, _P, _P, _P, C.c_int32, C.c_uint64, _P, _P, _P]),
    "talaria_prefix_match_resident": (C.c_int32, [_P, C.c_int32, _P, _P, C.c_int64, _P, C.c_int64, C.c_int32,
                                                  C.c_uint64, _P, _P]),
    "talaria_prefix_match_static": (C.c_int32, [C.c_int32, _P, _P, _P, _P, _P, C.c_int32, C.c_uint64, _P, _P, _P]),
    "talaria_prefix_agree": (C.c_int64, [C.c_int32, _P, _P, C.c_int64]),
    "talaria_registry_create": (C.c_int32, [C.POINTER(_P), C.c_int64]),
    "talaria_registry_destroy": (C.c_int32, [_P]),
    "talaria_registry_insert": (C.c_int32, [_P, _P, _P, C.c_int64, C.POINTER(C.c_int64)]),
    "talaria_registry_lookup_prefix": (C.c_int64, [_P, _P, C.c_int64, _P]),
    "talaria_registry_erase": (C.c_int32, [_P, _P, C.c_int64, C.POINTER(C.c_int64)]),
    "talaria_registry_size": (C.c_int64, [_P]),
    "talaria_kv_offload": (C.c_int32, [_P, C.POINTER(KvLayout), _P, C.c_int64, C.c_int64, _P, C.POINTER(HostLayout), _P]),
    "talaria_kv_restore": (C.c_int32, [_P, C.POINTER(KvLayout), _P, C.c_int64, C.c_int64, _P, C.POINTER(HostLayout), _P]),
    "talaria_kv_restore_layered": (C.c_int32, [_P, C.POINTER(KvLayout), _P, C.c_int64, C.c_int64, _P, C.POINTER(HostLayout), _P, _P]),
    "talaria_kv_offload_pages": (C.c_int32, [_P, C.POINTER(KvLayout), _P, C.c_int64, C.c_int64, _P, C.c_int64, _P, _P]),
    "talaria_kv_restore_pages": (C.c_int32, [_P, C.POINTER(KvLayout), _P, C.c_int64, C.c_int64, _P, C.c_int64, _P, _P]),
    "talaria_kv_gather": (C.c_int32, [_P, C.POINTER(KvLayout), _P, C.c_int64, C.c_int64, _P, C.POINTER(HostLayout), _P]),
    "talaria_kv_scatter": (C.c_int32, [_P, C.POINTER(KvLayout), _P, C.c_int64, C.c_int64, _P, C.POINTER(HostLayout), _P]),
    "talaria_kv_offload_batch": (C.c_int32, [_P, C.POINTER(KvLayout), C.POINTER(KvXfer), C.c_int32, _P]),
    "talaria_kv_restore_batch": (C.c_int32, [_P, C.POINTER(KvLayout), C.POINTER(KvXfer), C.c_int32, _P]),
    "talaria_stage": (C.c_int32, [_P, _P, C.c_int64, _P, C.POINTER(StageStats), _P]),
    "talaria_stage_plan_create": (C.c_int32, [_P, _P, C.c_int64, C.POINTER(_P)]),
    "talaria_stage_plan_run": (C.c_int32, [_P, _P, _P, C.POINTER(StageStats), _P]),
    "talaria_stage_plan_destroy": (C.c_int32, [_P, _P]),
    "talaria_prestage": (C.c_int32, [_P, _P, C.c_int64, _P, _P, _P, C.POINTER(StageStats), _P]),
    "talaria_mark_dirty": (C.c_int64, [_P, C.c_int64, _P, C.c_int64, _P, _P]),
    "talaria_bump_create": (C.c_int32, [C.POINTER(_P), _P, C.c_int64, C.c_int64, C.POINTER(ModelDesc), C.c_int32]),
    "talaria_bump_destroy": (C.c_int32, [_P]),
    "talaria_bump_view": (C.c_int32, [_P, C.c_int32, C.POINTER(BumpView), _P]),
    "talaria_bump_activate": (C.c_int32, [_P, C.c_int32, C.POINTER(BumpView)]),
    "talaria_bump_alloc_blocks": (C.c_int32, [_P, C.c_int64, _P, _P, _P, C.POINTER(C.c_int64)]),
    "talaria_bump_free_blocks": (C.c_int32, [_P, _P, C.c_int64]),
    "talaria_bump_free_count": (C.c_int64, [_P]),
    "talaria_bump_stage_place": (C.c_int32, [_P, C.c_int32, C.c_int64, _P, _P, C.c_int64, C.POINTER(C.c_int64),
                                             C.POINTER(C.c_int64)]),
    "talaria_bump_lock_chunk": (C.c_int32, [_P, C.c_int32, C.c_int32]),
    "talaria_bump_staging_slack": (C.c_int64, [_P, C.c_int32, C.c_int64]),
    "talaria_check_block_table": (C.c_int32, [_P, C.c_int64, C.c_int64, C.c_int32]),
    "talaria_check_image_layout": (C.c_int32, [C.POINTER(KvLayout), C.c_int64, C.POINTER(HostLayout), C.POINTER(C.c_int64)]),
    "talaria_check_stage_plan": (C.c_int32, [_P, C.c_int64, _P, C.POINTER(StageStats)]),
    "talaria_sync": (C.c_int32, [_P, _P]),
    "talaria_strerror": (C.c_char_p, [C.c_int32]),
    "talaria_last_cuda_error": (C.c_int32, [_P]),
    "talaria_get_counters": (C.c_int32, [_P, C.POINTER(Counters)]),
    "talaria_reset_counters": (C.c_int32, [_P]),
    "talaria_set_timing": (C.c_int32, [_P, C.c_int32]),
    "talaria_get_timing": (C.c_int32, [_P, C.POINTER(Timing)]),
}

_lib = None


def lib():
    """The loaded CUDA library.  Raises if it has not been built: there is no
    CPU or PyTorch fallback for any operation."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run __graft_entry__.build() (nvcc, sm_100a) first")
        _lib = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            f = getattr(_lib, name)
            f.restype, f.argtypes = res, args
    return _lib


class TalariaError(RuntimeError):
    def __init__(self, status: int, what: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        msg = lib().talaria_strerror(status).decode()
        super().__init__(f"{what}: {msg} (status {status}, cuda error {cuda_error})")


def _ptr(x) -> Optional[int]:
    """Raw address of a torch tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()  # torch tensor


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int64)


def kv_layout(shape, plane_ptrs: Sequence[int], num_blocks: int):
    """(KvLayout, keep-alive) from a shape with the paper's descriptor fields and a
    list of device addresses, one per (layer, plane)."""
    n = shape.num_layers * shape.num_planes
    assert len(plane_ptrs) == n
    arr = (C.c_void_p * n)(*plane_ptrs)
    kv = KvLayout(shape.num_layers, shape.num_kv_heads, shape.block_tokens, shape.head_dim,
                  shape.elt_bytes, shape.num_planes, num_blocks, C.cast(arr, C.POINTER(C.c_void_p)))
    return kv, arr


def host_layout(strides, capacity_bytes: int) -> HostLayout:
    return HostLayout(strides[0], strides[1], strides[2], capacity_bytes)


def check_block_table(block_table, num_blocks: int, reject_duplicates: bool) -> int:
    bt = _i32(block_table)
    return int(lib().talaria_check_block_table(_ptr(bt), bt.size, num_blocks, 1 if reject_duplicates else 0))


def check_image_layout(shape, num_blocks: int, n_blocks: int, strides, capacity_bytes: int):
    """(status, contiguous run bytes) of an image layout; needs no GPU."""
    kv = KvLayout(shape.num_layers, shape.num_kv_heads, shape.block_tokens, shape.head_dim, shape.elt_bytes,
                  shape.num_planes, num_blocks, None)
    hl = HostLayout(strides[0], strides[1], strides[2], capacity_bytes)
    run = C.c_int64()
    rc = int(lib().talaria_check_image_layout(C.byref(kv), n_blocks, C.byref(hl), C.byref(run)))
    return rc, run.value


def check_stage_plan(plan: np.ndarray, dirty_bitmap=None):
    """(status, StageStats) of a stage plan of COPY_DTYPE entries; needs no GPU."""
    plan = np.ascontiguousarray(plan, dtype=COPY_DTYPE)
    bm = None if dirty_bitmap is None else np.ascontiguousarray(dirty_bitmap, dtype=np.uint8)
    st = StageStats()
    rc = int(lib().talaria_check_stage_plan(_ptr(plan), plan.size, _ptr(bm), C.byref(st)))
    return rc, st


class Registry:
    """Host-side page registry: chained block hash -> page offset (needs no GPU)."""

    def __init__(self, expected_pages: int = 1024):
        self._h = C.c_void_p()
        rc = lib().talaria_registry_create(C.byref(self._h), expected_pages)
        if rc != OK:
            raise TalariaError(rc, "talaria_registry_create")

    def insert(self, hashes, page_offsets) -> int:
        h = np.ascontiguousarray(hashes, dtype=np.uint64)
        po = _i64(page_offsets)
        assert h.size == po.size
        n_new = C.c_int64()
        rc = lib().talaria_registry_insert(self._h, _ptr(h), _ptr(po), h.size, C.byref(n_new))
        if rc != OK:
            raise TalariaError(rc, "talaria_registry_insert")
        return n_new.value

    def lookup_prefix(self, hashes):
        h = np.ascontiguousarray(hashes, dtype=np.uint64)
        out = np.zeros(max(h.size, 1), np.int64)
        k = int(lib().talaria_registry_lookup_prefix(self._h, _ptr(h), h.size, _ptr(out)))
        return k, out[:k]

    def erase(self, hashes) -> int:
        h = np.ascontiguousarray(hashes, dtype=np.uint64)
        n = C.c_int64()
        rc = lib().talaria_registry_erase(self._h, _ptr(h), h.size, C.byref(n))
        if rc != OK:
            raise TalariaError(rc, "talaria_registry_erase")
        return n.value

    def __len__(self):
        return int(lib().talaria_registry_size(self._h))

    def destroy(self):
        if self._h:
            lib().talaria_registry_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Bump:
    """Stable-address layout of one managed HBM region (host arithmetic; needs no GPU).
    models: sequence of (weight_bytes, runtime_bytes, num_layers, num_planes, chunk_bytes)."""

    def __init__(self, region_base: int, region_bytes: int, models, align: int = 256):
        self._h = C.c_void_p()
        self.models = [ModelDesc(*m) for m in models]
        arr = (ModelDesc * len(self.models))(*self.models)
        rc = lib().talaria_bump_create(C.byref(self._h), region_base, region_bytes, align, arr, len(self.models))
        if rc != OK:
            self._h = C.c_void_p()
            raise TalariaError(rc, "talaria_bump_create")

    def _check(self, rc, what):
        if rc != OK:
            raise TalariaError(rc, what)

    def view(self, model: int):
        """(BumpView, list of plane base addresses) of a model: the same every time."""
        v = BumpView()
        d = self.models[model]
        planes = (C.c_void_p * (d.num_layers * d.num_planes))()
        self._check(lib().talaria_bump_view(self._h, model, C.byref(v), planes), "talaria_bump_view")
        return v, [int(p or 0) for p in planes]

    def activate(self, model: int) -> BumpView:
        v = BumpView()
        self._check(lib().talaria_bump_activate(self._h, model, C.byref(v)), "talaria_bump_activate")
        return v

    def alloc_blocks(self, n: int, staged_bitmap=None, dirty_bitmap=None):
        """(ids, number of chunks newly marked dirty); dirty_bitmap is updated in place."""
        ids = np.zeros(max(n, 1), np.int32)
        nd = C.c_int64()
        self._check(lib().talaria_bump_alloc_blocks(self._h, n, _ptr(ids), _ptr(staged_bitmap), _ptr(dirty_bitmap),
                                                    C.byref(nd)), "talaria_bump_alloc_blocks")
        return ids[:n], nd.value

    def free_blocks(self, ids):
        ids = _i32(ids)
        self._check(lib().talaria_bump_free_blocks(self._h, _ptr(ids), ids.size), "talaria_bump_free_blocks")

    def free_count(self) -> int:
        return int(lib().talaria_bump_free_count(self._h))

    def stage_place(self, next_model: int, chunk_bytes: int, host_weights: int = 0):
        """(plan as COPY_DTYPE array, chunks that found a staging slot)."""
        d = self.models[next_model]
        cap = max(1, -(-d.weight_bytes // chunk_bytes))
        plan = np.zeros(cap, COPY_DTYPE)
        n, placed = C.c_int64(), C.c_int64()
        self._check(lib().talaria_bump_stage_place(self._h, next_model, chunk_bytes, host_weights or None, _ptr(plan),
                                                   cap, C.byref(n), C.byref(placed)), "talaria_bump_stage_place")
        return plan[:n.value], placed.value

    def lock_chunk(self, chunk_id: int, locked: bool):
        self._check(lib().talaria_bump_lock_chunk(self._h, chunk_id, 1 if locked else 0), "talaria_bump_lock_chunk")

    def staging_slack(self, next_model: int, chunk_bytes: int) -> int:
        return int(lib().talaria_bump_staging_slack(self._h, next_model, chunk_bytes))

    def destroy(self):
        if self._h:
            lib().talaria_bump_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Talaria:
    """One library context on one CUDA device."""

    def __init__(self, device: int = 0, variant: int = VARIANT_AUTO, bounce_bytes: int = 0,
                 dma_min_bytes: int = 0, validate: bool = True, zc_ctas: int = 0, pack_ctas: int = 0,
                 host_match_bytes: int = 0, reload_ctas: int = 0):
        self._h = C.c_void_p()
        cfg = Config(bounce_bytes, dma_min_bytes, variant, 1 if validate else 0, zc_ctas, pack_ctas,
                     host_match_bytes, reload_ctas, 0)
        rc = lib().talaria_create(C.byref(self._h), device, C.byref(cfg))
        if rc != OK:
            self._h = C.c_void_p()
            raise TalariaError(rc, "talaria_create")

    def _check(self, rc: int, what: str):
        if rc != OK:
            raise TalariaError(rc, what, lib().talaria_last_cuda_error(self._h))

    def destroy(self):
        if self._h:
            lib().talaria_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- pinned memory ------------------------------------------------------
    def host_register(self, arr: np.ndarray):
        self._check(lib().talaria_host_register(self._h, arr.ctypes.data, arr.nbytes), "talaria_host_register")

    def host_unregister(self, arr: np.ndarray):
        self._check(lib().talaria_host_unregister(self._h, arr.ctypes.data), "talaria_host_unregister")

    # -- (1) hashing and matching ------------------------------------------
    def block_hash(self, d_tokens, n_tokens: int, block_tokens: int, seed: int, d_hashes_out, stream=None):
        self._check(lib().talaria_block_hash(self._h, _ptr(d_tokens), n_tokens, block_tokens,
                                             C.c_uint64(seed), _ptr(d_hashes_out), _stream_ptr(stream)),
                    "talaria_block_hash")

    def prefix_match(self, n_pairs: int, d_cont_tokens, cont_offsets, d_sess_tokens, sess_offsets,
                     d_sess_hashes, block_tokens: int, seed: int, d_cont_hashes_out, d_results, stream=None):
        co, so = _i64(cont_offsets), _i64(sess_offsets)
        self._check(lib().talaria_prefix_match(self._h, n_pairs, _ptr(d_cont_tokens), _ptr(co),
                                               _ptr(d_sess_tokens), _ptr(so), _ptr(d_sess_hashes),
                                               block_tokens, C.c_uint64(seed), _ptr(d_cont_hashes_out),
                                               _ptr(d_results), _stream_ptr(stream)), "talaria_prefix_match")

    def prefix_match_host(self, n_pairs: int, h_cont_tokens, cont_offsets, h_sess_tokens, sess_offsets,
                          h_sess_hashes, block_tokens: int, seed: int, h_cont_hashes_out, h_results,
                          stream=None):
        co, so = _i64(cont_offsets), _i64(sess_offsets)
        self._check(lib().talaria_prefix_match_host(self._h, n_pairs, _ptr(h_cont_tokens), _ptr(co),
                                                    _ptr(h_sess_tokens), _ptr(so), _ptr(h_sess_hashes),
                                                    block_tokens, C.c_uint64(seed), _ptr(h_cont_hashes_out),
                                                    _ptr(h_results), _stream_ptr(stream)),
                    "talaria_prefix_match_host")

    def prefix_match_resident(self, pairs, d_tokens, d_hashes, block_tokens: int, seed: int, h_results, stream=None):
        """pairs: sequence of (h_cont_tokens, cont_slot, cont_hash_slot, sess_slot, sess_tokens, sess_hash_slot);
        d_tokens / d_hashes: the caller's device arrays (int32 / 64-bit elements)."""
        arr = (ResidentPair * max(len(pairs), 1))()
        keep = []
        for q, (cont, cont_slot, cont_hash_slot, sess_slot, sess_tokens, sess_hash_slot) in enumerate(pairs):
            c = _i32(cont)
            keep.append(c)
            arr[q] = ResidentPair(_ptr(c), int(c.size), int(cont_slot), int(cont_hash_slot), int(sess_slot),
                                  int(sess_tokens), int(sess_hash_slot))
        self._check(lib().talaria_prefix_match_resident(self._h, len(pairs), C.cast(arr, _P), _ptr(d_tokens),
                                                        int(d_tokens.numel()), _ptr(d_hashes), int(d_hashes.numel()),
                                                        block_tokens, C.c_uint64(seed), _ptr(h_results),
                                                        _stream_ptr(stream)), "talaria_prefix_match_resident")

    @staticmethod
    def prefix_match_static(n_pairs: int, d_cont_tokens, cont_offsets, d_sess_tokens, sess_offsets,
                            d_sess_hashes, block_tokens: int, seed: int, d_cont_hashes_out, d_results,
                            stream=None):
        """Allocation-free form of prefix_match: no context, fixed scratch inside the library,
        at most 8 pairs.  Runs on the current CUDA device."""
        co, so = _i64(cont_offsets), _i64(sess_offsets)
        rc = lib().talaria_prefix_match_static(n_pairs, _ptr(d_cont_tokens), _ptr(co), _ptr(d_sess_tokens),
                                               _ptr(so), _ptr(d_sess_hashes), block_tokens, C.c_uint64(seed),
                                               _ptr(d_cont_hashes_out), _ptr(d_results), _stream_ptr(stream))
        if rc != OK:
            raise TalariaError(rc, "talaria_prefix_match_static")

    @staticmethod
    def prefix_agree(committed_blocks, hashes: np.ndarray) -> int:
        cb = _i64(committed_blocks)
        h = np.ascontiguousarray(hashes, dtype=np.uint64)
        assert h.ndim == 2 and h.shape[0] == cb.size
        return int(lib().talaria_prefix_agree(cb.size, _ptr(cb), _ptr(h), h.shape[1]))

    # -- (2)/(3) block-table copies ----------------------------------------
    def _kv(self, fn, what, kv, table, first, n, image, hl, stream):
        bt = _i32(table)
        self._check(fn(self._h, C.byref(kv), _ptr(bt), first, n, _ptr(image), C.byref(hl), _stream_ptr(stream)), what)

    def kv_offload(self, kv, block_table, first_block, n_blocks, host_dst, hl, stream=None):
        self._kv(lib().talaria_kv_offload, "talaria_kv_offload", kv, block_table, first_block, n_blocks, host_dst, hl, stream)

    def kv_restore(self, kv, new_block_table, first_block, n_blocks, host_src, hl, stream=None):
        self._kv(lib().talaria_kv_restore, "talaria_kv_restore", kv, new_block_table, first_block, n_blocks, host_src, hl, stream)

    def kv_restore_layered(self, kv, new_block_table, first_block, n_blocks, host_src, hl, layer_events, stream=None):
        """layer_events: one torch.cuda.Event (already recorded once, so its handle exists) or raw
        cudaEvent_t address per layer."""
        bt = _i32(new_block_table)
        handles = [e if isinstance(e, int) else e.cuda_event for e in layer_events]
        arr = (C.c_void_p * len(handles))(*handles)
        self._check(lib().talaria_kv_restore_layered(self._h, C.byref(kv), _ptr(bt), first_block, n_blocks,
                                                     _ptr(host_src), C.byref(hl), arr, _stream_ptr(stream)),
                    "talaria_kv_restore_layered")

    def kv_offload_pages(self, kv, block_table, first_block, n_blocks, host_pool, pool_bytes, page_offsets, stream=None):
        bt, po = _i32(block_table), _i64(page_offsets)
        self._check(lib().talaria_kv_offload_pages(self._h, C.byref(kv), _ptr(bt), first_block, n_blocks,
                                                   _ptr(host_pool), pool_bytes, _ptr(po), _stream_ptr(stream)),
                    "talaria_kv_offload_pages")

    def kv_restore_pages(self, kv, new_block_table, first_block, n_blocks, host_pool, pool_bytes, page_offsets, stream=None):
        bt, po = _i32(new_block_table), _i64(page_offsets)
        self._check(lib().talaria_kv_restore_pages(self._h, C.byref(kv), _ptr(bt), first_block, n_blocks,
                                                   _ptr(host_pool), pool_bytes, _ptr(po), _stream_ptr(stream)),
                    "talaria_kv_restore_pages")

    def kv_gather(self, kv, block_table, first_block, n_blocks, d_image, il, stream=None):
        self._kv(lib().talaria_kv_gather, "talaria_kv_gather", kv, block_table, first_block, n_blocks, d_image, il, stream)

    def kv_scatter(self, kv, new_block_table, first_block, n_blocks, d_image, il, stream=None):
        self._kv(lib().talaria_kv_scatter, "talaria_kv_scatter", kv, new_block_table, first_block, n_blocks, d_image, il, stream)

    def _batch(self, fn, what, kv, xfers, stream):
        """xfers: sequence of (block_table, first_block, n_blocks, host_image, HostLayout)."""
        arr = (KvXfer * max(len(xfers), 1))()
        keep = []
        for k, (bt, first, n, img, hl) in enumerate(xfers):
            bt = _i32(bt)
            keep.append(bt)
            arr[k] = KvXfer(_ptr(bt), first, n, _ptr(img), hl)
        self._check(fn(self._h, C.byref(kv), arr, len(xfers), _stream_ptr(stream)), what)

    def kv_offload_batch(self, kv, xfers, stream=None):
        self._batch(lib().talaria_kv_offload_batch, "talaria_kv_offload_batch", kv, xfers, stream)

    def kv_restore_batch(self, kv, xfers, stream=None):
        self._batch(lib().talaria_kv_restore_batch, "talaria_kv_restore_batch", kv, xfers, stream)

    # -- (4) staging --------------------------------------------------------
    def stage(self, plan: np.ndarray, dirty_bitmap: Optional[np.ndarray] = None, stream=None) -> StageStats:
        """plan: numpy structured array of COPY_DTYPE (raw addresses)."""
        plan = np.ascontiguousarray(plan, dtype=COPY_DTYPE)
        bm = None if dirty_bitmap is None else np.ascontiguousarray(dirty_bitmap, dtype=np.uint8)
        st = StageStats()
        self._check(lib().talaria_stage(self._h, _ptr(plan), plan.size, _ptr(bm), C.byref(st),
                                        _stream_ptr(stream)), "talaria_stage")
        return st

    def stage_plan_create(self, plan: np.ndarray):
        """Validate and upload a switch plan once; returns an opaque handle for stage_plan_run."""
        plan = np.ascontiguousarray(plan, dtype=COPY_DTYPE)
        h = C.c_void_p()
        self._check(lib().talaria_stage_plan_create(self._h, _ptr(plan), plan.size, C.byref(h)), "talaria_stage_plan_create")
        return h

    def stage_plan_run(self, prepared, dirty_bitmap: Optional[np.ndarray] = None, stream=None) -> StageStats:
        bm = None if dirty_bitmap is None else np.ascontiguousarray(dirty_bitmap, dtype=np.uint8)
        st = StageStats()
        self._check(lib().talaria_stage_plan_run(self._h, prepared, _ptr(bm), C.byref(st), _stream_ptr(stream)),
                    "talaria_stage_plan_run")
        return st

    def stage_plan_destroy(self, prepared):
        self._check(lib().talaria_stage_plan_destroy(self._h, prepared), "talaria_stage_plan_destroy")

    def prestage(self, plan: np.ndarray, blocked_bitmap, staged_bitmap: np.ndarray, dirty_bitmap: np.ndarray,
                 stream=None) -> StageStats:
        """staged_bitmap / dirty_bitmap: uint8 numpy arrays updated in place."""
        plan = np.ascontiguousarray(plan, dtype=COPY_DTYPE)
        bl = None if blocked_bitmap is None else np.ascontiguousarray(blocked_bitmap, dtype=np.uint8)
        st = StageStats()
        self._check(lib().talaria_prestage(self._h, _ptr(plan), plan.size, _ptr(bl), _ptr(staged_bitmap),
                                           _ptr(dirty_bitmap), C.byref(st), _stream_ptr(stream)), "talaria_prestage")
        return st

    @staticmethod
    def mark_dirty(plan: np.ndarray, alloc_base: int, alloc_bytes: int, staged_bitmap, dirty_bitmap: np.ndarray) -> int:
        plan = np.ascontiguousarray(plan, dtype=COPY_DTYPE)
        return int(lib().talaria_mark_dirty(_ptr(plan), plan.size, alloc_base, alloc_bytes, _ptr(staged_bitmap),
                                            _ptr(dirty_bitmap)))

    # -- completion and counters ---------------------------------------------
    def sync(self, stream=None):
        self._check(lib().talaria_sync(self._h, _stream_ptr(stream)), "talaria_sync")

    def get_counters(self) -> Counters:
        c = Counters()
        self._check(lib().talaria_get_counters(self._h, C.byref(c)), "talaria_get_counters")
        return c

    def set_timing(self, enabled: bool):
        self._check(lib().talaria_set_timing(self._h, 1 if enabled else 0), "talaria_set_timing")

    def get_timing(self) -> Timing:
        """Times of the last timed offload / restore / stage (waits for it to finish)."""
        t = Timing()
        self._check(lib().talaria_get_timing(self._h, C.byref(t)), "talaria_get_timing")
        return t

    def reset_counters(self):
        self._check(lib().talaria_reset_counters(self._h), "talaria_reset_counters")
