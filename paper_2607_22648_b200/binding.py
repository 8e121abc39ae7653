"""ctypes binding of libptstore.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the library's kernels.
Importing this module loads the library and raises if it has not been built (there is no fallback).
"""
import ctypes as C
import os

import torch

from . import build as _build

OK, E_INVAL, E_CUDA, E_NOMEM, E_LIMIT = 0, -1, -2, -3, -4
S_NOSPACE, S_TABLE_FULL, S_BOUNDS, S_STATE, S_TIMEOUT, S_INFLIGHT = 1, 2, 4, 8, 16, 32
PIN, NO_TOUCH = 1, 2
PINNED_LIST = 1
ASYNC_COPY = 1
COPY_BULK, COPY_VECTOR = 0, 1
EVICT_GDSF = 2
TIER_HBM, TIER_HOST = 0, 1


def lookup_lanes(n):
    return (n & 0xFF) << 8


def copy_variant(v):
    return (v & 0xF) << 16


def copy_ctas_per_sm(c):
    return (c & 0xFF) << 20


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("flags", C.c_uint32),
                ("num_layers", C.c_uint32), ("num_kv_heads", C.c_uint32), ("head_dim", C.c_uint32),
                ("elem_bytes", C.c_uint32), ("block_tokens", C.c_uint32), ("max_requests", C.c_uint32),
                ("max_batch_blocks", C.c_uint64), ("salt", C.c_uint64),
                ("hbm_pool", C.c_void_p), ("host_pool", C.c_void_p),
                ("hbm_blocks", C.c_uint32), ("host_blocks", C.c_uint32),
                ("table_slots", C.c_uint64), ("workspace", C.c_void_p), ("workspace_bytes", C.c_uint64),
                ("device", C.c_int32), ("reserved", C.c_int32)]


class PagedCache(C.Structure):
    _fields_ = [("layer_base", C.c_void_p), ("kv_stride_bytes", C.c_uint64), ("block_stride_bytes", C.c_uint64),
                ("num_blocks", C.c_uint32), ("reserved", C.c_uint32)]


class Stats(C.Structure):
    _fields_ = [("epoch", C.c_uint64), ("live_nodes", C.c_uint64 * 2), ("free_blocks", C.c_uint64 * 2),
                ("max_displacement", C.c_uint64), ("query_blocks", C.c_uint64), ("probes_issued", C.c_uint64),
                ("slots_visited", C.c_uint64), ("blocks_matched", C.c_uint64), ("blocks_fetched", C.c_uint64 * 2),
                ("blocks_inserted", C.c_uint64), ("blocks_denied", C.c_uint64), ("blocks_dropped", C.c_uint64 * 2),
                ("blocks_demoted", C.c_uint64), ("far_keys", C.c_uint64), ("blocks_promoted", C.c_uint64), ("gdsf_clock", C.c_uint64), ("blocks_fetched_distinct", C.c_uint64)]


EXPORTS = ["ptstore_workspace_bytes", "ptstore_create", "ptstore_destroy", "ptstore_hash", "ptstore_lookup",
           "ptstore_fetch", "ptstore_insert", "ptstore_release", "ptstore_evict", "ptstore_status", "ptstore_stats",
           "ptstore_launch_count", "ptstore_last_cuda_error", "ptstore_strerror", "ptstore_fetch_static", "ptstore_promote", "ptstore_evict_async", "ptstore_join", "ptstore_stats_enqueue", "ptstore_lookup_fetch",
           "ptstore_reserve", "ptstore_set_wait_limit", "ptstore_time_next_copy", "ptstore_copy_probe",
           "ptstore_insert_after_lookup", "ptstore_resumed_inserts"]


def _load():
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError("libptstore.so is not built: run paper_2607_22648_b200/build.py (needs nvcc)")
    lib = C.CDLL(path)
    vp, i32, u32, u64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64
    lib.ptstore_workspace_bytes.restype = u64
    lib.ptstore_workspace_bytes.argtypes = [C.POINTER(Config)]
    lib.ptstore_create.argtypes = [C.POINTER(Config), C.POINTER(vp), vp]
    lib.ptstore_destroy.argtypes = [vp]
    lib.ptstore_hash.argtypes = [vp, vp, vp, i32, i32, vp, vp]
    lib.ptstore_lookup.argtypes = [vp, vp, vp, i32, i32, u32, vp, vp, vp]
    lib.ptstore_fetch.argtypes = [vp, vp, vp, i32, i32, C.POINTER(PagedCache), vp, vp]
    lib.ptstore_lookup_fetch.argtypes = [vp, vp, vp, i32, i32, u32, C.POINTER(PagedCache), vp, vp, vp, vp]
    lib.ptstore_reserve.argtypes = [vp, C.c_int64, i32, vp, i32, u32, vp, vp, i32, vp]
    lib.ptstore_set_wait_limit.argtypes = [vp, u32]
    lib.ptstore_time_next_copy.argtypes = [vp, vp, vp]
    lib.ptstore_copy_probe.argtypes = [vp, vp, u64, i32, u32, i32, u32, i32, i32, vp, vp]
    lib.ptstore_insert.argtypes = [vp, vp, vp, i32, i32, C.POINTER(PagedCache), vp, vp, vp, vp]
    lib.ptstore_insert_after_lookup.argtypes = [vp, vp, vp, i32, i32, C.POINTER(PagedCache), vp, vp, vp, vp]
    lib.ptstore_resumed_inserts.restype = u64
    lib.ptstore_resumed_inserts.argtypes = [vp]
    lib.ptstore_release.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.ptstore_evict.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.ptstore_evict_async.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.ptstore_join.argtypes = [vp, vp]
    lib.ptstore_promote.argtypes = [vp, vp, vp, i32, i32, u32, i32, vp, vp]
    lib.ptstore_status.argtypes = [vp, vp, C.POINTER(u32)]
    lib.ptstore_stats.argtypes = [vp, vp, C.POINTER(Stats)]
    lib.ptstore_stats_enqueue.argtypes = [vp, vp, vp]
    lib.ptstore_launch_count.restype = u64
    lib.ptstore_launch_count.argtypes = [vp]
    lib.ptstore_last_cuda_error.argtypes = [vp]
    lib.ptstore_fetch_static.argtypes = [vp, u32, u32, u64, vp, vp, i32, i32, C.POINTER(PagedCache), vp, vp, vp]
    lib.ptstore_strerror.restype = C.c_char_p
    lib.ptstore_strerror.argtypes = [C.c_int]
    return lib


lib = _load()


class PTStoreError(RuntimeError):
    def __init__(self, code, what):
        super().__init__("%s: %s (%d)" % (what, lib.ptstore_strerror(code).decode(), code))
        self.code = code


def _ptr(t):
    return t.data_ptr() if t is not None else None


def _stream():
    return torch.cuda.current_stream().cuda_stream


class PagedKV:
    """A vLLM-style paged cache: one uint8 tensor [2, num_blocks, chunk_bytes] per layer, plus the
    device array of layer pointers the library wants."""

    def __init__(self, layers, num_blocks, chunk_bytes, device="cuda", tensors=None):
        self.tensors = tensors if tensors is not None else [
            torch.empty((2, num_blocks, chunk_bytes), dtype=torch.uint8, device=device) for _ in range(layers)]
        self.num_blocks = num_blocks
        self.ptrs = torch.tensor([t.data_ptr() for t in self.tensors], dtype=torch.int64, device=device)
        t0 = self.tensors[0]
        self.desc = PagedCache(self.ptrs.data_ptr(), t0.stride(0) * t0.element_size(), t0.stride(1) * t0.element_size(),
                               num_blocks, 0)


PROBE_READ, PROBE_WRITE, PROBE_COPY, PROBE_MIX = 0, 1, 2, 3


def copy_probe(src, dst, nbytes, mode, writes_x100=100, stages=3, stage_bytes=32768, ctas_per_sm=1, scatter=True, status=None):
    """ptstore_copy_probe: one launch of the bulk copy ring over plain buffers (uint8 device tensors) in one traffic pattern."""
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=src.device)
    rc = lib.ptstore_copy_probe(_ptr(src), _ptr(dst), nbytes, mode, writes_x100, stages, stage_bytes, ctas_per_sm, 1 if scatter else 0,
                                _ptr(status), _stream())
    if rc:
        raise PTStoreError(rc, "ptstore_copy_probe")
    return status


STATIC_MAX_REQUESTS, STATIC_MAX_PAIRS = 1024, 65536


def fetch_static(hbm_pool, hbm_blocks, layers, chunk_bytes, ids, matched, cache, block_tables, status_out=None):
    """ptstore_fetch_static: the gather for callers that may not allocate device memory.  Needs no store
    handle; scratch is a fixed array inside the library (limits STATIC_MAX_REQUESTS / STATIC_MAX_PAIRS).
    Calls that overlap on the GPU race on that array; the first call per device should precede any stream
    capture.  Raises PTStoreError on a refused call."""
    R, mb = ids.shape
    rc = lib.ptstore_fetch_static(_ptr(hbm_pool), hbm_blocks, layers, chunk_bytes, _ptr(ids), _ptr(matched), R, mb,
                                  C.byref(cache.desc), _ptr(block_tables), _ptr(status_out), _stream())
    if rc:
        raise PTStoreError(rc, "ptstore_fetch_static")


class PTStore:
    """One store on one GPU.  Allocates pool and workspace with torch and hands them to the library."""

    def __init__(self, layers, heads, dim, block_tokens, hbm_blocks, max_requests, max_batch_blocks, elem_bytes=2,
                 host_blocks=0, table_slots=None, salt=0, flags=0, device=None, hbm_pool=None, host_pool=None):
        if device is None:
            device = torch.cuda.current_device()       # one process per GPU: the rank's own device
        self.device = torch.device("cuda", device)
        self.layers, self.block_tokens = layers, block_tokens
        self.chunk_bytes = block_tokens * heads * dim * elem_bytes
        self.block_bytes = 2 * layers * self.chunk_bytes
        self.hbm_blocks, self.host_blocks = hbm_blocks, host_blocks
        n = hbm_blocks + host_blocks
        self.table_slots = table_slots or max(int(n / 0.7) + 1, n + 2)
        self.hbm_pool = hbm_pool if hbm_pool is not None else torch.empty(hbm_blocks * self.block_bytes, dtype=torch.uint8,
                                                                         device=self.device)
        self.host_pool = host_pool
        host_ptr = None
        if host_blocks:
            if self.host_pool is None:
                self.host_pool = torch.empty(host_blocks * self.block_bytes, dtype=torch.uint8, pin_memory=True)
            host_ptr = self.host_pool.data_ptr()   # pinned memory shares the unified address space
        cfg = Config(C.sizeof(Config), flags, layers, heads, dim, elem_bytes, block_tokens, max_requests,
                     max_batch_blocks, salt, self.hbm_pool.data_ptr(), host_ptr, hbm_blocks, host_blocks,
                     self.table_slots, None, 0, device, 0)
        need = lib.ptstore_workspace_bytes(C.byref(cfg))
        if need == 0:
            raise PTStoreError(E_INVAL, "ptstore_workspace_bytes")
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        cfg.workspace, cfg.workspace_bytes = base, need
        self.cfg = cfg
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = lib.ptstore_create(C.byref(cfg), C.byref(h), _stream())
        if rc:
            raise PTStoreError(rc, "ptstore_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            torch.cuda.synchronize(self.device)
            lib.ptstore_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, what):
        if rc:
            raise PTStoreError(rc, what)

    # every method takes device tensors (int32 tokens/ids/tables, int64 offsets) and returns device tensors
    def hash(self, tokens, offsets, max_blocks):
        R = offsets.numel() - 1
        keys = torch.empty((R, max_blocks), dtype=torch.int64, device=self.device)
        self._check(lib.ptstore_hash(self.h, _ptr(tokens), _ptr(offsets), R, max_blocks, _ptr(keys), _stream()), "ptstore_hash")
        return keys

    def lookup(self, tokens, offsets, max_blocks, flags=0, matched=None, ids=None):
        R = offsets.numel() - 1
        if matched is None:
            matched = torch.empty(R, dtype=torch.int32, device=self.device)
        if ids is None:
            ids = torch.empty((R, max_blocks), dtype=torch.int32, device=self.device)
        self._check(lib.ptstore_lookup(self.h, _ptr(tokens), _ptr(offsets), R, max_blocks, flags, _ptr(matched), _ptr(ids),
                                       _stream()), "ptstore_lookup")
        return matched, ids

    def fetch(self, ids, matched, cache, block_tables):
        R, mb = ids.shape
        self._check(lib.ptstore_fetch(self.h, _ptr(ids), _ptr(matched), R, mb, C.byref(cache.desc), _ptr(block_tables),
                                      _stream()), "ptstore_fetch")

    def lookup_fetch(self, tokens, offsets, max_blocks, cache, block_tables, flags=0, matched=None, ids=None):
        R = offsets.numel() - 1
        if matched is None:
            matched = torch.empty(R, dtype=torch.int32, device=self.device)
        if ids is None:
            ids = torch.empty((R, max_blocks), dtype=torch.int32, device=self.device)
        self._check(lib.ptstore_lookup_fetch(self.h, _ptr(tokens), _ptr(offsets), R, max_blocks, flags, C.byref(cache.desc),
                                             _ptr(block_tables), _ptr(matched), _ptr(ids), _stream()), "ptstore_lookup_fetch")
        return matched, ids

    def reserve(self, want_free, minus=None, flags=0, max_victims=0, n_evicted=None, victims=None, headroom=0):
        """Evicts need + headroom blocks from HBM if need = want_free - sum(minus) - free HBM blocks is positive, decided on
        the device."""
        if n_evicted is None:
            n_evicted = torch.zeros(2, dtype=torch.int32, device=self.device)
        if victims is None and max_victims:
            victims = torch.full((2 * max_victims,), -1, dtype=torch.int32, device=self.device)
        self._check(lib.ptstore_reserve(self.h, int(want_free), int(headroom), _ptr(minus), minus.numel() if minus is not None else 0, flags,
                                        _ptr(n_evicted), _ptr(victims), max_victims, _stream()), "ptstore_reserve")
        return n_evicted, victims

    def time_next_copy(self, before, after):
        """before / after: torch.cuda.Event(enable_timing=True) that have been recorded once (so that they exist)."""
        self._check(lib.ptstore_time_next_copy(self.h, before.cuda_event, after.cuda_event), "ptstore_time_next_copy")

    def set_wait_limit(self, polls):
        self._check(lib.ptstore_set_wait_limit(self.h, polls), "ptstore_set_wait_limit")

    def insert(self, tokens, offsets, max_blocks, cache=None, block_tables=None, ids=None, new_blocks=None, after_lookup=False):
        """after_lookup: ptstore_insert_after_lookup (reuses the keys of the last lookup if it saw these very tensors)."""
        R = offsets.numel() - 1
        if ids is None:
            ids = torch.empty((R, max_blocks), dtype=torch.int32, device=self.device)
        if new_blocks is None:
            new_blocks = torch.empty(R, dtype=torch.int32, device=self.device)
        desc = C.byref(cache.desc) if cache is not None else None
        fn = lib.ptstore_insert_after_lookup if after_lookup else lib.ptstore_insert
        self._check(fn(self.h, _ptr(tokens), _ptr(offsets), R, max_blocks, desc, _ptr(block_tables),
                       _ptr(ids), _ptr(new_blocks), _stream()), "ptstore_insert")
        return ids, new_blocks

    def resumed_inserts(self):
        return int(lib.ptstore_resumed_inserts(self.h))

    def release(self, ids, matched):
        R, mb = ids.shape
        self._check(lib.ptstore_release(self.h, _ptr(ids), _ptr(matched), R, mb, _stream()), "ptstore_release")

    def evict(self, tier, n, want_victims=True, n_evicted=None, victims=None, asynchronous=False):
        if n_evicted is None:
            n_evicted = torch.zeros(2, dtype=torch.int32, device=self.device)
        if victims is None and want_victims:
            victims = torch.full((max(2 * n, 1),), -1, dtype=torch.int32, device=self.device)
        fn = lib.ptstore_evict_async if asynchronous else lib.ptstore_evict
        self._check(fn(self.h, tier, n, _ptr(n_evicted), _ptr(victims), _stream()), "ptstore_evict")
        return n_evicted, victims

    def join(self):
        self._check(lib.ptstore_join(self.h, _stream()), "ptstore_join")

    def promote(self, ids, matched, flags, max_promote, n_promoted=None):
        """Rewrites `ids` in place; returns the device counter of blocks moved."""
        R, mb = ids.shape
        if n_promoted is None:
            n_promoted = torch.zeros(1, dtype=torch.int32, device=self.device)
        self._check(lib.ptstore_promote(self.h, _ptr(ids), _ptr(matched), R, mb, flags, max_promote, _ptr(n_promoted), _stream()),
                    "ptstore_promote")
        return n_promoted

    def status(self):
        out = C.c_uint32(0)
        self._check(lib.ptstore_status(self.h, _stream(), C.byref(out)), "ptstore_status")
        return out.value

    def stats(self):
        out = Stats()
        self._check(lib.ptstore_stats(self.h, _stream(), C.byref(out)), "ptstore_stats")
        return out

    def stats_enqueue(self, pinned_bytes):
        """Writes the counters into `pinned_bytes` (a pinned uint8 host tensor of sizeof(Stats)) without blocking;
        read it with Stats.from_buffer_copy(...) once the stream (or a later event) has completed."""
        self._check(lib.ptstore_stats_enqueue(self.h, pinned_bytes.data_ptr(), _stream()), "ptstore_stats_enqueue")

    def launch_count(self):
        return int(lib.ptstore_launch_count(self.h))
