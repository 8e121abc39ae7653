"""ctypes wrapper of the C++ oracle (test infrastructure; see ptstore_oracle.cpp for what it follows).

Everything here is argument marshalling: numpy arrays in, numpy arrays out.  The paged cache of the
oracle is a list of per-layer uint8 arrays of shape [2, num_blocks, chunk_bytes] in host memory.
"""
import ctypes as C
import os
import subprocess

import numpy as np

PIN, NO_TOUCH = 1, 2
S_NOSPACE, S_TABLE_FULL, S_BOUNDS, S_STATE = 1, 2, 4, 8

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ptstore_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


_SANITIZE = os.environ.get("PTSTORE_ORACLE_SANITIZE") == "1"   # checker build: AddressSanitizer + UBSan (the process must preload libasan)


def build_oracle(force=False, sanitize=_SANITIZE):
    """Compile the oracle with g++ unless the shared object was already built from exactly this source."""
    import hashlib
    lib = _LIB.replace(".so", "_san.so") if sanitize else _LIB
    flags = ["-O1", "-g", "-fno-omit-frame-pointer", "-fsanitize=address,undefined", "-fno-sanitize-recover=undefined"] if sanitize else ["-O2"]
    want = hashlib.sha256(open(_SRC, "rb").read() + " ".join(flags).encode()).hexdigest()
    stamp = lib + ".srchash"
    if force or not os.path.exists(lib) or not os.path.exists(stamp) or open(stamp).read().strip() != want:
        tmp = lib + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-std=c++17"] + flags + ["-Wall", "-shared", "-fPIC", "-pthread", "-o", tmp, _SRC])
        os.replace(tmp, lib)
        with open(stamp, "w") as f:
            f.write(want)
    return lib


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build_oracle())
        u64, i32, vp = C.c_uint64, C.c_int32, C.c_void_p
        lib.oracle_mix.restype = u64; lib.oracle_mix.argtypes = [u64]
        lib.oracle_root.restype = u64; lib.oracle_root.argtypes = [u64]
        lib.oracle_chain.restype = u64; lib.oracle_chain.argtypes = [u64, u64]
        lib.oracle_content.restype = u64; lib.oracle_content.argtypes = [vp, i32]
        lib.oracle_create.restype = vp
        lib.oracle_create.argtypes = [i32, i32, i32, i32, i32, u64, i32, i32, i32]
        lib.oracle_destroy.argtypes = [vp]
        lib.oracle_set_policy.argtypes = [vp, i32]
        lib.oracle_inflation.restype = u64; lib.oracle_inflation.argtypes = [vp]
        lib.oracle_hash.argtypes = [vp, vp, vp, i32, i32, vp]
        lib.oracle_lookup.argtypes = [vp, vp, vp, i32, i32, C.c_uint32, vp, vp]
        lib.oracle_fetch.argtypes = [vp, vp, vp, i32, i32, vp, u64, u64, C.c_uint32, vp]
        lib.oracle_lookup_fetch_threads.argtypes = [vp, vp, vp, i32, i32, vp, u64, u64, C.c_uint32, vp, i32, vp, vp]
        lib.oracle_insert.argtypes = [vp, vp, vp, i32, i32, vp, u64, u64, C.c_uint32, vp, vp, vp, vp]
        lib.oracle_release.argtypes = [vp, vp, vp, i32, i32]
        lib.oracle_evict.argtypes = [vp, i32, i32, i32, vp, vp]
        lib.oracle_promote.argtypes = [vp, vp, vp, i32, i32, C.c_uint32, i32, vp]
        lib.oracle_status.restype = C.c_uint32; lib.oracle_status.argtypes = [vp]
        lib.oracle_epoch.restype = u64; lib.oracle_epoch.argtypes = [vp]
        lib.oracle_collisions.restype = u64; lib.oracle_collisions.argtypes = [vp]
        lib.oracle_free_count.restype = i32; lib.oracle_free_count.argtypes = [vp, i32]
        lib.oracle_free_list.argtypes = [vp, i32, vp]
        lib.oracle_live_count.restype = i32; lib.oracle_live_count.argtypes = [vp, i32]
        lib.oracle_block_info.argtypes = [vp, i32, vp]
        lib.oracle_block_tags.argtypes = [vp, vp, C.c_int64, vp]
        lib.oracle_pool_ptr.restype = vp; lib.oracle_pool_ptr.argtypes = [vp, i32]
        lib.oracle_block_bytes.restype = u64; lib.oracle_block_bytes.argtypes = [vp]
        lib.oracle_poke.argtypes = [vp, i32, C.c_int64, u64]
        _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def hash_parts():
    """The oracle's hash building blocks as python callables (for known-answer tests)."""
    lib = _load()

    def content(tokens):
        t = _i32(tokens)
        return int(lib.oracle_content(_p(t), len(t)))

    return dict(mix=lambda x: int(lib.oracle_mix(x)), root=lambda s: int(lib.oracle_root(s)),
                chain=lambda p, c: int(lib.oracle_chain(p, c)), content=content)


class Oracle:
    def __init__(self, layers, heads, dim, elem_bytes, block_tokens, salt, hbm_blocks, host_blocks=0,
                 byte_mode=True, policy="lru"):
        self.lib = _load()
        self.layers, self.B = layers, block_tokens
        self.chunk_bytes = block_tokens * heads * dim * elem_bytes
        self.block_bytes = 2 * layers * self.chunk_bytes
        self.hbm_blocks, self.host_blocks = hbm_blocks, host_blocks
        self.byte_mode = byte_mode
        self.h = self.lib.oracle_create(layers, heads, dim, elem_bytes, block_tokens, salt, hbm_blocks,
                                        host_blocks, 1 if byte_mode else 0)
        self.lib.oracle_set_policy(self.h, 1 if policy == "gdsf" else 0)

    def close(self):
        if self.h:
            self.lib.oracle_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- cache helpers -------------------------------------------------------------------------------
    def new_cache(self, num_blocks, fill=0):
        return [np.full((2, num_blocks, self.chunk_bytes), fill, dtype=np.uint8) for _ in range(self.layers)]

    @staticmethod
    def _cache_args(cache):
        if cache is None:
            return None, None, 0, 0, 0
        ptrs = (C.c_void_p * len(cache))(*[a.ctypes.data for a in cache])
        a0 = cache[0]
        return ptrs, C.cast(ptrs, C.c_void_p), a0.strides[0], a0.strides[1], a0.shape[1]

    # -- the path ------------------------------------------------------------------------------------
    def hash(self, tokens, offsets, max_blocks):
        tokens, offsets = _i32(tokens), np.ascontiguousarray(offsets, dtype=np.int64)
        R = len(offsets) - 1
        keys = np.zeros((R, max_blocks), dtype=np.uint64)
        self.lib.oracle_hash(self.h, _p(tokens), _p(offsets), R, max_blocks, _p(keys))
        return keys

    def lookup(self, tokens, offsets, max_blocks, flags=0):
        tokens, offsets = _i32(tokens), np.ascontiguousarray(offsets, dtype=np.int64)
        R = len(offsets) - 1
        matched = np.zeros(R, dtype=np.int32)
        ids = np.zeros((R, max_blocks), dtype=np.int32)
        self.lib.oracle_lookup(self.h, _p(tokens), _p(offsets), R, max_blocks, flags, _p(matched), _p(ids))
        return matched, ids

    def fetch(self, ids, matched, cache, block_tables):
        ids, matched, bt = _i32(ids), _i32(matched), _i32(block_tables)
        R, maxB = ids.shape
        keep, ptrs, kvs, bs, nb = self._cache_args(cache)
        self.lib.oracle_fetch(self.h, _p(ids), _p(matched), R, maxB, ptrs, kvs, bs, nb, _p(bt))

    def lookup_fetch_threads(self, tokens, offsets, max_blocks, cache, block_tables, n_threads):
        """Read-only lookup (no stamp, no pin) + fetch with the requests split over n_threads host threads."""
        tokens, offsets, bt = _i32(tokens), np.ascontiguousarray(offsets, dtype=np.int64), _i32(block_tables)
        R = len(offsets) - 1
        matched = np.zeros(R, dtype=np.int32)
        ids = np.zeros((R, max_blocks), dtype=np.int32)
        keep, ptrs, kvs, bs, nb = self._cache_args(cache)
        self.lib.oracle_lookup_fetch_threads(self.h, _p(tokens), _p(offsets), R, max_blocks, ptrs, kvs, bs, nb, _p(bt),
                                             int(n_threads), _p(matched), _p(ids))
        return matched, ids

    def insert(self, tokens, offsets, max_blocks, cache=None, block_tables=None, tags=None):
        tokens, offsets = _i32(tokens), np.ascontiguousarray(offsets, dtype=np.int64)
        R = len(offsets) - 1
        bt = _i32(block_tables) if block_tables is not None else None
        tg = np.ascontiguousarray(tags, dtype=np.uint64) if tags is not None else None
        ids = np.zeros((R, max_blocks), dtype=np.int32)
        newb = np.zeros(R, dtype=np.int32)
        keep, ptrs, kvs, bs, nb = self._cache_args(cache)
        self.lib.oracle_insert(self.h, _p(tokens), _p(offsets), R, max_blocks, ptrs, kvs, bs, nb, _p(bt), _p(tg),
                               _p(ids), _p(newb))
        return ids, newb

    def release(self, ids, matched):
        ids, matched = _i32(ids), _i32(matched)
        R, maxB = ids.shape
        self.lib.oracle_release(self.h, _p(ids), _p(matched), R, maxB)

    def evict(self, tier, n, literal=True):
        """Returns (n_evicted[2], victims) — see oracle_evict in the C++ source for the layout."""
        ne = np.zeros(2, dtype=np.int32)
        victims = np.full(max(2 * n, 1), -1, dtype=np.int32)
        self.lib.oracle_evict(self.h, tier, n, 0 if literal else 1, _p(ne), _p(victims))
        return ne, victims[: int(ne[0] + ne[1])]

    def promote(self, ids, matched, pinned_list, max_promote):
        """Moves host-tier blocks of the list into HBM; returns (rewritten ids, number moved)."""
        ids, matched = _i32(ids).copy(), _i32(matched)
        R, maxB = ids.shape
        n = np.zeros(1, dtype=np.int32)
        self.lib.oracle_promote(self.h, _p(ids), _p(matched), R, maxB, 1 if pinned_list else 0, int(max_promote), _p(n))
        return ids, int(n[0])

    # -- introspection -------------------------------------------------------------------------------
    def status(self):
        return int(self.lib.oracle_status(self.h))

    def epoch(self):
        return int(self.lib.oracle_epoch(self.h))

    def inflation(self):
        return int(self.lib.oracle_inflation(self.h))

    def collisions(self):
        return int(self.lib.oracle_collisions(self.h))

    def free_count(self, tier):
        return int(self.lib.oracle_free_count(self.h, tier))

    def free_list(self, tier):
        out = np.zeros(self.free_count(tier), dtype=np.int32)
        self.lib.oracle_free_list(self.h, tier, _p(out))
        return out

    def live_count(self, tier):
        return int(self.lib.oracle_live_count(self.h, tier))

    def block_info(self, block_id):
        info = np.zeros(9, dtype=np.uint64)
        self.lib.oracle_block_info(self.h, int(block_id), _p(info))
        return dict(live=bool(info[0]), refcount=int(info[1]), last_use=int(info[2]), depth=int(info[3]),
                    parent=int(np.int64(info[4])), key=int(info[5]), tag=int(info[6]), children=int(info[7]), freq=int(info[8]))

    def block_tags(self, ids):
        ids = _i32(ids).ravel()
        out = np.zeros(len(ids), dtype=np.uint64)
        self.lib.oracle_block_tags(self.h, _p(ids), len(ids), _p(out))
        return out

    def pool(self, tier):
        """Byte view [n_blocks, block_bytes] of a tier's pool (byte mode only)."""
        n = self.hbm_blocks if tier == 0 else self.host_blocks
        ptr = self.lib.oracle_pool_ptr(self.h, tier)
        if not ptr or n == 0:
            return np.zeros((0, self.block_bytes), dtype=np.uint8)
        buf = (C.c_uint8 * (n * self.block_bytes)).from_address(ptr)
        return np.frombuffer(buf, dtype=np.uint8).reshape(n, self.block_bytes)

    def poke(self, block_id, refcount, last_use):
        self.lib.oracle_poke(self.h, int(block_id), int(refcount), int(last_use))
