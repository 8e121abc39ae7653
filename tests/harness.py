"""Lock-step driver for parity tests: runs every call on the CPU oracle and on the CUDA library with
the same seeded inputs and compares every output element by element (all integer / byte work, so the
bar is bit-exact)."""
import numpy as np
import torch

from oracle import Oracle
from paper_2607_22648_b200 import binding as G
from paper_2607_22648_b200 import workloads as W


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


class Pair:
    def __init__(self, shape, hbm_blocks, host_blocks=0, salt=0, flags=0, max_requests=64, max_batch_blocks=4096,
                 table_slots=None, byte_mode=True, policy="lru"):
        self.shape = shape
        if policy == "gdsf":
            flags |= G.EVICT_GDSF
        self.o = Oracle(shape.layers, shape.heads, shape.dim, shape.elem_bytes, shape.block_tokens, salt, hbm_blocks,
                        host_blocks, byte_mode=byte_mode, policy=policy)
        self.g = G.PTStore(shape.layers, shape.heads, shape.dim, shape.block_tokens, hbm_blocks, max_requests,
                           max_batch_blocks, elem_bytes=shape.elem_bytes, host_blocks=host_blocks, salt=salt, flags=flags,
                           table_slots=table_slots)
        self.byte_mode = byte_mode

    def close(self):
        self.g.close()
        self.o.close()

    # -- caches -----------------------------------------------------------------------------------------
    def gpu_cache(self, np_cache):
        tensors = [dev(a) for a in np_cache]
        return G.PagedKV(self.shape.layers, np_cache[0].shape[1], self.shape.chunk_bytes, tensors=tensors)

    # -- calls ------------------------------------------------------------------------------------------
    def hash(self, seqs, max_blocks):
        toks, offs = W.ragged(seqs)
        ko = self.o.hash(toks, offs, max_blocks)
        kg = self.g.hash(dev(toks), dev(offs), max_blocks).cpu().numpy().view(np.uint64)
        assert (ko == kg).all(), "keys differ"
        return ko

    def lookup(self, seqs, max_blocks, flags=0):
        toks, offs = W.ragged(seqs)
        mo, io = self.o.lookup(toks, offs, max_blocks, flags)
        self._last_batch = (dev(toks), dev(offs))
        mg, ig = self.g.lookup(self._last_batch[0], self._last_batch[1], max_blocks, flags)
        assert (mo == mg.cpu().numpy()).all(), "matched lengths differ"
        assert (io == ig.cpu().numpy()).all(), "block ids differ"
        return mo, io, mg, ig

    def lookup_fetch(self, seqs, max_blocks, np_cache, block_tables, flags=0):
        """The fused call against the oracle's lookup followed by its fetch (np_cache is modified by the oracle)."""
        toks, offs = W.ragged(seqs)
        gc = self.gpu_cache(np_cache)
        mo, io = self.o.lookup(toks, offs, max_blocks, flags)
        self.o.fetch(io, mo, np_cache, block_tables)
        self._last_batch = (dev(toks), dev(offs))          # kept: an insert_after_lookup must be handed these very tensors
        mg, ig = self.g.lookup_fetch(self._last_batch[0], self._last_batch[1], max_blocks, gc, dev(block_tables), flags)
        assert (mo == mg.cpu().numpy()).all(), "matched lengths differ"
        assert (io == ig.cpu().numpy()).all(), "block ids differ"
        for l in range(self.shape.layers):
            assert torch.equal(gc.tensors[l].cpu(), torch.from_numpy(np_cache[l])), "fetched bytes differ in layer %d" % l
        return mo, io

    def reserve(self, want_free, minus, literal=True, asynchronous=False, max_victims=None, headroom=0):
        """ptstore_reserve against the oracle's evict of the count the definition gives."""
        n = int(want_free) - int(np.maximum(minus, 0).sum()) - self.o.free_count(0)
        n = n + headroom if n > 0 else 0
        cap = n if max_victims is None else max_victims
        n = min(n, cap)
        ne_o, v_o = self.o.evict(0, n, literal=literal)
        ne_g, v_g = self.g.reserve(want_free, dev(minus.astype(np.int32)), G.ASYNC_COPY if asynchronous else 0, max_victims=max(cap, 1),
                                   headroom=headroom)
        ne_g = ne_g.cpu().numpy()
        assert ne_o.tolist() == ne_g.tolist(), ("evicted counts differ", ne_o, ne_g)
        k = int(ne_o.sum())
        assert v_o.tolist() == v_g.cpu().numpy()[:k].tolist(), "victims differ"
        return ne_o, v_o

    def fetch(self, ids, matched, np_cache, block_tables):
        """np_cache is modified by the oracle; a device copy of its ORIGINAL content by the library; then compared."""
        gc = self.gpu_cache(np_cache)
        self.o.fetch(ids, matched, np_cache, block_tables)
        self.g.fetch(dev(ids), dev(matched), gc, dev(block_tables))
        for l in range(self.shape.layers):
            assert torch.equal(gc.tensors[l].cpu(), torch.from_numpy(np_cache[l])), "fetched bytes differ in layer %d" % l
        return gc

    def insert(self, seqs, max_blocks, np_cache=None, block_tables=None, tags=None, after_lookup=False):
        """after_lookup: ptstore_insert_after_lookup with the device tensors of the preceding lookup / lookup_fetch."""
        toks, offs = W.ragged(seqs)
        io, no = self.o.insert(toks, offs, max_blocks, np_cache, block_tables, tags)
        gc = self.gpu_cache(np_cache) if np_cache is not None else None
        dt, do = self._last_batch if after_lookup else (dev(toks), dev(offs))
        ig, ng = self.g.insert(dt, do, max_blocks, gc, dev(block_tables) if block_tables is not None else None, after_lookup=after_lookup)
        assert (io == ig.cpu().numpy()).all(), "inserted ids differ"
        assert (no == ng.cpu().numpy()).all(), "new block counts differ"
        return io, no

    def promote(self, ids, matched, pinned_list, max_promote):
        new_o, n_o = self.o.promote(ids, matched, pinned_list, max_promote)
        ig = dev(ids)
        n_g = self.g.promote(ig, dev(matched), G.PINNED_LIST if pinned_list else 0, max_promote)
        assert n_o == int(n_g.item()), ("promoted counts differ", n_o, int(n_g.item()))
        assert (new_o == ig.cpu().numpy()).all(), "rewritten ids differ"
        return new_o, n_o

    def release(self, ids, matched):
        self.o.release(ids, matched)
        self.g.release(dev(ids), dev(matched))

    def evict(self, tier, n, literal=True, asynchronous=False):
        ne_o, v_o = self.o.evict(tier, n, literal=literal)
        ne_g, v_g = self.g.evict(tier, n, asynchronous=asynchronous)
        ne_g = ne_g.cpu().numpy()
        assert ne_o.tolist() == ne_g.tolist(), ("evicted counts differ", ne_o, ne_g)
        k = int(ne_o.sum())
        assert v_o.tolist() == v_g.cpu().numpy()[:k].tolist(), "victims differ"
        return ne_o, v_o

    def check_status(self):
        so, sg = self.o.status(), self.g.status()
        assert so == sg, ("status words differ", so, sg)
        return so

    def check_pools(self):
        """Every live block's bytes agree (free blocks may hold stale data on either side)."""
        self.g.join()
        torch.cuda.synchronize()
        pool_g = self.g.hbm_pool.cpu().numpy().reshape(self.g.hbm_blocks, -1)
        pool_o = self.o.pool(0)
        host_g = self.g.host_pool.numpy().reshape(self.g.host_blocks, -1) if self.g.host_blocks else None
        host_o = self.o.pool(1)
        n = 0
        for i in range(self.g.hbm_blocks + self.g.host_blocks):
            if not self.o.block_info(i)["live"]:
                continue
            n += 1
            if i < self.g.hbm_blocks:
                assert (pool_g[i] == pool_o[i]).all(), "pool block %d differs" % i
            else:
                assert (host_g[i - self.g.hbm_blocks] == host_o[i - self.g.hbm_blocks]).all(), "host block %d differs" % i
        return n

    def check_counts(self):
        torch.cuda.synchronize()
        s = self.g.stats()
        for t in (0, 1):
            assert s.live_nodes[t] == self.o.live_count(t), ("live", t, s.live_nodes[t], self.o.live_count(t))
            assert s.free_blocks[t] == self.o.free_count(t), ("free", t)
        assert s.epoch == self.o.epoch()
        assert s.gdsf_clock == self.o.inflation()
        return s
