"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C ABI.

Sizes are small enough for the oracle to finish in seconds but span several copy tiles, several lookup
chunks and ragged tails.  Everything is integer / byte work: the bar is bit-exact.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2607_22648_b200 import workloads as W


def _imports():
    from tests.harness import Pair, dev
    from paper_2607_22648_b200 import binding as G
    return Pair, dev, G


ENGINES = [
    ("vector", lambda G: G.COPY_VECTOR),
    ("vector_u8", lambda G: G.COPY_VECTOR | G.copy_variant(1)),
    ("vector_512", lambda G: G.COPY_VECTOR | G.copy_variant(2)),
    ("bulk_auto", lambda G: G.COPY_BULK),
    ("bulk_8x8k_3cta", lambda G: G.COPY_BULK | G.copy_variant(1)),
    ("bulk_3x32k", lambda G: G.COPY_BULK | G.copy_variant(2)),
    ("bulk_12x16k", lambda G: G.COPY_BULK | G.copy_variant(4)),
    ("bulk_group2", lambda G: G.COPY_BULK | G.copy_variant(5)),
    ("bulk_l2hint", lambda G: G.COPY_BULK | G.copy_variant(6)),
    ("bulk_3x64k", lambda G: G.COPY_BULK | G.copy_variant(7)),
]


@pytest.mark.parametrize("lanes", [0, 4, 8, 16, 32])
def test_hash_matches_oracle(lanes):
    Pair, dev, G = _imports()
    rng = np.random.default_rng(lanes)
    for B, shape in [(16, W.TINY), (1, W.KVShape(1, 1, 8, 1)), (3, W.KVShape(1, 2, 8, 3)), (32, W.KVShape(1, 1, 8, 32))]:
        p = Pair(shape, 16, flags=G.lookup_lanes(lanes), salt=int(rng.integers(0, 1 << 62)), max_requests=64,
                 max_batch_blocks=64 * 80)
        seqs = [rng.integers(-5, 32000, size=int(rng.integers(0, 70 * B)), dtype=np.int32) for _ in range(37)]
        seqs[3] = np.zeros(0, dtype=np.int32)
        seqs[5] = seqs[4][: max(len(seqs[4]) - 1, 0)]            # unaligned start of the next request
        for mb in (1, 7, 70, 80):
            p.hash(seqs, mb)
        p.close()


def tiny_flow(flags, seed=0):
    Pair, dev, G = _imports()
    w = W.tiny()
    sh = w.shape
    B = sh.block_tokens
    rng = np.random.default_rng(seed)
    p = Pair(sh, w.pool_blocks, flags=flags, max_requests=16, max_batch_blocks=16 * 64)
    smb = W.max_blocks_of(w.store_seqs, B)
    for i in range(0, len(w.store_seqs), 16):
        part = w.store_seqs[i:i + 16]
        need = sum(len(s) // B for s in part)
        src = W.random_kv_cache(seed * 100 + i, sh, need + 3)
        bt = W.shuffled_block_tables(rng, part, B, smb, need + 3)
        p.insert(part, smb, src, bt)
    assert p.check_status() == 0
    live = p.check_pools()
    assert live == p.o.live_count(0) > 300
    qmb = W.max_blocks_of(w.queries, B)
    mo, io, _, _ = p.lookup(w.queries, qmb, flags=1)
    assert mo.max() > 0
    nd = int(mo.sum()) + 9
    dst = [np.full((2, nd, sh.chunk_bytes), 0x5A, dtype=np.uint8) for _ in range(sh.layers)]
    qbt = np.full((len(w.queries), qmb), -1, dtype=np.int32)
    perm = rng.permutation(nd).astype(np.int32)
    k = 0
    for r in range(len(w.queries)):
        for j in range(mo[r]):
            qbt[r, j] = perm[k]
            k += 1
    p.fetch(io, mo, dst, qbt)
    p.release(io, mo)
    assert p.check_status() == 0
    p.check_counts()
    return p


@pytest.mark.parametrize("name,mk", ENGINES, ids=[e[0] for e in ENGINES])
def test_tiny_config_insert_lookup_fetch(name, mk):
    Pair, dev, G = _imports()
    p = tiny_flow(mk(G))
    # evict a third, compare victims, look up again
    ne, v = p.evict(0, 700)
    assert ne[0] == 700
    w = W.tiny()
    p.lookup(w.queries, 64)
    p.lookup(w.store_seqs[:16], 32)
    p.check_counts()
    p.close()


def test_insert_dedupe_denial_and_alloc_order():
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 2)
    p = Pair(sh, 5, max_requests=8, max_batch_blocks=64)
    a = np.array([1, 1, 2, 2, 3, 3], dtype=np.int32)
    b = np.array([1, 1, 2, 2, 4, 4, 5, 5], dtype=np.int32)
    c = np.array([9, 9], dtype=np.int32)
    rng = np.random.default_rng(0)
    src = W.random_kv_cache(1, sh, 16)
    bt = W.shuffled_block_tables(rng, [a, b, a, c], 2, 4, 16)
    ids, newb = p.insert([a, b, a, c], 4, src, bt)
    assert ids.tolist() == [[0, 1, 2, -1], [0, 1, 3, 4], [0, 1, 2, -1], [-1, -1, -1, -1]]
    assert newb.tolist() == [3, 2, 0, 0]
    assert p.check_status() == G.S_NOSPACE
    p.check_pools()
    p.check_counts()
    # the denied prefix is not findable, the granted ones are
    mo, io, _, _ = p.lookup([a, b, c], 4)
    assert mo.tolist() == [3, 4, 0]
    p.evict(0, 2)
    p.insert([c, np.array([9, 9, 7, 7, 6, 6], dtype=np.int32)], 4, src, bt[:2])
    p.check_status()
    p.check_pools()
    p.check_counts()
    p.close()


@pytest.mark.parametrize("host,policy,async_demote", [(0, "lru", False), (24, "lru", False), (0, "gdsf", False), (24, "gdsf", False),
                                                      (24, "lru", True)])
def test_random_churn_lockstep(host, policy, async_demote):
    """Random interleaving of lookup(PIN) / fetch / evict / insert / release, compared call by call."""
    Pair, dev, G = _imports()
    sh = W.KVShape(2, 1, 8, 2)
    B = 2
    for seed in range(6):
        rng = np.random.default_rng(100 + seed)
        p = Pair(sh, 40, host_blocks=host, salt=seed, max_requests=8, max_batch_blocks=8 * 12, table_slots=211 if seed % 2 else 401,
                 policy=policy)
        seqs, pinned = [], []
        for step in range(60):
            base = seqs[int(rng.integers(0, len(seqs)))] if seqs and rng.random() < 0.75 else np.zeros(0, dtype=np.int32)
            cut = int(rng.integers(0, len(base) + 1))
            s = np.concatenate([base[:cut], rng.integers(0, 3, size=int(rng.integers(1, 10)), dtype=np.int32)])[:24]
            seqs.append(s)
            batch = [seqs[int(rng.integers(0, len(seqs)))] for _ in range(int(rng.integers(1, 5)))] + [s]
            mb = 12
            op = rng.random()
            mo, io, _, _ = p.lookup(batch, mb, flags=1)
            nd = max(int(mo.sum()), 1) + 2
            dst = [np.full((2, nd, sh.chunk_bytes), 7, dtype=np.uint8) for _ in range(sh.layers)]
            bt = np.full((len(batch), mb), -1, dtype=np.int32)
            perm = rng.permutation(nd)
            k = 0
            for r in range(len(batch)):
                for j in range(mo[r]):
                    bt[r, j] = perm[k]; k += 1
            if host and rng.random() < 0.6:                    # move some of the host-tier hits into HBM first
                io, _n = p.promote(io, mo, True, int(rng.integers(0, 6)))
            tier = int(rng.integers(0, 2)) if host else 0
            n_ev = int(rng.integers(0, 12))
            if async_demote and op < 0.7:                      # demotion copy on the side stream, overlapping the fetch
                p.evict(tier, n_ev, literal=bool(step % 2), asynchronous=True)
            p.fetch(io, mo, dst, bt)
            if not async_demote and op < 0.7:
                p.evict(tier, n_ev, literal=bool(step % 2))
            need = sum(len(x) // B for x in batch)
            src = W.random_kv_cache(seed * 1000 + step, sh, need + 1)
            sbt = W.shuffled_block_tables(rng, batch, B, mb, need + 1)
            p.insert(batch, mb, src, sbt)
            if rng.random() < 0.8:
                p.release(io, mo)
            else:
                pinned.append((io, mo))
            if pinned and rng.random() < 0.3:
                io2, mo2 = pinned.pop()
                p.release(io2, mo2)
            p.check_status()
            if step % 10 == 9:
                p.check_pools()
                p.check_counts()
        p.check_pools()
        s = p.check_counts()
        p.close()


def test_promotion_worked_example_and_unpinned_lists():
    Pair, dev, G = _imports()
    sh = W.KVShape(2, 1, 8, 2)
    p = Pair(sh, 8, host_blocks=6, max_requests=4, max_batch_blocks=16)
    rng = np.random.default_rng(0)
    a = np.array([1, 1, 2, 2, 3, 3, 4, 4], dtype=np.int32)
    b = np.array([1, 1, 5, 5], dtype=np.int32)
    src = W.random_kv_cache(1, sh, 8)
    p.insert([a, b], 4, src, W.shuffled_block_tables(rng, [a, b], 2, 4, 8))
    p.evict(0, 5)
    mo, io, _, _ = p.lookup([a, b], 4, flags=1)
    new_ids, n = p.promote(io, mo, True, 3)
    assert n == 3 and new_ids.tolist() == [[5, 6, 7, 8], [5, 11, -1, -1]]
    p.check_pools()
    p.check_counts()
    dst = [np.zeros((2, 8, sh.chunk_bytes), dtype=np.uint8) for _ in range(sh.layers)]
    p.fetch(new_ids, mo, dst, np.array([[0, 1, 2, 3], [4, 5, -1, -1]], dtype=np.int32))
    mo2, io2, _, _ = p.lookup([b], 4, flags=1)
    moved, n = p.promote(new_ids, mo, True, 10)
    assert n == 1 and moved.tolist() == [[5, 6, 7, 3], [5, 11, -1, -1]]
    p.release(io2, mo2)
    p.release(moved, mo)
    mo3, io3, _, _ = p.lookup([b], 4)
    moved3, n = p.promote(io3, mo3, False, 10)
    assert n == 1 and moved3.tolist() == [[5, 2, -1, -1]]
    same, n = p.promote(moved3, mo3, False, 0)
    assert n == 0
    p.lookup([a, b], 4)
    assert p.check_status() == 0
    p.check_pools()
    s = p.check_counts()
    assert s.blocks_promoted == 5 and s.live_nodes[1] == 0
    with pytest.raises(G.PTStoreError):
        Pair(sh, 8).g.promote(dev(io3), dev(mo3), 0, 1)          # no host tier
    p.close()


def test_gdsf_keeps_frequent_blocks_that_lru_would_evict():
    Pair, dev, G = _imports()
    hot = np.array([1, 1, 2, 2], dtype=np.int32)
    cold = np.array([7, 7, 8, 8], dtype=np.int32)
    out = {}
    for policy in ("lru", "gdsf"):
        p = Pair(W.KVShape(1, 1, 8, 2), 8, max_requests=4, max_batch_blocks=16, policy=policy)
        p.insert([hot], 2)
        for _ in range(5):
            p.lookup([hot, hot[:2]], 2)                      # two requests per call touch the first block
        p.insert([cold], 2)
        ne, v = p.evict(0, 2)
        out[policy] = v.tolist()
        p.insert([cold, cold], 2)
        p.lookup([hot, cold], 2, flags=1)
        p.evict(0, 8)
        p.check_counts()
        p.close()
    assert out["lru"] == [1, 0] and out["gdsf"] == [3, 2]


def test_gdsf_priority_above_calls_times_requests_is_ordered_whole():
    """A block's priority H = L + F reaches 256 after 3 calls of 64 requests: the eviction order has to take the whole
    priority into account, or the hot parent is taken before the cold leaf."""
    Pair, dev, G = _imports()
    p = Pair(W.KVShape(1, 1, 8, 2), 8, max_requests=64, max_batch_blocks=128, policy="gdsf")
    bv = np.array([1, 1, 2, 2], dtype=np.int32)
    b = bv[:2]
    p.insert([bv] * 64, 2)
    mo, io, _, _ = p.lookup([b] * 64, 2, flags=1)
    ne, v = p.evict(0, 1)
    assert v.tolist() == [1]
    p.lookup([b] * 64, 2)
    p.release(io, mo)
    p.insert([np.array([1, 1, 3, 3], dtype=np.int32)], 2)
    s = p.check_counts()
    assert s.gdsf_clock == 64 and p.o.block_info(0)["last_use"] == 257
    ne, v = p.evict(0, 1)
    assert v.tolist() == [2]
    ne, v = p.evict(0, 1)
    assert v.tolist() == [0]
    assert p.check_counts().gdsf_clock == 257
    assert p.check_status() == 0
    p.close()


@pytest.mark.parametrize("host", [0, 4])
def test_gdsf_long_history_of_single_requests_lockstep(host):
    """One request per call (max_requests 1) for 300 steps: priorities outgrow the call count; victims compared in order."""
    from tests.histories import small_request_gdsf_history
    Pair, dev, G = _imports()
    p = Pair(W.KVShape(1, 1, 8, 1), 6, host_blocks=host, max_requests=1, max_batch_blocks=4, policy="gdsf", table_slots=23)
    worst = 0
    for k, (op, arg) in enumerate(small_request_gdsf_history(300)):
        if op == "lookup":
            p.lookup([arg], 4)
        elif op == "insert":
            p.insert([arg], 4)
        else:
            p.evict(0, arg, literal=bool(k % 2))
        worst = max([worst] + [p.o.block_info(i)["last_use"] - p.o.epoch() for i in range(6 + host) if p.o.block_info(i)["live"]])
        if k % 50 == 49:
            p.check_counts()
    assert worst > 0
    p.check_counts()
    p.check_status()
    p.close()


def test_lookup_stress_small_matches_oracle():
    Pair, dev, G = _imports()
    ws = W.lookup_stress(n_roots=1500, n_queries=2048)
    sh = W.KVShape(1, 1, 8, 16)
    for lanes in (4, 8, 16, 32):
        p = Pair(sh, ws.n_nodes, flags=G.lookup_lanes(lanes), max_requests=2048, max_batch_blocks=2048 * 64,
                 table_slots=ws.table_slots, byte_mode=False)
        for i in range(0, len(ws.store_seqs), 2048):
            p.insert(ws.store_seqs[i:i + 2048], 16)
        assert p.check_status() == 0
        mo, io, _, _ = p.lookup(ws.queries, 64)
        assert (mo == ws.hit_depth).all()
        p.lookup(ws.queries, 64, flags=3)
        s = p.check_counts()
        assert s.live_nodes[0] == ws.n_nodes
        assert s.query_blocks == 2 * 2048 * 64
        assert s.blocks_matched == 2 * int(ws.hit_depth.sum())
        p.release(io, mo)
        assert p.check_status() == 0
        p.close()


def test_llama8b_shape_fetch_and_insert_span_many_tiles():
    """2 MiB blocks, 32 KiB chunks: every engine, payload regenerated from tags."""
    Pair, dev, G = _imports()
    sh = W.LLAMA3_8B
    for name, mk in ENGINES:
        st = W.doc_stream(7, sh, n_docs=6, len_range=(100, 400), zipf_s=1.1, vocab=128256, suffix_range=(5, 40))
        rng = np.random.default_rng(3)
        p = Pair(sh, 120, flags=mk(G), max_requests=8, max_batch_blocks=8 * st.max_blocks, byte_mode=False)
        mb = st.max_blocks
        wpb = sh.block_bytes // 4
        g = p.g
        for step in range(3):
            seqs, tags = st.batch(5)
            tm = W.tags_matrix(tags, mb)
            mo, io, mg, ig = p.lookup(seqs, mb, flags=1)
            # fetch on the GPU into a device cache; expected content regenerated from the oracle's tags
            need = sum(len(s) // sh.block_tokens for s in seqs)
            cache = G.PagedKV(sh.layers, need + 2, sh.chunk_bytes)
            for t in cache.tensors:
                t.fill_(0x33)
            bt = W.shuffled_block_tables(rng, seqs, sh.block_tokens, mb, need + 2)
            g.fetch(ig, mg, cache, dev(bt))
            exp_tags = p.o.block_tags(io)
            for r in range(len(seqs)):
                for j in range(mo[r]):
                    want = torch.from_numpy(W.payload_words([exp_tags[r * mb + j]], wpb)).view(torch.uint8).reshape(sh.layers, 2, sh.chunk_bytes)
                    for l in (0, 13, sh.layers - 1):
                        got = cache.tensors[l][:, bt[r, j]].cpu()
                        assert torch.equal(got, want[l]), (name, step, r, j, l)
            untouched = set(range(need + 2)) - {int(bt[r, j]) for r in range(len(seqs)) for j in range(mo[r])}
            for b in list(untouched)[:5]:
                assert bool((cache.tensors[5][:, b] == 0x33).all())
            # now fill the cache with this batch's payload (as if computed) and insert
            for r in range(len(seqs)):
                nb = len(seqs[r]) // sh.block_tokens
                words = W.payload_words(torch.from_numpy(tm[r, :nb].astype(np.int64)).cuda(), wpb, xp=torch)
                blk = words.view(torch.uint8).reshape(nb, sh.layers, 2, sh.chunk_bytes)
                idx = torch.from_numpy(bt[r, :nb].astype(np.int64)).cuda()
                for l in range(sh.layers):
                    cache.tensors[l][:, idx] = blk[:, l].permute(1, 0, 2)
            toks, offs = W.ragged(seqs)
            io2, no2 = p.o.insert(toks, offs, mb, None, None, tm)
            ig2, ng2 = g.insert(dev(toks), dev(offs), mb, cache, dev(bt))
            assert (io2 == ig2.cpu().numpy()).all() and (no2 == ng2.cpu().numpy()).all()
            p.release(io, mo)
            # every live pool block holds the payload of its tag
            pool = g.hbm_pool.view(torch.int32).reshape(g.hbm_blocks, wpb)
            live = [i for i in range(g.hbm_blocks) if p.o.block_info(i)["live"]]
            lt = p.o.block_tags(np.array(live, dtype=np.int32))
            want = W.payload_words(torch.from_numpy(lt.astype(np.int64)).cuda(), wpb, xp=torch)
            assert torch.equal(pool[torch.tensor(live, device="cuda")], want), (name, step)
            if step == 1:
                p.evict(0, 30)
            p.check_status()
        p.check_counts()
        p.close()


def test_edge_cases_and_errors():
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 4)
    p = Pair(sh, 8, max_requests=4, max_batch_blocks=32)
    g = p.g
    # empty batch, empty requests, requests shorter than a block
    z = np.zeros(0, dtype=np.int32)
    p.lookup([z, z], 4)
    p.insert([z, np.array([1, 2, 3], dtype=np.int32)], 4)
    p.hash([z], 4)
    mo, io, mg, ig = p.lookup([], 4)                       # R = 0: accepted, the clock still advances
    assert mg.numel() == 0
    # limits and bad arguments are refused on the host
    with pytest.raises(G.PTStoreError) as e:
        g.lookup(dev(z), dev(np.zeros(6, dtype=np.int64)), 4)
    assert e.value.code == G.E_LIMIT
    with pytest.raises(G.PTStoreError) as e:
        g.lookup(dev(z), dev(np.zeros(3, dtype=np.int64)), 0)
    assert e.value.code == G.E_INVAL
    with pytest.raises(G.PTStoreError):
        g.evict(1, 1)                                    # no host tier
    with pytest.raises(G.PTStoreError) as e:
        g.reserve(4, torch.zeros(5, dtype=torch.int32, device="cuda"))       # more entries than max_requests
    assert e.value.code == G.E_LIMIT
    with pytest.raises(G.PTStoreError) as e:
        g.reserve(-1)
    assert e.value.code == G.E_INVAL
    ne, _ = g.reserve(3)                                 # an empty store has room: nothing to evict, no victim list wanted
    assert ne.tolist() == [0, 0]
    # out-of-range block table entries and ids are skipped and flagged, nothing else is touched
    s = np.arange(16, dtype=np.int32)
    src = W.random_kv_cache(0, sh, 4)
    p.insert([s], 4, src, np.array([[0, 1, 2, 3]], dtype=np.int32))
    mo, io, _, _ = p.lookup([s], 4)
    dst = [np.full((2, 4, sh.chunk_bytes), 9, dtype=np.uint8)]
    bad_bt = np.array([[0, 7, -3, 1]], dtype=np.int32)
    p.fetch(io, mo, dst, bad_bt)
    assert p.check_status() == G.S_BOUNDS
    bad_ids = io.copy(); bad_ids[0, 1] = 1000
    p.fetch(bad_ids, mo, dst, np.array([[0, 1, 2, 3]], dtype=np.int32))
    assert p.check_status() == G.S_BOUNDS
    # releasing what was never pinned is flagged and leaves counts at zero
    p.release(io, mo)
    assert p.check_status() == G.S_STATE
    ne, v = p.evict(0, 100)
    assert ne.tolist() == [4, 0]
    p.check_counts()
    # max_blocks cap
    p.insert([s], 2, src, np.array([[0, 1]], dtype=np.int32))
    mo, io, _, _ = p.lookup([s], 4)
    assert mo.tolist() == [2]
    assert g.launch_count() > 10
    # the non-blocking counters equal the blocking ones
    buf = torch.zeros(__import__("ctypes").sizeof(G.Stats), dtype=torch.uint8).pin_memory()
    g.stats_enqueue(buf)
    torch.cuda.synchronize()
    a, b = G.Stats.from_buffer_copy(buf.numpy().tobytes()), g.stats()
    assert bytes(a) == bytes(b)
    p.close()


@pytest.mark.parametrize("table_slots", [150, 257])
def test_table_under_delete_heavy_churn(table_slots):
    """Many evict / insert rounds on a small table.  Deleted keys leave empty slots that later keys reuse; with 150 slots
    for 128 blocks (and up to 64 claims of an insert on top of 76 live keys) the table runs close to full, keys land 24 and more slots from home, and lookups have to take the
    long way (and clear a home's group mark when the last such key has gone)."""
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 1)
    p = Pair(sh, 128, max_requests=8, max_batch_blocks=8 * 8, table_slots=table_slots)
    rng = np.random.default_rng(0)
    prev = None
    for step in range(120):
        vocab = 50 if step % 3 == 0 else 50000          # few distinct prefixes (shared, re-found) or all new
        batch = [rng.integers(0, vocab, size=8, dtype=np.int32) for _ in range(8)]
        p.evict(0, 52, literal=False)
        p.insert(batch, 8)
        p.lookup(batch, 8)
        if prev is not None:
            p.lookup(prev, 8)                            # partly evicted by now: hits, then misses
        prev = batch
        assert p.check_status() in (0, G.S_NOSPACE)
    s = p.check_counts()
    if table_slots == 150:
        assert s.far_keys > 0 and 24 <= s.max_displacement < table_slots
    p.close()


@pytest.mark.parametrize("pool,slots", [(5, 8), (12, 16), (20, 30), (40, 45), (100, 108)])
def test_tiny_tables_wrap_around(pool, slots):
    """Tables of a few slots, nearly as many blocks as slots: every window and every flagged distance wraps around the end
    of the table, and an insert may claim the very last empty slot.  Batches never present more new blocks than there are
    slots left, so the table cannot overflow and every result must equal the oracle's."""
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 1)
    room = slots - pool
    p = Pair(sh, pool, max_requests=4, max_batch_blocks=4 * room, table_slots=slots)
    rng = np.random.default_rng(pool)
    seqs = []
    for step in range(200):
        batch, left = [], room
        while left > 0 and len(batch) < 4:
            n = int(rng.integers(1, left + 1))
            base = seqs[int(rng.integers(0, len(seqs)))] if seqs and rng.random() < 0.5 else np.zeros(0, dtype=np.int32)
            s = np.concatenate([base[: int(rng.integers(0, len(base) + 1))], rng.integers(0, 9, size=n, dtype=np.int32)])[:n]
            batch.append(s); seqs.append(s); left -= n
        p.evict(0, int(rng.integers(0, room + 2)), literal=bool(step % 2))
        p.insert(batch, room)
        p.lookup((batch + [seqs[int(rng.integers(0, len(seqs)))]])[:4], room)
        assert p.check_status() in (0, G.S_NOSPACE)
        seqs = seqs[-30:]
    p.check_counts()
    p.close()


def test_table_almost_full_keys_far_from_home():
    """1,024 blocks in a table of 1,100 slots, filled to the brim and then churned: runs of occupied slots grow to hundreds
    of slots, so keys land beyond the exact bits and the group bits of their home slot (distance 248 and more: the far
    bit, every slot up to the largest distance ever used is compared).  Every lookup result is compared with the oracle."""
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 1)
    p = Pair(sh, 1024, max_requests=8, max_batch_blocks=8 * 8, table_slots=1100)
    rng = np.random.default_rng(12)
    history = []
    for step in range(15):                                   # 15 x 64 new nodes
        batch = [rng.integers(0, 1 << 30, size=8, dtype=np.int32) for _ in range(8)]
        p.insert(batch, 8)
        history.append(batch)
    for step in range(150):
        batch = [rng.integers(0, 1 << 30, size=8, dtype=np.int32) for _ in range(8)]
        p.evict(0, 30 + step % 40, literal=False)            # room for about half of the 64 new nodes: the rest is denied
        p.insert(batch, 8)
        history.append(batch)
        p.lookup(batch, 8)
        p.lookup(history[int(rng.integers(0, len(history)))], 8)          # an old batch: partly or wholly evicted
        assert p.check_status() in (0, G.S_NOSPACE)
    s = p.check_counts()
    assert s.far_keys > 100 and s.max_displacement >= 248
    p.close()


@pytest.mark.parametrize("name,mk", [ENGINES[0], ENGINES[3], ENGINES[4]], ids=["vector", "bulk", "bulk_8x8k_3cta"])
def test_many_requests_share_one_prefix(name, mk):
    """40 identical prompts: every pool block has 40 destinations (more than the per-unit destination cache holds),
    plus a few prompts that share only the front of the prefix."""
    Pair, dev, G = _imports()
    sh = W.TINY
    B = sh.block_tokens
    rng = np.random.default_rng(9)
    doc = rng.integers(0, 32000, size=20 * B + 5, dtype=np.int32)
    other = np.concatenate([doc[:7 * B], rng.integers(0, 32000, size=6 * B, dtype=np.int32)])
    p = Pair(sh, 64, flags=mk(G), max_requests=64, max_batch_blocks=64 * 24)
    src = W.random_kv_cache(4, sh, 40)
    p.insert([doc, other], 24, src, W.shuffled_block_tables(rng, [doc, other], B, 24, 40))
    batch = [doc] * 40 + [other] * 3 + [doc[: 3 * B + 1]]
    mo, io, _, _ = p.lookup(batch, 24, flags=1)
    assert mo.tolist() == [20] * 40 + [13] * 3 + [3]
    nd = int(mo.sum()) + 7
    dst = [np.full((2, nd, sh.chunk_bytes), 0x11, dtype=np.uint8) for _ in range(sh.layers)]
    bt = np.full((len(batch), 24), -1, dtype=np.int32)
    perm, k = rng.permutation(nd), 0
    for r in range(len(batch)):
        for j in range(mo[r]):
            bt[r, j] = perm[k]
            k += 1
    p.fetch(io, mo, dst, bt)
    s = p.check_counts()
    assert s.blocks_fetched[0] == int(mo.sum()) and s.blocks_fetched_distinct == 26      # 20 + 6 distinct source blocks
    p.release(io, mo)
    assert p.check_status() == 0
    p.close()


def test_degenerate_shapes():
    Pair, dev, G = _imports()
    rng = np.random.default_rng(3)
    # a pool of one block, one block per request
    p = Pair(W.KVShape(1, 1, 8, 1), 1, max_requests=4, max_batch_blocks=4, table_slots=3)
    src = W.random_kv_cache(0, W.KVShape(1, 1, 8, 1), 4)
    p.insert([np.array([5], dtype=np.int32), np.array([6], dtype=np.int32)], 1, src, np.array([[0], [1]], dtype=np.int32))
    assert p.check_status() == G.S_NOSPACE
    mo, io, _, _ = p.lookup([np.array([5, 6], dtype=np.int32), np.array([6], dtype=np.int32)], 1)
    assert mo.tolist() == [1, 0]
    p.evict(0, 1)
    p.insert([np.array([6], dtype=np.int32)], 1, src, np.array([[2]], dtype=np.int32))
    p.check_pools(); p.check_counts(); p.check_status()
    p.close()
    # one very long request: hundreds of chained chunks per warp, max_blocks in the thousands
    sh = W.KVShape(1, 1, 8, 1)
    p = Pair(sh, 6000, max_requests=4, max_batch_blocks=4 * 5000, byte_mode=False)
    long_seq = rng.integers(0, 1000, size=5000, dtype=np.int32)
    p.hash([long_seq, long_seq[:4321]], 5000)
    p.insert([long_seq[:4000]], 5000)
    mo, io, _, _ = p.lookup([long_seq, long_seq[:1234], np.concatenate([long_seq[:77], long_seq[:50]])], 5000, flags=1)
    assert mo.tolist() == [4000, 1234, 77]
    p.release(io, mo)
    ne, v = p.evict(0, 1500)
    assert ne[0] == 1500 and v[0] == 3999 and v[-1] == 2500
    p.lookup([long_seq], 5000)
    p.check_counts(); assert p.check_status() == 0
    p.close()
    # very many short requests
    p = Pair(sh, 30000, max_requests=20000, max_batch_blocks=20000 * 2, byte_mode=False)
    many = [rng.integers(0, 150, size=int(rng.integers(0, 3)), dtype=np.int32) for _ in range(20000)]
    p.insert(many, 2)
    mo, io, _, _ = p.lookup(many[::-1], 2, flags=1)
    assert (mo == np.array([len(x) for x in many[::-1]])).all()
    p.release(io, mo)
    p.evict(0, 12345)
    p.lookup(many, 2)
    p.check_counts(); assert p.check_status() == 0
    p.close()


def test_random_histories_across_all_option_combinations():
    """Tiers x eviction policy x (a)synchronous demotion x copy engine, with promotion, held pins and random evictions:
    every call compared with the oracle, pools compared every 20 steps."""
    import itertools
    Pair, dev, G = _imports()
    sh = W.KVShape(2, 1, 8, 2)
    B = 2
    runs = 0
    for seed, (host, policy, asyn, engine) in itertools.product(range(3), itertools.product((0, 30), ("lru", "gdsf"), (False, True),
                                                                                          ("vector", "bulk"))):
        if asyn and not host:
            continue
        rng = np.random.default_rng(2000 + seed)
        p = Pair(sh, 48, host_blocks=host, salt=seed, flags=G.COPY_VECTOR if engine == "vector" else G.COPY_BULK, max_requests=8,
                 max_batch_blocks=8 * 14, table_slots=509, policy=policy)
        seqs, held = [], []
        for step in range(60):
            base = seqs[int(rng.integers(0, len(seqs)))] if seqs and rng.random() < 0.8 else np.zeros(0, dtype=np.int32)
            cut = int(rng.integers(0, len(base) + 1))
            s = np.concatenate([base[:cut], rng.integers(0, 3, size=int(rng.integers(1, 12)), dtype=np.int32)])[:28]
            seqs.append(s)
            batch = [seqs[int(rng.integers(0, len(seqs)))] for _ in range(int(rng.integers(1, 7)))] + [s]
            mb = 14
            mo, io, _, _ = p.lookup(batch, mb, flags=1)
            if host and rng.random() < 0.6:
                io, _ = p.promote(io, mo, True, int(rng.integers(0, 8)))
            nd = max(int(mo.sum()), 1) + 2
            dst = [np.full((2, nd, sh.chunk_bytes), 7, dtype=np.uint8) for _ in range(sh.layers)]
            bt = np.full((len(batch), mb), -1, dtype=np.int32)
            perm, k = rng.permutation(nd), 0
            for r in range(len(batch)):
                for j in range(mo[r]):
                    bt[r, j] = perm[k]
                    k += 1
            tier = int(rng.integers(0, 2)) if host else 0
            n_ev = int(rng.integers(0, 16))
            do_ev = rng.random() < 0.75
            if asyn and do_ev:
                p.evict(tier, n_ev, literal=False, asynchronous=True)
            p.fetch(io, mo, dst, bt)
            if not asyn and do_ev:
                p.evict(tier, n_ev, literal=bool(step % 2))
            need = sum(len(x) // B for x in batch)
            src = W.random_kv_cache(seed * 1000 + step, sh, need + 1)
            p.insert(batch, mb, src, W.shuffled_block_tables(rng, batch, B, mb, need + 1))
            if rng.random() < 0.8:
                p.release(io, mo)
            else:
                held.append((io, mo))
            if held and rng.random() < 0.4:
                p.release(*held.pop())
            p.check_status()
            if step % 20 == 19:
                p.check_pools()
                p.check_counts()
        p.close()
        runs += 1
    assert runs == 36


def test_maximum_depth_request():
    """max_blocks at its limit of 65,535: one request of 65,535 one-token blocks; the eviction order still puts the
    deepest block first (the depth field of the sort key is 16 bits wide)."""
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 1)
    rng = np.random.default_rng(12)
    seq = rng.integers(0, 50000, size=65535, dtype=np.int32)
    p = Pair(sh, 70000, max_requests=2, max_batch_blocks=2 * 65535, byte_mode=False)
    ids, newb = p.insert([seq], 65535)
    assert newb.tolist() == [65535] and ids[0, -1] == 65534
    mo, io, _, _ = p.lookup([seq, seq[:40000]], 65535, flags=1)
    assert mo.tolist() == [65535, 40000]
    p.release(io, mo)
    ne, v = p.evict(0, 3)
    assert v.tolist() == [65534, 65533, 65532]
    with pytest.raises(G.PTStoreError) as e:
        p.g.lookup(dev(seq), dev(np.array([0, 65535], dtype=np.int64)), 65536)
    assert e.value.code == G.E_INVAL
    p.check_counts()
    assert p.check_status() == 0
    p.close()


def test_maximum_depth_requests_are_looked_up_and_gathered_in_one_launch():
    """Two requests of 65,535 and 40,000 one-token blocks over the same stored prompt: the one-launch lookup + gather with
    block depths up to the 16 bits an owned-list entry has, every block of the shorter request shared with the longer one."""
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 1)
    rng = np.random.default_rng(13)
    seq = rng.integers(0, 50000, size=65535, dtype=np.int32)
    p = Pair(sh, 66000, max_requests=2, max_batch_blocks=2 * 65535)
    tab = np.arange(65535, dtype=np.int32)[None, :]
    p.insert([seq], 65535, W.random_kv_cache(5, sh, 65535), tab)
    nd = 65535 + 40000
    bt = np.full((2, 65535), -1, dtype=np.int32)
    perm = rng.permutation(nd).astype(np.int32)
    bt[0, :] = perm[:65535]
    bt[1, :40000] = perm[65535:]
    dst = [np.full((2, nd, sh.chunk_bytes), 0x11, dtype=np.uint8) for _ in range(sh.layers)]
    before = p.g.launch_count()
    s0 = p.g.stats()
    mo, io = p.lookup_fetch([seq, seq[:40000]], 65535, dst, bt)
    assert p.g.launch_count() - before == 1
    assert mo.tolist() == [65535, 40000]
    s1 = p.g.stats()
    assert s1.blocks_fetched[0] - s0.blocks_fetched[0] == nd and s1.blocks_fetched_distinct - s0.blocks_fetched_distinct == 65535
    assert p.check_status() == 0
    p.close()


@pytest.mark.parametrize("engine", ["bulk", "vector"])
def test_chunk_sizes_that_do_not_divide_into_stages(engine):
    """Chunks of 48 KiB (a 32 KiB piece and a 16 KiB tail), 1600 B and 80 B: byte-exact insert and fetch."""
    Pair, dev, G = _imports()
    rng = np.random.default_rng(21)
    for sh in (W.KVShape(2, 8, 128, 24), W.KVShape(3, 1, 8, 100), W.KVShape(2, 1, 8, 5)):
        B = sh.block_tokens
        p = Pair(sh, 40, flags=G.COPY_VECTOR if engine == "vector" else G.COPY_BULK, max_requests=8, max_batch_blocks=8 * 8)
        base = rng.integers(0, 1000, size=6 * B + 3, dtype=np.int32)
        seqs = [base, np.concatenate([base[:2 * B], rng.integers(0, 1000, size=3 * B, dtype=np.int32)]), base[:4 * B]]
        need = sum(len(s) // B for s in seqs)
        src = W.random_kv_cache(5, sh, need + 2)
        p.insert(seqs, 8, src, W.shuffled_block_tables(rng, seqs, B, 8, need + 2))
        p.check_pools()
        mo, io, _, _ = p.lookup(seqs + [base], 8)
        assert mo.tolist() == [6, 5, 4, 6]
        nd = int(mo.sum()) + 3
        dst = [np.full((2, nd, sh.chunk_bytes), 0x77, dtype=np.uint8) for _ in range(sh.layers)]
        bt = np.full((4, 8), -1, dtype=np.int32)
        perm, k = rng.permutation(nd), 0
        for r in range(4):
            for j in range(mo[r]):
                bt[r, j] = perm[k]
                k += 1
        p.fetch(io, mo, dst, bt)
        assert p.check_status() == 0
        p.close()


# ---- fused entry points ----------------------------------------------------------------------------------------------
def _tables_for(rng, matched_upper, n_req, mb, nd):
    """Block tables with a distinct destination for every (request, block) position that could match."""
    bt = np.full((n_req, mb), -1, dtype=np.int32)
    perm, k = rng.permutation(nd), 0
    for r in range(n_req):
        for j in range(matched_upper[r]):
            bt[r, j] = perm[k]
            k += 1
    return bt


@pytest.mark.parametrize("name,mk", [ENGINES[0], ENGINES[3], ENGINES[4]], ids=["vector", "bulk", "bulk_8x8k_3cta"])
def test_lookup_fetch_equals_lookup_then_fetch(name, mk):
    """The fused call on the tiny config: many requests of one block column (sub-warps of 8 and 16 lanes), few long
    requests (the split path), shared prefixes (several destinations per source block) and misses."""
    Pair, dev, G = _imports()
    w = W.tiny()
    sh, B = w.shape, w.shape.block_tokens
    rng = np.random.default_rng(5)
    p = Pair(sh, w.pool_blocks, flags=mk(G), max_requests=1200, max_batch_blocks=1200 * 8)
    smb = W.max_blocks_of(w.store_seqs, B)
    for i in range(0, len(w.store_seqs), 16):
        part = w.store_seqs[i:i + 16]
        need = sum(len(s) // B for s in part)
        p.insert(part, smb, W.random_kv_cache(i, sh, need + 3), W.shuffled_block_tables(rng, part, B, smb, need + 3))
    batches = [
        (w.queries, W.max_blocks_of(w.queries, B)),                                   # 8 long requests: split path
        ([w.store_seqs[i % 64] for i in range(40)] + w.queries[:3], 32),              # 43 requests, shared prefixes, L = 32
        ([w.store_seqs[i % 64][: 8 * B] for i in range(1100)], 8),                    # 1100 short requests: L = 8
        ([w.store_seqs[i % 64][: 12 * B] for i in range(1030)], 9),                   # capped at 9 blocks, L = 16
    ]
    for seqs, mb in batches:
        upper = [min(len(s) // B, mb) for s in seqs]
        nd = sum(upper) + 5
        bt = _tables_for(rng, upper, len(seqs), mb, nd)
        dst = [np.full((2, nd, sh.chunk_bytes), 0x3C, dtype=np.uint8) for _ in range(sh.layers)]
        mo, io = p.lookup_fetch(seqs, mb, dst, bt, flags=1)
        assert mo.sum() > 0
        if seqs is w.queries:
            first_matched = mo
        p.release(io, mo)
        assert p.check_status() == 0
    s = p.check_counts()
    assert s.blocks_fetched[0] == s.blocks_matched
    # an out-of-range table entry is skipped and flagged exactly as by the separate calls
    seqs, mb = batches[0]
    upper = [min(len(x) // B, mb) for x in seqs]
    nd = sum(upper) + 5
    bt = _tables_for(rng, upper, len(seqs), mb, nd)
    r0 = int(np.argmax(first_matched > 0))
    bt[r0, 0] = nd + 7
    dst = [np.full((2, nd, sh.chunk_bytes), 0x3C, dtype=np.uint8) for _ in range(sh.layers)]
    p.lookup_fetch(seqs, mb, dst, bt)
    assert p.check_status() == G.S_BOUNDS
    p.close()


@pytest.mark.parametrize("policy", ["lru", "gdsf"])
def test_small_batch_of_long_prompts_is_looked_up_and_gathered_in_one_launch(policy):
    """Up to 16 prompts of more than 32 blocks: one cooperative launch in which the copy CTAs follow the lookups' progress.
    Match lengths of zero, inside a chunk of 32, on chunk borders and the whole prompt; prompts that share blocks; chunks
    that split into several pieces and units; pinning; then the same batches one request too wide (two launches)."""
    Pair, dev, G = _imports()
    rng = np.random.default_rng(31)
    for sh, mbs in ((W.KVShape(2, 1, 8, 2), (33, 100, 260)), (W.KVShape(2, 8, 136, 16), (70,))):   # chunks of 32 B and of 34 KiB
        B = sh.block_tokens
        pool = 900
        p = Pair(sh, pool, max_requests=20, max_batch_blocks=20 * 260, policy=policy)
        for mb in mbs:
            base = rng.integers(0, 60000, size=mb * B, dtype=np.int32)
            other = rng.integers(0, 60000, size=mb * B, dtype=np.int32)
            stored = min(mb, 70)
            for doc in (base[: stored * B], other[: (stored // 2) * B]):
                nb = len(doc) // B
                tab = np.full((1, mb), -1, dtype=np.int32); tab[0, :nb] = rng.permutation(nb + 2)[:nb]
                p.insert([doc], mb, W.random_kv_cache(mb, sh, nb + 2), tab)
            fresh = lambda n: rng.integers(60000, 99999, size=max(n, 0) * B, dtype=np.int32)
            cuts = [k for k in (0, 1, 31, 32, 33, 64, stored) if k <= stored]
            batch = [np.concatenate([base[: k * B], fresh(mb - k)])[: mb * B] for k in cuts]
            batch += [base, other, other[: 5 * B], base[: 40 * B + B // 2], fresh(2)]
            for R in (1, 3, len(batch), 16, 17):
                seqs = [batch[i % len(batch)] for i in range(R)]
                upper = [min(len(s) // B, mb) for s in seqs]
                nd = sum(upper) + 3
                bt = _tables_for(rng, upper, R, mb, nd)
                dst = [np.full((2, nd, sh.chunk_bytes), 0x5A, dtype=np.uint8) for _ in range(sh.layers)]
                before = p.g.launch_count()
                mo, io = p.lookup_fetch(seqs, mb, dst, bt, flags=R % 2)
                assert p.g.launch_count() - before == (1 if R <= 16 else 2)
                if R >= len(batch):
                    assert mo[: len(cuts)].tolist() == cuts
                if R % 2:
                    p.release(io, mo)
                assert p.check_status() == 0
            # an out-of-range destination and a negative one: those entries are skipped, the first is flagged, the rest copied
            seqs = [base, other]
            upper = [mb, mb]
            nd = 2 * mb + 1
            bt = _tables_for(rng, upper, 2, mb, nd)
            bt[0, 3] = nd + 9
            bt[1, 0] = -1
            dst = [np.full((2, nd, sh.chunk_bytes), 0x5A, dtype=np.uint8) for _ in range(sh.layers)]
            p.lookup_fetch(seqs, mb, dst, bt)
            assert p.check_status() == G.S_BOUNDS
            # the same where prompts share blocks (read once, written to every prompt that names them): a bad entry of the
            # lowest prompt and one of a prompt that shares with it are skipped, every other destination is written
            seqs = [base, base, base[: 10 * B], other, base]
            upper = [min(len(x) // B, mb) for x in seqs]
            nd = sum(upper) + 1
            bt = _tables_for(rng, upper, len(seqs), mb, nd)
            bt[0, 3] = nd + 9
            bt[1, 5] = -4
            bt[4, 5] = nd
            dst = [np.full((2, nd, sh.chunk_bytes), 0x5A, dtype=np.uint8) for _ in range(sh.layers)]
            before = p.g.stats()
            p.lookup_fetch(seqs, mb, dst, bt)
            assert p.check_status() == G.S_BOUNDS
            after = p.g.stats()
            stored_other = min(mb, 70) // 2
            assert after.blocks_fetched_distinct - before.blocks_fetched_distinct == min(mb, 70) + stored_other   # base's and other's blocks, once each
            assert after.blocks_fetched[0] - before.blocks_fetched[0] == sum(min(u, 70) for u in upper[:3]) + stored_other + min(mb, 70) - 3   # entries copied
        s = p.check_counts()
        assert s.blocks_fetched[0] == s.blocks_matched - 5 * len(mbs)       # all but the five bad table entries per size
        p.close()


def test_one_launch_lookup_gather_gives_up_on_a_wait_that_runs_out():
    """One poll per copy wait: the fused kernel's copiers give up at their first wait, drain and return; S_TIMEOUT is
    raised, matched lengths and ids are still right, and with the limit restored the same call is byte-exact."""
    Pair, dev, G = _imports()
    sh = W.LLAMA3_8B
    B = sh.block_tokens
    rng = np.random.default_rng(4)
    mb = 40
    p = Pair(sh, 48, max_requests=4, max_batch_blocks=4 * mb)
    doc = rng.integers(0, 1000, size=36 * B, dtype=np.int32)
    tab = np.full((1, mb), -1, dtype=np.int32); tab[0, :36] = np.arange(36)
    p.insert([doc], mb, W.random_kv_cache(3, sh, 36), tab)
    toks, offs = W.ragged([doc, doc[: 20 * B]])
    bt = np.full((2, mb), -1, dtype=np.int32); bt[0, :36] = np.arange(36); bt[1, :20] = np.arange(36, 56)
    mo, io = p.o.lookup(toks, offs, mb, 0)
    cache = G.PagedKV(sh.layers, 56, sh.chunk_bytes)
    p.g.set_wait_limit(1)
    before = p.g.launch_count()
    mg, ig = p.g.lookup_fetch(dev(toks), dev(offs), mb, cache, dev(bt), 0)
    assert p.g.launch_count() - before == 1
    assert p.g.status() & G.S_TIMEOUT
    assert (mg.cpu().numpy() == mo).all() and (ig.cpu().numpy() == io).all()
    p.g.set_wait_limit(0)
    dst = [np.zeros((2, 56, sh.chunk_bytes), dtype=np.uint8) for _ in range(sh.layers)]
    p.lookup_fetch([doc, doc[: 20 * B]], mb, dst, bt)
    assert p.check_status() == 0
    p.check_counts()
    p.close()


@pytest.mark.parametrize("host,policy,mb", [(0, "lru", 12), (20, "lru", 12), (20, "gdsf", 12), (0, "lru", 40), (0, "gdsf", 40)])
def test_fused_step_lockstep(host, policy, mb):
    """A serving loop made of the fused calls only: lookup_fetch(PIN) -> reserve -> insert -> release, random batches,
    compared call by call; with a host tier the reserve demotes (synchronously or with the copy on the side stream).
    With 40 blocks per prompt and no host tier the lookup_fetch is the single cooperative launch, between the cooperative
    kernels of reserve and insert, for enough steps that their barrier counters are reused many times."""
    Pair, dev, G = _imports()
    sh = W.KVShape(2, 1, 8, 2)
    B = 2
    for seed in range(4):
        rng = np.random.default_rng(700 + seed)
        p = Pair(sh, 36 if mb == 12 else 150, host_blocks=host, salt=seed, max_requests=8, max_batch_blocks=8 * mb, table_slots=307 if mb == 12 else 1201,
                 policy=policy)
        seqs = []
        for step in range(50 if mb == 12 else 80):
            base = seqs[int(rng.integers(0, len(seqs)))] if seqs and rng.random() < 0.75 else np.zeros(0, dtype=np.int32)
            cut = int(rng.integers(0, len(base) + 1))
            s = np.concatenate([base[:cut], rng.integers(0, 3, size=int(rng.integers(1, 10 if mb == 12 else 50)), dtype=np.int32)])[: 2 * mb]
            seqs.append(s)
            batch = [seqs[int(rng.integers(0, len(seqs)))] for _ in range(int(rng.integers(1, 6)))] + [s]
            upper = [len(x) // B for x in batch]
            nd = sum(upper) + 2
            bt = _tables_for(rng, upper, len(batch), mb, nd)
            dst = W.random_kv_cache(seed * 1000 + step, sh, nd)          # holds the new blocks' K/V; hits overwrite their part
            mo, io = p.lookup_fetch(batch, mb, dst, bt, flags=1)
            asyn = bool(host) and step % 3 == 0
            p.reserve(sum(upper), mo, literal=bool(step % 2), asynchronous=asyn, max_victims=40 if step % 5 else 3,
                      headroom=(0, 0, 5)[step % 3])
            p.insert(batch, mb, dst, bt, after_lookup=bool(step % 4))
            p.release(io, mo)
            p.check_status()
            if step % 10 == 9:
                p.check_pools()
                p.check_counts()
        p.check_pools()
        p.check_counts()
        p.close()


def test_few_long_full_hit_prompts_with_little_slack_lockstep():
    """The latency workload in small: 32 stored documents of 256 blocks, prompts of a whole document plus 4 fresh blocks,
    batches of 1, 4 and 16, a pool with so little slack that room is made all the time (at one point the free blocks are
    exactly what the batch needs).  Every step is lookup_fetch(PIN) -> reserve -> insert_after_lookup -> release, compared
    call by call; the insert and evict kernels run with several CTAs here, between the one-launch lookup + gather."""
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 2)
    B, n_docs, doc_blocks, suf_blocks = 2, 32, 256, 4
    mb = doc_blocks + suf_blocks
    pool = n_docs * doc_blocks + 8 * n_docs * suf_blocks
    rng = np.random.default_rng(77)
    p = Pair(sh, pool, max_requests=16, max_batch_blocks=16 * mb)
    docs = [rng.integers(0, 128256, size=doc_blocks * B, dtype=np.int32) for _ in range(n_docs)]
    for k in range(0, n_docs, 16):
        part = docs[k:k + 16]
        bt = np.arange(len(part) * mb, dtype=np.int32).reshape(len(part), mb)
        p.insert(part, mb, W.random_kv_cache(k, sh, len(part) * mb), bt)
    next_doc = 0
    for b, n_steps in ((1, 70), (4, 40), (16, 30)):
        for step in range(n_steps):
            batch = []
            for _ in range(b):
                batch.append(np.concatenate([docs[next_doc % n_docs], rng.integers(0, 128256, size=suf_blocks * B, dtype=np.int32)]))
                next_doc += 1
            bt = rng.permutation(b * mb).astype(np.int32).reshape(b, mb)
            dst = W.random_kv_cache(1000 * b + step, sh, b * mb)
            mo, io = p.lookup_fetch(batch, mb, dst, bt, flags=1)
            assert (mo == doc_blocks).all()
            p.reserve(b * mb, mo, headroom=64 if b < 16 else 0)
            _, newb = p.insert(batch, mb, dst, bt, after_lookup=bool(step % 2))      # resumed behind the lookup's keys, or hashed anew
            assert (newb == suf_blocks).all()
            p.release(io, mo)
            assert p.check_status() == 0
        p.check_pools()
        p.check_counts()
    assert p.g.resumed_inserts() == 70
    # uneven work for the insert's CTAs (long and one-block prompts by turns, hashed anew): one CTA is through its hash
    # chains long before the other, so the phases only come out right if the grid-wide barriers between them hold
    for step in range(24):
        batch = []
        for i in range(5):
            fresh = rng.integers(0, 128256, size=(suf_blocks if i % 2 == 0 else 1) * B, dtype=np.int32)
            batch.append(np.concatenate([docs[next_doc % n_docs], fresh]) if i % 2 == 0 else fresh)
            next_doc += 1
        bt = rng.permutation(5 * mb).astype(np.int32).reshape(5, mb)
        dst = W.random_kv_cache(5000 + step, sh, 5 * mb)
        mo, io = p.lookup_fetch(batch, mb, dst, bt, flags=1)
        p.reserve(5 * mb, mo, headroom=8)
        p.insert(batch, mb, dst, bt)
        p.release(io, mo)
        assert p.check_status() == 0
    p.check_pools()
    p.check_counts()
    p.close()


def test_insert_after_lookup_resumes_behind_the_lookups_keys():
    """Long prompts (a warp per request, with and without the separate content pass): the insert that follows a lookup of
    the same device tensors reuses its keys; first-miss positions at the start, in the middle of a chunk, on a chunk border
    and past the end are all covered, as is an eviction between the two calls and a fallback when the tensors differ."""
    Pair, dev, G = _imports()
    sh = W.KVShape(1, 1, 8, 1)
    rng = np.random.default_rng(8)
    for mb in (24, 100):                                   # 24: one chunk of 32 lanes per request; 100: the split path
        p = Pair(sh, 600, max_requests=8, max_batch_blocks=8 * mb, byte_mode=False)
        base = rng.integers(0, 50000, size=mb, dtype=np.int32)
        p.insert([base[:70]], mb)                          # stored prefix of 70 (or 24) blocks
        fresh = lambda n: rng.integers(50000, 99999, size=n, dtype=np.int32)
        batch = [np.concatenate([base[:k], fresh(max(mb - k, 0))])[:mb] for k in (0, 5, 32, 64, 70)] + [base, base[:33], fresh(3)]
        mo, io, _, _ = p.lookup(batch, mb, flags=1)
        assert mo.tolist() == [min(k, mb, 70) for k in (0, 5, 32, 64, 70)] + [min(mb, 70), min(33, mb), 0]
        p.evict(0, 3)                                      # keys stay valid across changes to the store
        before = p.g.resumed_inserts()
        p.insert(batch, mb, after_lookup=True)
        assert p.g.resumed_inserts() == before + 1
        p.release(io, mo)
        p.lookup(batch, mb)
        # other tensors than the lookup saw, or a call in between that used the key scratch: a plain insert
        other = [fresh(mb) for _ in range(3)]
        p.lookup(batch[:3], mb)
        p.insert(other, mb, after_lookup=False)
        p.insert(batch[:3], mb, after_lookup=True)
        assert p.g.resumed_inserts() == before + 1
        p.check_counts()
        assert p.check_status() in (0, G.S_NOSPACE)
        p.close()


def test_fetch_of_a_block_in_flight_is_skipped_and_flagged():
    """After an asynchronous demotion and before the join, a fetch that names a block whose copy may still be running
    must not read it: the entry is skipped and S_INFLIGHT raised; after the join the same fetch is byte-exact."""
    Pair, dev, G = _imports()
    sh = W.KVShape(2, 1, 8, 2)
    p = Pair(sh, 6, host_blocks=6, max_requests=2, max_batch_blocks=8)
    rng = np.random.default_rng(1)
    a = np.array([1, 1, 2, 2, 3, 3, 4, 4], dtype=np.int32)
    src = W.random_kv_cache(1, sh, 4)
    p.insert([a], 4, src, np.array([[0, 1, 2, 3]], dtype=np.int32))
    p.evict(0, 2, asynchronous=True)                     # blocks 3 and 2 move to the host tier, copy on the side stream
    mo, io, mg, ig = p.lookup([a], 4)
    assert io.tolist() == [[0, 1, 7, 6]]
    bt = np.array([[0, 1, 2, 3]], dtype=np.int32)
    cache = p.gpu_cache([np.full((2, 4, sh.chunk_bytes), 0x44, dtype=np.uint8) for _ in range(sh.layers)])
    p.g.fetch(ig, mg, cache, dev(bt))
    assert p.g.status() == G.S_INFLIGHT
    for l in range(sh.layers):
        got = cache.tensors[l].cpu().numpy()
        assert (got[:, 2:] == 0x44).all() and (got[:, 0] == src[l][:, 0]).all() and (got[:, 1] == src[l][:, 1]).all()
    p.g.join()
    dst = [np.full((2, 4, sh.chunk_bytes), 0x44, dtype=np.uint8) for _ in range(sh.layers)]
    p.fetch(io, mo, dst, bt)
    assert p.check_status() == 0
    p.close()


@pytest.mark.parametrize("engine", ["bulk", "bulk_multi"])
def test_bounded_wait_runs_out_and_the_store_stays_usable(engine):
    """With one poll per wait every copy CTA gives up at its first wait: the call returns, S_TIMEOUT is raised, nothing
    hangs; with the limit restored the same copy is byte-exact (the CTAs drained what they had in flight)."""
    Pair, dev, G = _imports()
    sh = W.LLAMA3_8B
    B = sh.block_tokens
    rng = np.random.default_rng(2)
    p = Pair(sh, 48, max_requests=4, max_batch_blocks=4 * 16)
    doc = rng.integers(0, 1000, size=12 * B, dtype=np.int32)
    src = W.random_kv_cache(9, sh, 12)
    tab = np.arange(12, dtype=np.int32)[None, :].repeat(1, 0)
    tab16 = np.full((1, 16), -1, dtype=np.int32); tab16[0, :12] = tab[0]
    if engine == "bulk":                                  # the insert copy uses copy_bulk_kernel
        p.g.set_wait_limit(1)
        toks, offs = W.ragged([doc])
        p.o.insert(toks, offs, 16, src, tab16)
        p.g.insert(dev(toks), dev(offs), 16, p.gpu_cache(src), dev(tab16))
        assert p.g.status() & G.S_TIMEOUT
        p.g.set_wait_limit(0)
        p.evict(0, 12)                                    # both sides drop the (incompletely copied) blocks
        p.insert([doc], 16, src, tab16)
        p.check_pools()
    else:                                                 # the fetch copy uses copy_bulk_multi_kernel
        p.insert([doc], 16, src, tab16)
        mo, io, mg, ig = p.lookup([doc, doc], 16)
        bt = np.full((2, 16), -1, dtype=np.int32); bt[0, :12] = np.arange(12); bt[1, :12] = np.arange(12, 24)
        cache = G.PagedKV(sh.layers, 24, sh.chunk_bytes)
        p.g.set_wait_limit(1)
        p.g.fetch(ig, mg, cache, dev(bt))
        assert p.g.status() & G.S_TIMEOUT
        p.g.set_wait_limit(0)
        dst = [np.zeros((2, 24, sh.chunk_bytes), dtype=np.uint8) for _ in range(sh.layers)]
        p.fetch(io, mo, dst, bt)
    assert p.check_status() == 0
    p.check_counts()
    p.close()


def test_copy_probe_moves_what_it_says():
    """The measurement kernel really copies: a linear 1:1 copy reproduces the source, the mix writes every piece to two or
    three destinations, the paged-like layout is a permutation of the pieces, and nothing else is touched."""
    Pair, dev, G = _imports()
    n, SB = 64 << 20, 32768
    pieces = n // SB
    src = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
    dst = torch.full((3 * n,), 0xAB, dtype=torch.uint8, device="cuda")
    status = G.copy_probe(src, dst, n, G.PROBE_COPY, scatter=False)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(dst[:n], src) and bool((dst[n:] == 0xAB).all())
    dst.fill_(0xAB)
    G.copy_probe(src, dst, n, G.PROBE_MIX, writes_x100=250, scatter=False, status=status)
    torch.cuda.synchronize()
    assert torch.equal(dst[:n], src) and torch.equal(dst[n:2 * n], src)
    third = dst[2 * n:].view(pieces, SB)
    written = (third != 0xAB).any(dim=1)
    assert 0.4 < float(written.float().mean()) < 0.6
    assert torch.equal(third[written], src.view(pieces, SB)[written])
    dst.fill_(0xAB)
    G.copy_probe(src, dst, n, G.PROBE_COPY, scatter=True, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(torch.sort(dst[:n].view(pieces, SB).long().sum(dim=1)).values, torch.sort(src.view(pieces, SB).long().sum(dim=1)).values)
    before = dst.clone()
    G.copy_probe(src, dst, n, G.PROBE_READ, status=status)
    torch.cuda.synchronize()
    assert torch.equal(dst, before) and int(status.item()) == 0
    with pytest.raises(G.PTStoreError):
        G.copy_probe(src, dst, n + 16, G.PROBE_COPY)


def test_plain_c_client_runs_the_path_through_the_c_abi():
    """tests/abi_client.c: insert, fused lookup + gather, reserve, insert, release from a C program that links the library
    directly; it checks ids, matched lengths, counters and every fetched byte itself."""
    import subprocess
    import tempfile
    from tests.test_abi_cpu import build_c_client
    with tempfile.TemporaryDirectory() as d:
        exe = build_c_client(d)
        r = subprocess.run([exe], capture_output=True, text=True, timeout=120)
        assert r.returncode == 0, r.stdout + r.stderr
        assert r.stdout.startswith("abi client ok")
