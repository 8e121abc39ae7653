"""Pins of the CPU oracle against things other than itself (no GPU).

hash     : constants re-derived here from integer square roots, checked through the INVERSE of mix
           (so a wrong shift, constant or operand order fails), known answers from tests/golden.
lookup   : brute-force longest common prefix over the list of stored token sequences.
trie     : one node per distinct block-aligned prefix; parent/child stamps and counts.
copies   : byte-for-byte round trips with canaries.
evict    : literal greedy loop vs sorted closed form; pinned chains survive; free counts.
alloc    : k-th new unique block gets id k.
"""
import os
from math import isqrt

import numpy as np
import pytest

from oracle import Oracle, hash_parts, PIN, NO_TOUCH, S_NOSPACE, S_STATE
from paper_2607_22648_b200 import workloads as W
from tests.histories import small_request_gdsf_history

M64 = (1 << 64) - 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hash_kat.txt")


# ---- independent derivation of the constants and of mix^-1 -----------------------------------------
def frac_sqrt(n):
    return isqrt(n << 128) & M64


K1 = ((isqrt(5 << 128) - (1 << 64)) >> 1) & M64        # floor(2^64 / phi) = 2^64 (sqrt5 - 1)/2
K2 = frac_sqrt(2) | 1
K3 = frac_sqrt(3)
K5 = frac_sqrt(5)


def unxorshift(y, s):
    x = y
    for _ in range(64 // s + 1):
        x = y ^ (x >> s)
    return x


def unmix(y):
    y = unxorshift(y, 32)
    y = (y * pow(K5, -1, 1 << 64)) & M64
    y = unxorshift(y, 29)
    y = (y * pow(K3, -1, 1 << 64)) & M64
    return unxorshift(y, 32)


H = hash_parts()


def golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, *vals = line.split()
        out[name] = [int(v, 16) for v in vals]
    return out


def test_constants_are_odd_where_multiplied():
    assert K3 % 2 == 1 and K5 % 2 == 1 and K1 % 2 == 1


def test_mix_inverts_with_rederived_constants():
    rng = np.random.default_rng(1)
    assert H["mix"](0) == 0
    for x in [1, 2, M64, 1 << 63, 0x0123456789ABCDEF] + [int(v) for v in rng.integers(0, 1 << 63, 200)]:
        assert unmix(H["mix"](x)) == x


def test_root_chain_content_structure():
    rng = np.random.default_rng(2)
    for _ in range(100):
        s, p, c = (int(v) for v in rng.integers(0, 1 << 63, 3))
        assert unmix(H["root"](s)) ^ s == K2
        assert (unmix(H["chain"](p, c)) - c) & M64 == (p * K1) & M64
        t = int(rng.integers(0, 1 << 31))
        assert unmix(H["content"]([t])) ^ K1 == t                               # position 0
        j = int(rng.integers(1, 40))
        blk = [int(v) for v in rng.integers(0, 1 << 31, j + 1)]
        last = (H["content"](blk) - H["content"](blk[:-1])) & M64                  # wrapping sum: last term alone
        assert unmix(last) ^ K1 == blk[-1] | (j << 32)
    # negative token ids use their low 32 bits
    assert unmix(H["content"]([-1])) ^ K1 == 0xFFFFFFFF


def test_reserved_keys_are_remapped():
    # mix(0) = 0, so root(C2) and chain(0,0) would be 0 without the remap to >= 2
    assert H["root"](K2) == 2
    assert H["chain"](0, 0) == 2
    y1 = unmix(1)                                                                  # the preimage of 1
    assert H["chain"](0, y1) == 3 and H["root"](y1 ^ K2) == 3


def test_known_answers():
    g = golden()
    assert H["mix"](1) == g["mix_1"][0]
    assert H["mix"](M64) == g["mix_allones"][0]
    assert H["root"](0) == g["root_salt0"][0]
    assert H["content"](list(range(16))) == g["content_tokens_0_15"][0]
    o = Oracle(1, 1, 8, 2, 16, 0, 4)
    k = o.hash(np.arange(48), [0, 48], 3)
    assert [int(v) for v in k[0]] == g["keys_tokens_0_47_B16_salt0"]
    k = o.hash(np.full(32, 7), [0, 32], 2)
    assert [int(v) for v in k[0]] == g["keys_token7_x32_B16_salt0"]
    o1 = Oracle(1, 1, 8, 2, 16, 1, 4)
    assert int(o1.hash(np.arange(48), [0, 48], 3)[0, 0]) == g["key0_tokens_0_47_B16_salt1"][0]


def test_hash_sensitivity_and_prefix_sharing():
    rng = np.random.default_rng(3)
    o = Oracle(1, 1, 8, 2, 16, 5, 4)
    a = rng.integers(0, 32000, 64).astype(np.int32)
    ka = o.hash(a, [0, 64], 4)[0]
    b = a.copy(); b[40] += 1                       # block 2 changes -> keys 2,3 change, 0,1 stay
    kb = o.hash(b, [0, 64], 4)[0]
    assert (ka[:2] == kb[:2]).all() and ka[2] != kb[2] and ka[3] != kb[3]
    c = a.copy(); c[[16, 17]] = c[[17, 16]]        # swapping two tokens of a block changes its key
    if a[16] != a[17]:
        assert o.hash(c, [0, 64], 4)[0, 1] != ka[1]
    o2 = Oracle(1, 1, 8, 2, 16, 6, 4)              # another salt changes every key
    assert (o2.hash(a, [0, 64], 4)[0] != ka).all()
    # trailing partial block ignored, entries beyond the length are 0
    k = o.hash(a[:50], [0, 50], 4)[0]
    assert (k[:3] == ka[:3]).all() and k[3] == 0
    # ragged batch: each request hashed from its own offset
    toks, offs = W.ragged([a[:20], a, a[:33]])
    kk = o.hash(toks, offs, 4)
    assert kk[0, 0] == ka[0] and kk[0, 1] == 0 and (kk[1] == ka).all() and (kk[2, :2] == ka[:2]).all() and kk[2, 2] == 0


# ---- longest prefix vs brute force -------------------------------------------------------------------
def lcp_tokens(a, b):
    n = min(len(a), len(b))
    neq = np.nonzero(a[:n] != b[:n])[0]
    return int(neq[0]) if len(neq) else n


def brute_matched(query, stored, B, max_blocks):
    best = 0
    for s in stored:
        best = max(best, min(lcp_tokens(query, s), (len(s) // B) * B))
    return min(best // B, len(query) // B, max_blocks)


def insert_all(o, seqs, B, max_blocks=None, cache_blocks=None, seed=0, chunk=7):
    """Insert sequences in small batches with a random paged cache; returns the caches used."""
    rng = np.random.default_rng(seed)
    mb = max_blocks or W.max_blocks_of(seqs, B)
    shape = W.KVShape(o.layers, 1, o.chunk_bytes // (2 * B) if o.chunk_bytes % (2 * B) == 0 else 1, B)
    for i in range(0, len(seqs), chunk):
        part = seqs[i:i + chunk]
        need = sum(len(s) // B for s in part)
        cache = [rng.integers(0, 256, size=(2, max(need, 1), o.chunk_bytes), dtype=np.uint8) for _ in range(o.layers)]
        bt = W.shuffled_block_tables(rng, part, B, mb, max(need, 1))
        toks, offs = W.ragged(part)
        o.insert(toks, offs, mb, cache, bt)
    return mb


@pytest.mark.parametrize("B", [1, 2, 16])
def test_lookup_equals_brute_force_small_random(B):
    rng = np.random.default_rng(10 + B)
    for trial in range(40):
        vocab = int(rng.integers(2, 5))           # tiny vocab -> many accidental shared prefixes
        n = int(rng.integers(1, 9))
        stored = [rng.integers(0, vocab, size=int(rng.integers(0, 6 * B + B)), dtype=np.int32) for _ in range(n)]
        o = Oracle(1, 1, 8, 2, B, trial, 256)
        mb = insert_all(o, stored, B, max_blocks=8, seed=trial)
        qs = [rng.integers(0, vocab, size=int(rng.integers(0, 8 * B)), dtype=np.int32) for _ in range(12)]
        qs += [s.copy() for s in stored[:3]]
        toks, offs = W.ragged(qs)
        m, ids = o.lookup(toks, offs, mb)
        for r, q in enumerate(qs):
            assert m[r] == brute_matched(q, stored, B, mb), (trial, r)
            assert (ids[r, :m[r]] >= 0).all() and (ids[r, m[r]:] == -1).all()
        assert o.collisions() == 0


def test_lookup_equals_brute_force_tiny_config():
    w = W.tiny()
    B = w.shape.block_tokens
    o = Oracle(w.shape.layers, w.shape.heads, w.shape.dim, 2, B, 0, w.pool_blocks)
    insert_all(o, w.store_seqs, B, seed=1, chunk=16)
    toks, offs = W.ragged(w.queries)
    mb = W.max_blocks_of(w.queries, B)
    m, ids = o.lookup(toks, offs, mb)
    want = [brute_matched(q, w.store_seqs, B, mb) for q in w.queries]
    assert list(m) == want
    assert max(want) > 0 and min(want) < max(want)
    # I3: matched*B <= true LCP < (matched+1)*B unless limited by lengths
    for r, q in enumerate(w.queries):
        true = max(lcp_tokens(q, s) for s in w.store_seqs)
        assert m[r] * B <= true
        if m[r] < min(len(q) // B, 512 // B):
            assert (m[r] + 1) * B > true
    # I1: one node per distinct block-aligned prefix
    distinct = set()
    for s in w.store_seqs:
        for j in range(1, len(s) // B + 1):
            distinct.add(s[:j * B].tobytes())
    assert o.live_count(0) == len(distinct)
    assert o.free_count(0) + o.live_count(0) == w.pool_blocks
    # matched ids follow parent links: id j's parent is id j-1, depth j, key = chained key
    keys = o.hash(toks, offs, mb)
    for r in range(len(w.queries)):
        for j in range(m[r]):
            info = o.block_info(ids[r, j])
            assert info["live"] and info["depth"] == j and info["key"] == int(keys[r, j])
            assert info["parent"] == (ids[r, j - 1] if j else -1)


def test_max_blocks_cap_and_empty_requests():
    B = 4
    o = Oracle(1, 1, 8, 2, B, 0, 64)
    s = np.arange(40, dtype=np.int32)
    insert_all(o, [s], B, max_blocks=10)
    toks, offs = W.ragged([s, s[:3], np.zeros(0, dtype=np.int32), s[:17]])
    m, ids = o.lookup(toks, offs, 6)
    assert list(m) == [6, 0, 0, 4]
    m, ids = o.lookup(toks[:0], np.zeros(1, dtype=np.int64), 6)
    assert len(m) == 0


# ---- allocation order, dedupe inside a batch, denial ---------------------------------------------------
def test_allocation_order_closed_form_and_batch_dedupe():
    B = 2
    o = Oracle(1, 1, 8, 2, B, 0, 32)
    a = np.array([1, 1, 2, 2, 3, 3], dtype=np.int32)
    b = np.array([1, 1, 2, 2, 4, 4, 5, 5], dtype=np.int32)
    c = np.array([9, 9], dtype=np.int32)
    toks, offs = W.ragged([a, b, a, c])
    ids, newb = o.insert(toks, offs, 4)
    assert ids.tolist() == [[0, 1, 2, -1], [0, 1, 3, 4], [0, 1, 2, -1], [5, -1, -1, -1]]
    assert newb.tolist() == [3, 2, 0, 1]
    ids2, newb2 = o.insert(*W.ragged([np.array([9, 9, 8, 8], dtype=np.int32)]), 4)
    assert ids2.tolist() == [[5, 6, -1, -1]] and newb2.tolist() == [1]
    assert o.free_list(0).tolist() == list(range(7, 32))


def test_insert_denied_when_pool_runs_dry():
    B = 2
    o = Oracle(1, 1, 8, 2, B, 0, 3)
    a = np.array([1, 1, 2, 2, 3, 3, 4, 4], dtype=np.int32)
    b = np.array([1, 1, 2, 2, 7, 7], dtype=np.int32)
    ids, newb = o.insert(*W.ragged([a, b]), 4)
    assert ids.tolist() == [[0, 1, 2, -1], [0, 1, -1, -1]]
    assert newb.tolist() == [3, 0]
    assert o.status() & S_NOSPACE
    assert o.status() == 0


# ---- byte copies ---------------------------------------------------------------------------------------
def test_insert_fetch_round_trip_bytes_and_canaries():
    w = W.tiny(n_store=12, store_len=128, n_query=6, query_len=192)
    sh = w.shape
    B = sh.block_tokens
    o = Oracle(sh.layers, sh.heads, sh.dim, 2, B, 0, w.pool_blocks)
    rng = np.random.default_rng(5)
    mb = W.max_blocks_of(w.store_seqs, B)
    need = sum(len(s) // B for s in w.store_seqs)
    src = W.random_kv_cache(7, sh, need + 5)
    bt = W.shuffled_block_tables(rng, w.store_seqs, B, mb, need + 5)
    toks, offs = W.ragged(w.store_seqs)
    ids, newb = o.insert(toks, offs, mb, src, bt)
    pool = o.pool(0).reshape(w.pool_blocks, sh.layers, 2, sh.chunk_bytes)
    # a new node's bytes are the bytes of the request that created it (lowest index presenting the prefix)
    seen = set()
    for r in range(len(w.store_seqs)):
        for j in range(len(w.store_seqs[r]) // B):
            i = ids[r, j]
            if i in seen:
                continue
            seen.add(i)
            for l in range(sh.layers):
                for s in range(2):
                    assert (pool[i, l, s] == src[l][s, bt[r, j]]).all()
    assert int(newb.sum()) == len(seen)
    # fetch into a cache filled with a canary: matched chunks equal pool chunks, all others untouched
    qt, qo = W.ragged(w.queries)
    qmb = W.max_blocks_of(w.queries, B)
    m, qids = o.lookup(qt, qo, qmb)
    nd = 80
    dst = o.new_cache(nd, fill=0xA5)
    qbt = W.shuffled_block_tables(rng, w.queries, B, qmb, nd)
    o.fetch(qids, m, dst, qbt)
    written = set()
    for r in range(len(w.queries)):
        for j in range(m[r]):
            written.add(int(qbt[r, j]))
            for l in range(sh.layers):
                for s in range(2):
                    assert (dst[l][s, qbt[r, j]] == pool[qids[r, j], l, s]).all()
    assert len(written) > 0
    for b in range(nd):
        if b not in written:
            for l in range(sh.layers):
                assert (dst[l][:, b] == 0xA5).all()


# ---- refcounts, stamps, eviction -------------------------------------------------------------------------
def random_store(seed, B=2, pool=96, host=0, n_seq=14):
    rng = np.random.default_rng(seed)
    o = Oracle(1, 1, 8, 2, B, seed, pool, host)
    seqs = []
    for i in range(n_seq):
        s = rng.integers(0, 3, size=int(rng.integers(B, 9 * B)), dtype=np.int32)
        if i and rng.random() < 0.7:
            src = seqs[int(rng.integers(0, i))]
            L = int(rng.integers(0, len(src) + 1))
            s = np.concatenate([src[:L], s])[: 10 * B]
        seqs.append(s)
    mb = 10
    for i in range(0, n_seq, 3):                       # several insert calls -> several stamps
        o.insert(*W.ragged(seqs[i:i + 3]), mb, None, None)
        if rng.random() < 0.5:                         # touch something in between
            o.lookup(*W.ragged([seqs[int(rng.integers(0, i + 1))]]), mb)
    return o, seqs, mb, rng


def all_nodes(o):
    total = o.hbm_blocks + o.host_blocks
    return {i: o.block_info(i) for i in range(total) if o.block_info(i)["live"]}


def check_invariants(o):
    nodes = all_nodes(o)
    for i, nd in nodes.items():
        p = nd["parent"]
        if p >= 0:
            assert p in nodes, "I2 parent live"
            assert nodes[p]["refcount"] >= nd["refcount"], "I4"
            assert nodes[p]["last_use"] >= nd["last_use"], "I5"
            assert nodes[p]["depth"] + 1 == nd["depth"]
        else:
            assert nd["depth"] == 0
    for tier in (0, 1):
        n = o.hbm_blocks if tier == 0 else o.host_blocks
        fl = o.free_list(tier).tolist()
        assert len(set(fl)) == len(fl)
        live = [i for i in nodes if (i < o.hbm_blocks) == (tier == 0)]
        assert len(fl) + len(live) == n, "I7"
        assert not set(fl) & set(nodes)
    assert len({nd["key"] for nd in nodes.values()}) == len(nodes)
    return nodes


def test_pin_release_balance_and_stamps():
    o, seqs, mb, rng = random_store(21)
    check_invariants(o)
    toks, offs = W.ragged(seqs[:6] + seqs[:2])         # two requests repeat -> multiplicity 2
    e0 = o.epoch()
    m, ids = o.lookup(toks, offs, mb, PIN)
    assert o.epoch() == e0 + 1
    nodes = check_invariants(o)
    count = {}
    for r in range(len(m)):
        for j in range(m[r]):
            count[int(ids[r, j])] = count.get(int(ids[r, j]), 0) + 1
    for i, nd in nodes.items():
        assert nd["refcount"] == count.get(i, 0)
        if i in count:
            assert nd["last_use"] == e0 + 1
    # NO_TOUCH leaves stamps alone but still advances the clock
    before = {i: nd["last_use"] for i, nd in nodes.items()}
    o.lookup(toks, offs, mb, NO_TOUCH)
    assert o.epoch() == e0 + 2
    assert {i: nd["last_use"] for i, nd in all_nodes(o).items()} == before
    o.release(ids, m)
    assert all(nd["refcount"] == 0 for nd in all_nodes(o).values())
    assert o.status() == 0
    o.release(ids, m)                                  # second release underflows: flagged, counts stay 0
    assert o.status() & S_STATE
    assert all(nd["refcount"] == 0 for nd in all_nodes(o).values())


def clone_state(seed, host, pins):
    """Two identical oracles (same seed, same calls) to compare the two eviction forms."""
    out = []
    for _ in range(2):
        o, seqs, mb, rng = random_store(seed, host=host)
        rp = np.random.default_rng(seed + 1000)
        for _p in range(pins):
            s = seqs[int(rp.integers(0, len(seqs)))]
            cut = int(rp.integers(0, len(s) + 1))
            o.lookup(*W.ragged([s[:cut]]), mb, PIN if rp.random() < 0.6 else 0)
        out.append((o, seqs, mb))
    return out


@pytest.mark.parametrize("host", [0, 40])
def test_evict_literal_equals_sorted_closed_form(host):
    for seed in range(60):
        (a, seqs, mb), (b, _, _) = clone_state(seed, host, pins=3)
        rng = np.random.default_rng(seed + 5)
        for step in range(6):
            tier = int(rng.integers(0, 2)) if host else 0
            n = int(rng.integers(0, 25))
            na, va = a.evict(tier, n, literal=True)
            nb, vb = b.evict(tier, n, literal=False)
            assert na.tolist() == nb.tolist() and va.tolist() == vb.tolist(), (seed, step, tier, n)
            assert a.free_list(0).tolist() == b.free_list(0).tolist()
            assert a.free_list(1).tolist() == b.free_list(1).tolist()
            check_invariants(a)
            # interleave new inserts so HBM children appear under host-tier parents
            s = seqs[int(rng.integers(0, len(seqs)))]
            ext = np.concatenate([s, rng.integers(0, 3, size=4, dtype=np.int32)])[: 10 * 2]
            ia, _ = a.insert(*W.ragged([ext]), mb)
            ib, _ = b.insert(*W.ragged([ext]), mb)
            assert ia.tolist() == ib.tolist()
            a.status(); b.status()


def test_evict_never_takes_pinned_and_frees_what_it_reports():
    o, seqs, mb, rng = random_store(33)
    toks, offs = W.ragged(seqs[:3])
    m, ids = o.lookup(toks, offs, mb, PIN)
    pinned = {int(ids[r, j]) for r in range(len(m)) for j in range(m[r])}
    live0, free0 = o.live_count(0), o.free_count(0)
    ne, victims = o.evict(0, 5)
    assert ne[0] == 5 and not set(victims.tolist()) & pinned
    assert o.free_count(0) == free0 + 5 and o.live_count(0) == live0 - 5
    assert o.free_list(0).tolist()[-5:] == victims.tolist()          # freed ids go to the back, in victim order
    ne, victims = o.evict(0, 10 ** 6)                                  # everything unpinned goes
    assert not set(victims.tolist()) & pinned
    assert set(all_nodes(o)) == pinned
    # victims come leaves-first in (stamp, deeper first, id) order
    o2, seqs2, mb2, _ = random_store(34)
    nodes = all_nodes(o2)
    ne, victims = o2.evict(0, 10 ** 6)
    order = sorted(nodes, key=lambda i: (nodes[i]["last_use"], -nodes[i]["depth"], i))
    assert victims.tolist() == order


def test_demotion_keeps_bytes_ids_and_trie():
    sh = W.KVShape(2, 1, 8, 2)
    B = 2
    o = Oracle(sh.layers, sh.heads, sh.dim, 2, B, 0, 8, 6)
    rng = np.random.default_rng(0)
    a = np.array([1, 1, 2, 2, 3, 3, 4, 4], dtype=np.int32)
    b = np.array([1, 1, 5, 5], dtype=np.int32)
    src = W.random_kv_cache(1, sh, 8)
    bt = W.shuffled_block_tables(rng, [a, b], B, 4, 8)
    ids, _ = o.insert(*W.ragged([a, b]), 4, src, bt)
    assert ids.tolist() == [[0, 1, 2, 3], [0, 4, -1, -1]]
    before = o.pool(0).copy()
    o.lookup(*W.ragged([b]), 4)                                        # b's chain is now the most recent
    ne, victims = o.evict(0, 3)
    assert ne.tolist() == [3, 0] and victims.tolist() == [3, 2, 1]     # a's tail, deepest first
    m, qids = o.lookup(*W.ragged([a]), 4)
    assert m.tolist() == [4] and qids.tolist() == [[0, 10, 9, 8]]       # host ids 8.. handed out front first
    hp = o.pool(1)
    for old, new in zip([3, 2, 1], [8, 9, 10]):
        assert (hp[new - 8] == before[old]).all()
    assert o.free_list(0).tolist() == [5, 6, 7, 3, 2, 1]
    # fetch reads host-tier blocks from the host pool
    dst = o.new_cache(4, fill=1)
    o.fetch(qids, m, dst, np.array([[0, 1, 2, 3]], dtype=np.int32))
    pool_now = {0: o.pool(0), 1: o.pool(1)}
    for j, i in enumerate(qids[0]):
        blk = (pool_now[0][i] if i < 8 else pool_now[1][i - 8]).reshape(sh.layers, 2, sh.chunk_bytes)
        for l in range(sh.layers):
            for s in range(2):
                assert (dst[l][s, j] == blk[l, s]).all()
    # a new block under a host-tier parent lands in HBM; the host parent can then not be dropped
    c = np.array([1, 1, 2, 2, 9, 9], dtype=np.int32)
    ids, _ = o.insert(*W.ragged([c]), 4, src, np.array([[0, 1, 2, -1]], dtype=np.int32))
    assert ids.tolist() == [[0, 10, 5, -1]]
    ne, victims = o.evict(1, 10)
    assert victims.tolist() == [8, 9]                                  # 10 has a live HBM child and must stay
    # room-making: host ring has 5 free; ask to demote 7 -> 2 shortfall dropped from host first
    check_invariants(o)


def test_demote_makes_room_by_dropping_host_first():
    B = 1
    o = Oracle(1, 1, 8, 2, B, 0, 6, 3)
    for i in range(6):
        o.insert(*W.ragged([np.array([10 + i], dtype=np.int32)]), 2)   # six one-block roots, stamps 1..6
    ne, v = o.evict(0, 3)
    assert ne.tolist() == [3, 0] and v.tolist() == [0, 1, 2]           # now host ids 6,7,8 hold them
    ne, v = o.evict(0, 2)                                              # host full: drop 2 oldest host blocks, then demote 2
    assert ne.tolist() == [2, 2] and v.tolist() == [3, 4, 6, 7]
    assert o.free_list(1).tolist() == []
    assert o.free_list(0).tolist() == [0, 1, 2, 3, 4]
    m, ids = o.lookup(*W.ragged([np.array([10 + i], dtype=np.int32) for i in range(6)]), 2)
    assert m.tolist() == [0, 0, 1, 1, 1, 1]
    assert ids[:, 0].tolist() == [-1, -1, 8, 6, 7, 5]
    check_invariants(o)


# ---- promotion of host-tier blocks ----------------------------------------------------------------------------
def test_promotion_front_of_prefix_first_with_budget_and_pins():
    sh = W.KVShape(2, 1, 8, 2)
    B = 2
    o = Oracle(sh.layers, sh.heads, sh.dim, 2, B, 0, 8, 6)
    rng = np.random.default_rng(0)
    a = np.array([1, 1, 2, 2, 3, 3, 4, 4], dtype=np.int32)
    b = np.array([1, 1, 5, 5], dtype=np.int32)
    src = W.random_kv_cache(1, sh, 8)
    bt = W.shuffled_block_tables(rng, [a, b], B, 4, 8)
    o.insert(*W.ragged([a, b]), 4, src, bt)                                 # ids a: 0 1 2 3, b: 0 4
    original = {i: o.pool(0)[i].copy() for i in range(5)}
    ne, v = o.evict(0, 5)                                                   # everything goes to host, deepest first
    assert ne.tolist() == [5, 0] and v.tolist() == [3, 2, 1, 4, 0]          # host ids 8 9 10 11 12 in that order
    m, ids = o.lookup(*W.ragged([a, b]), 4, PIN)
    assert ids.tolist() == [[12, 10, 9, 8], [12, 11, -1, -1]]
    # budget 3: the shared first block, then a's second and third (front of the prefix first); HBM ids from the ring front
    new_ids, n = o.promote(ids, m, True, 3)
    assert n == 3 and new_ids.tolist() == [[5, 6, 7, 8], [5, 11, -1, -1]]
    assert o.free_list(0).tolist() == [3, 2, 1, 4, 0] and o.free_list(1).tolist() == [13, 12, 10, 9]
    for new, old in ((5, 0), (6, 1), (7, 2)):
        assert (o.pool(0)[new] == original[old]).all()                      # bytes travelled with the node
    info = o.block_info(5)
    assert info["refcount"] == 2 and info["depth"] == 0 and o.block_info(6)["parent"] == 5
    check_invariants(o)
    # a second list pinning the same blocks: a block whose count exceeds this list's own pins stays where it is
    m2, ids2 = o.lookup(*W.ragged([b]), 4, PIN)                              # pins 5 and 11 once more
    moved, n = o.promote(new_ids, m, True, 10)                               # list 1 names 11 once, its refcount is 2
    assert n == 1 and moved.tolist() == [[5, 6, 7, 3], [5, 11, -1, -1]]       # only a's last block (8) can move
    o.release(ids2, m2)
    o.release(moved, m)
    assert all(nd["refcount"] == 0 for nd in all_nodes(o).values())
    # unpinned list: moves only blocks nobody pins
    m3, ids3 = o.lookup(*W.ragged([b]), 4)
    moved3, n = o.promote(ids3, m3, False, 10)
    assert n == 1 and moved3.tolist() == [[5, 2, -1, -1]]
    check_invariants(o)
    assert o.live_count(1) == 0 and o.free_count(1) == 6
    # no free HBM block, or no budget: nothing moves
    o.evict(0, 2)
    m4, ids4 = o.lookup(*W.ragged([a]), 4)
    same, n = o.promote(ids4, m4, False, 0)
    assert n == 0 and (same == ids4).all()


def test_promotion_random_histories_keep_invariants_and_lookup_results():
    for seed in range(30):
        o, seqs, mb, rng = random_store(seed + 500, pool=40, host=40)
        o.evict(0, int(rng.integers(5, 40)), literal=False)
        for step in range(6):
            batch = [seqs[int(rng.integers(0, len(seqs)))] for _ in range(3)]
            toks, offs = W.ragged(batch)
            m, ids = o.lookup(toks, offs, mb, PIN)
            hbm_free = o.free_count(0)
            host_named = len({int(i) for r in range(len(m)) for i in ids[r, :m[r]] if i >= o.hbm_blocks})
            budget = int(rng.integers(0, 8))
            new_ids, n = o.promote(ids, m, True, budget)
            assert n <= min(budget, hbm_free, host_named)
            m2, ids2 = o.lookup(toks, offs, mb, NO_TOUCH)                   # same matches, ids as rewritten
            assert (m2 == m).all() and (ids2 == new_ids).all()
            o.release(new_ids, m)
            check_invariants(o)
            o.evict(0, int(rng.integers(0, 6)), literal=bool(step % 2))


# ---- frequency-aware eviction (GDSF with equal block size and cost) ---------------------------------------------
def test_gdsf_keeps_frequent_blocks_that_lru_would_evict():
    hot = np.array([1, 1, 2, 2], dtype=np.int32)           # two blocks, asked for five times early on
    cold = np.array([7, 7, 8, 8], dtype=np.int32)          # two blocks, stored last, never asked for again
    out = {}
    for policy in ("lru", "gdsf"):
        o = Oracle(1, 1, 8, 2, 2, 0, 8, policy=policy)
        o.insert(*W.ragged([hot]), 2)                       # ids 0 1
        for _ in range(5):
            o.lookup(*W.ragged([hot]), 2)
        o.insert(*W.ragged([cold]), 2)                      # ids 2 3, most recent
        ne, v = o.evict(0, 2)
        out[policy] = v.tolist()
        if policy == "gdsf":
            assert o.block_info(0)["freq"] == 6 and o.block_info(0)["last_use"] == 6     # H = L + F with L = 0
            assert o.inflation() == 1                       # the victims had H = 0 + 1
            o.insert(*W.ragged([cold]), 2)                  # re-stored after the eviction: H = L + 1 = 2; ids 4 5 (ring front)
            assert o.block_info(4)["last_use"] == 2 and o.block_info(4)["freq"] == 1
    assert out["lru"] == [1, 0]                             # least recently used: the hot pair goes
    assert out["gdsf"] == [3, 2]                            # least frequently used: the cold pair goes, deeper first


def test_gdsf_priority_grows_past_the_accesses_of_any_one_block():
    """H = L + F with L itself a sum of earlier victims' priorities: a hand-worked history in which a block's priority
    (256) exceeds calls x requests per call (3 x 64 = 192), so no bound built from the access count alone holds it."""
    o = Oracle(1, 1, 8, 2, 2, 0, 8, policy="gdsf")
    bv = np.array([1, 1, 2, 2], dtype=np.int32)             # blocks B (id 0) and V (id 1)
    b = bv[:2]
    o.insert(*W.ragged([bv] * 64), 2)                       # call 1: 64 requests store B and V: F = 64, H = 0 + 64 each
    assert [o.block_info(i)["last_use"] for i in (0, 1)] == [64, 64]
    m, ids = o.lookup(*W.ragged([b] * 64), 2, PIN)          # call 2: B asked for 64 times and pinned: F = 128, H = 128
    assert o.block_info(0)["last_use"] == 128 and o.block_info(0)["refcount"] == 64
    ne, v = o.evict(0, 1)                                   # only V is evictable: L = H(V) = 64
    assert v.tolist() == [1] and o.inflation() == 64
    o.lookup(*W.ragged([b] * 64), 2)                        # call 3: F = 192, H = L + F = 64 + 192
    assert o.epoch() == 3 and o.block_info(0)["freq"] == 192 and o.block_info(0)["last_use"] == 256
    o.release(ids, m)
    bw = np.array([1, 1, 3, 3], dtype=np.int32)
    o.insert(*W.ragged([bw]), 2)                            # W (id 2): F = 1, H = 65; B: F = 193, H = 257
    assert o.block_info(2)["last_use"] == 65 and o.block_info(0)["last_use"] == 257
    ne, v = o.evict(0, 1)
    assert v.tolist() == [2] and o.inflation() == 65        # the leaf with the low priority goes, not the hot parent
    ne, v = o.evict(0, 1)
    assert v.tolist() == [0] and o.inflation() == 257


def test_gdsf_priority_exceeds_the_call_count_in_a_long_single_request_history():
    o = Oracle(1, 1, 8, 2, 1, 0, 6, policy="gdsf")
    worst = 0
    for op, arg in small_request_gdsf_history(300):
        if op == "lookup":
            o.lookup(*W.ragged([arg]), 4)
        elif op == "insert":
            o.insert(*W.ragged([arg]), 4)
        else:
            o.evict(0, arg)
        for i in range(6):
            nd = o.block_info(i)
            if nd["live"]:
                worst = max(worst, nd["last_use"] - o.epoch())
    assert worst > 0                                        # some live priority was above calls x 1 request per call


@pytest.mark.parametrize("host", [0, 40])
def test_gdsf_literal_loop_equals_sorted_form_and_priorities_are_monotone(host):
    for seed in range(40):
        rng = np.random.default_rng(seed)
        # a random script of serving steps, generated once and then run on two oracles
        seqs, script = [], []
        for step in range(30):
            base = seqs[int(rng.integers(0, len(seqs)))] if seqs and rng.random() < 0.7 else np.zeros(0, dtype=np.int32)
            cut = int(rng.integers(0, len(base) + 1))
            seqs.append(np.concatenate([base[:cut], rng.integers(0, 3, size=int(rng.integers(2, 9)), dtype=np.int32)])[:20])
            batch = [seqs[int(rng.integers(0, len(seqs)))] for _ in range(int(rng.integers(1, 4)))] + [seqs[-1]]
            script.append((batch, bool(rng.random() < 0.5), int(rng.integers(0, 2)) if host else 0, int(rng.integers(0, 12)),
                           bool(rng.random() < 0.7)))
        logs = []
        for literal in (True, False):
            o = Oracle(1, 1, 8, 2, 2, seed, 96, host, policy="gdsf")
            log, held = [], []
            for batch, pin, tier, n, release_now in script:
                m, ids = o.lookup(*W.ragged(batch), 10, PIN if pin else 0)
                l0 = o.inflation()
                ne, v = o.evict(tier, n, literal=literal)
                assert o.inflation() >= l0
                ins, newb = o.insert(*W.ragged(batch), 10)
                if pin:
                    if release_now:
                        o.release(ids, m)
                    else:
                        held.append((ids, m))
                log.append((m.tolist(), ids.tolist(), ne.tolist(), v.tolist(), ins.tolist(), newb.tolist(), o.inflation(), o.status()))
            nodes = all_nodes(o)
            for i, nd in nodes.items():
                if nd["parent"] >= 0:
                    assert nodes[nd["parent"]]["last_use"] >= nd["last_use"]       # priority never rises towards the leaves
                    assert nodes[nd["parent"]]["freq"] >= nd["freq"]
                    assert nodes[nd["parent"]]["refcount"] >= nd["refcount"]
            logs.append(log)
        assert logs[0] == logs[1], seed


def test_mix_avalanche():
    """Flipping one input bit flips every output bit with probability close to one half."""
    rng = np.random.default_rng(7)
    trials = 4000
    counts = np.zeros(64, dtype=np.int64)
    for _ in range(trials):
        x = int(rng.integers(0, 1 << 63)) | (int(rng.integers(0, 2)) << 63)
        bit = int(rng.integers(0, 64))
        d = H["mix"](x) ^ H["mix"](x ^ (1 << bit))
        counts += np.array([(d >> b) & 1 for b in range(64)])
    p = counts / trials
    assert 0.45 < p.min() and p.max() < 0.55, (p.min(), p.max())


def test_chained_keys_spread_evenly_over_a_table():
    """Home slots floor(key * slots / 2^64) of 50,000 chained keys fill a 71,429-slot table like uniform draws would."""
    rng = np.random.default_rng(8)
    o = Oracle(1, 1, 8, 2, 16, 3, 4)
    seqs = [rng.integers(0, 128000, size=16 * 10, dtype=np.int32) for _ in range(5000)]
    keys = o.hash(*W.ragged(seqs), 10).ravel()
    assert len(np.unique(keys)) == 50000
    slots = 71429
    home = np.array([(int(k) * slots) >> 64 for k in keys])
    occupied = len(np.unique(home))
    expect = slots * (1 - np.exp(-50000 / slots))                      # balls into bins
    assert abs(occupied - expect) / expect < 0.01
    assert np.bincount(home, minlength=slots).max() <= 8


def test_threaded_read_only_pass_equals_the_single_threaded_functions():
    """The baseline's all-cores variant (lookup without stamps or pins + fetch, requests split over threads) against the
    plain functions on the tiny config, for several thread counts including more threads than requests."""
    w = W.tiny()
    sh, B = w.shape, w.shape.block_tokens
    rng = np.random.default_rng(3)
    o = Oracle(sh.layers, sh.heads, sh.dim, sh.elem_bytes, B, 0, w.pool_blocks)
    smb = W.max_blocks_of(w.store_seqs, B)
    need = sum(len(s) // B for s in w.store_seqs)
    o.insert(*W.ragged(w.store_seqs), smb, W.random_kv_cache(1, sh, need), W.shuffled_block_tables(rng, w.store_seqs, B, smb, need))
    batch = w.queries + w.store_seqs[:9]
    mb = W.max_blocks_of(batch, B)
    toks, offs = W.ragged(batch)
    nd = sum(len(s) // B for s in batch) + 3
    bt = W.shuffled_block_tables(rng, batch, B, mb, nd)
    m0, i0 = o.lookup(toks, offs, mb, NO_TOUCH)
    want = o.new_cache(nd, fill=9)
    o.fetch(i0, m0, want, bt)
    stamps = [o.block_info(i)["last_use"] for i in range(64)]
    for threads in (1, 2, 5, 64):
        got = o.new_cache(nd, fill=9)
        e0 = o.epoch()
        m, ids = o.lookup_fetch_threads(toks, offs, mb, got, bt, threads)
        assert (m == m0).all() and (ids == i0).all() and o.epoch() == e0 + 1
        for l in range(sh.layers):
            assert (got[l] == want[l]).all()
    assert stamps == [o.block_info(i)["last_use"] for i in range(64)] and o.status() == 0
