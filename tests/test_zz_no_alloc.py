"""ptstore_fetch_static — the gather for callers that cannot allocate device memory (for example code that
runs after a serving engine has fixed its memory budget, or a plugin that is given pointers but no
allocator).  Its scratch is a fixed array inside the library, shared by all calls, so stale contents from
one call must not leak into the next: the test makes two calls in a row with different batches and
compares each, byte for byte, with what the CPU oracle's fetch writes for the same inputs (and with the
ordinary ptstore_fetch, which has to agree with both).

Collected last on purpose (file name), so that a run that stops at the first failure has already run
every other test.  Passes alone in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2607_22648_b200 import workloads as W


def test_fetch_static_matches_fetch_twice_in_a_row():
    from paper_2607_22648_b200 import binding as G
    from oracle import Oracle
    sh = W.TINY
    B = sh.block_tokens
    w = W.tiny(seed=W.BASE_SEED + 50, n_store=24, store_len=320, n_query=8, query_len=480)
    rng = np.random.default_rng(11)
    st = G.PTStore(sh.layers, sh.heads, sh.dim, B, 512, max_requests=32, max_batch_blocks=32 * 32)

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    # fill the store through the ordinary path
    mb = W.max_blocks_of(w.store_seqs, B)
    need = sum(len(s) // B for s in w.store_seqs)
    src_np = W.random_kv_cache(3, sh, need)
    src = G.PagedKV(sh.layers, need, sh.chunk_bytes, tensors=[dev(a) for a in src_np])
    toks, offs = W.ragged(w.store_seqs)
    src_bt = W.shuffled_block_tables(rng, w.store_seqs, B, mb, need)
    st.insert(dev(toks), dev(offs), mb, src, dev(src_bt))
    assert st.status() == 0
    # the CPU oracle holds the same store: it supplies the expected bytes
    o = Oracle(sh.layers, sh.heads, sh.dim, sh.elem_bytes, B, 0, 512)
    o.insert(toks, offs, mb, src_np, src_bt)

    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    # two different batches, back to back: the second is smaller, so leftovers of the first would show
    for batch in (w.queries + w.store_seqs[:8], w.queries[:3]):
        qmb = W.max_blocks_of(batch, B)
        qt, qo = W.ragged(batch)
        matched, ids = st.lookup(dev(qt), dev(qo), qmb)
        mo, io = o.lookup(qt, qo, qmb)
        assert (mo == matched.cpu().numpy()).all() and (io == ids.cpu().numpy()).all()
        total = int(matched.sum().item())
        assert total > 0
        nd = total + 5
        bt = np.full((len(batch), qmb), -1, dtype=np.int32)
        perm, k = rng.permutation(nd), 0
        mh = matched.cpu().numpy()
        for r in range(len(batch)):
            for j in range(mh[r]):
                bt[r, j] = perm[k]
                k += 1
        bt_d = dev(bt)
        want = G.PagedKV(sh.layers, nd, sh.chunk_bytes)
        got = G.PagedKV(sh.layers, nd, sh.chunk_bytes)
        for t in want.tensors + got.tensors:
            t.fill_(0xEE)
        st.fetch(ids, matched, want, bt_d)
        G.fetch_static(st.hbm_pool, st.hbm_blocks, sh.layers, sh.chunk_bytes, ids, matched, got, bt_d, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        expect = o.new_cache(nd, fill=0xEE)
        o.fetch(io, mo, expect, bt)
        for l in range(sh.layers):
            assert torch.equal(got.tensors[l].cpu(), torch.from_numpy(expect[l])), "layer %d differs from the oracle" % l
            assert torch.equal(got.tensors[l], want.tensors[l]), "layer %d differs from ptstore_fetch" % l
        assert not bool((got.tensors[0] == 0xEE).all())          # something was written
    # out-of-range entries are skipped and reported, as in ptstore_fetch
    bad = bt_d.clone()
    r0 = int(torch.nonzero(matched)[0].item())             # a request that matched something
    bad[r0, 0] = nd + 100
    G.fetch_static(st.hbm_pool, st.hbm_blocks, sh.layers, sh.chunk_bytes, ids, matched, got, bad, status)
    torch.cuda.synchronize()
    assert int(status.item()) == G.S_BOUNDS
    # sizes beyond the fixed scratch are refused with a clear error, before anything is enqueued
    big_ids = torch.zeros((G.STATIC_MAX_REQUESTS + 1, 1), dtype=torch.int32, device="cuda")
    big_m = torch.zeros(G.STATIC_MAX_REQUESTS + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(G.PTStoreError) as e:
        G.fetch_static(st.hbm_pool, st.hbm_blocks, sh.layers, sh.chunk_bytes, big_ids, big_m, got, big_ids, status)
    assert e.value.code == G.E_LIMIT
    wide = torch.zeros((2, G.STATIC_MAX_PAIRS // 2 + 1), dtype=torch.int32, device="cuda")
    with pytest.raises(G.PTStoreError) as e:
        G.fetch_static(st.hbm_pool, st.hbm_blocks, sh.layers, sh.chunk_bytes, wide, big_m[:2], got, wide, status)
    assert e.value.code == G.E_LIMIT
    st.close()
    o.close()
