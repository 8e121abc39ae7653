"""The seeded input generators: reproducible, and shaped as the five workload descriptions say."""
import numpy as np

from paper_2607_22648_b200 import workloads as W


def test_generators_are_deterministic():
    a, b = W.tiny(), W.tiny()
    assert all((x == y).all() for x, y in zip(a.store_seqs + a.queries, b.store_seqs + b.queries))
    s1, s2 = W.llama8b_stream(n_docs=20), W.llama8b_stream(n_docs=20)
    for _ in range(3):
        (q1, t1), (q2, t2) = s1.batch(5), s2.batch(5)
        assert all((x == y).all() for x, y in zip(q1, q2)) and all((x == y).all() for x, y in zip(t1, t2))
    c1, c2 = W.conversation_stream(n_conversations=6), W.conversation_stream(n_conversations=6)
    for _ in range(4):
        assert all((x == y).all() for x, y in zip(c1.batch(3)[0], c2.batch(3)[0]))


def test_tiny_config_shape():
    w = W.tiny()
    assert len(w.store_seqs) == 64 and all(len(s) == 512 for s in w.store_seqs)
    assert len(w.queries) == 8 and all(len(q) == 1024 for q in w.queries)
    assert w.shape.chunk_bytes == 8192 and w.shape.block_bytes == 32768 and w.pool_blocks == 2048
    # stored sequences branch: some share a prefix with an earlier one, not block aligned in general
    shared = [max(int(np.argmax(a[:512] != b[:512])) if (a != b).any() else 512 for b in w.store_seqs[:i])
              for i, a in enumerate(w.store_seqs) if i]
    assert max(shared) > 256 and any(x % 16 for x in shared)


def test_llama_shapes_and_stream_statistics():
    assert W.LLAMA3_8B.chunk_bytes == 32 << 10 and W.LLAMA3_8B.block_bytes == 2 << 20
    assert W.LLAMA3_70B.chunk_bytes == 64 << 10 and W.LLAMA3_70B.block_bytes == 10 << 20
    st = W.llama8b_stream()
    lens = np.array([len(d) for d in st.docs])
    assert len(st.docs) == 500 and lens.min() >= 2000 and lens.max() <= 6000 and st.max_blocks == 391
    assert abs(st.probs.sum() - 1) < 1e-12 and st.probs.max() / np.sort(st.probs)[-2] > 2.0     # Zipf(1.1): p1/p2 = 2^1.1
    seqs, tags = st.batch(64)
    for s, t in zip(seqs, tags):
        assert 64 <= len(s) - max(len(d) for d in st.docs if len(d) <= len(s) and (s[:len(d)] == d).all()) <= 256
        assert len(t) == len(s) // 16
    # tags: equal for equal block-aligned prefixes, distinct otherwise
    seen = {}
    for s, t in zip(seqs, tags):
        for j, tag in enumerate(t):
            key = s[:(j + 1) * 16].tobytes()
            assert seen.setdefault(key, int(tag)) == int(tag)
    assert len(set(seen.values())) == len(seen)


def test_lookup_stress_shape():
    ws = W.lookup_stress(n_roots=500, n_queries=256)
    assert ws.n_nodes == 500 * 20 and ws.table_slots == int(np.ceil(500 * 20 / 0.7))
    assert len(ws.store_seqs) == 1500 and all(len(q) == 1024 for q in ws.queries)
    distinct = set()
    for s in ws.store_seqs:
        for j in range(1, len(s) // 16 + 1):
            distinct.add(s[:j * 16].tobytes())
    assert len(distinct) == ws.n_nodes
    assert 4.0 < ws.hit_depth.mean() < 9.0
    full = W.lookup_stress.__defaults__
    assert full[1] == 50000 and full[4] == 16384 and full[5] == 64          # 10^6 nodes, 16,384 x 64 probe blocks


def test_payload_generator_numpy_equals_torch():
    import torch
    tags = np.array([1, (3 << 24) | 7, ((1 << 30) + 5) << 24 | 300], dtype=np.uint64)
    a = W.payload_words(tags, 1000)
    b = W.payload_words(torch.from_numpy(tags.astype(np.int64)), 1000, xp=torch).numpy()
    assert (a == b).all()
    halves = a.view(np.uint16)
    assert not (halves & 0x4000).any()                                       # bf16 exponent bit 14 clear: finite, |x| < 2
    assert len(np.unique(a[0])) > 900 and (a[0] != a[1]).mean() > 0.99
