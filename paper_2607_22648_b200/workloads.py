"""Seeded synthetic inputs shaped like long-shared-passage Q&A serving.

This module only PRODUCES INPUTS (token sequences, request streams, block tables, K/V payload bytes).
It holds none of the store's arithmetic (no hashing of blocks into keys, no trie, no matching) and is
the one module both the CUDA path's tests and the CPU oracle's tests draw from.

The paper's workloads are question answering over long shared passages: a request is one long
document followed by a short unique question, and documents are drawn with a heavy-tailed popularity
(Section 6.1).  The generators below reproduce that SHAPE with uniform random token ids; they stand in
for the datasets, which are not available here.

Numpy only; `payload_words` also accepts torch tensors so the same generator can fill device memory.
"""
from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 226070


@dataclass(frozen=True)
class KVShape:
    layers: int
    heads: int
    dim: int
    block_tokens: int
    elem_bytes: int = 2

    @property
    def chunk_bytes(self):
        return self.block_tokens * self.heads * self.dim * self.elem_bytes

    @property
    def block_bytes(self):
        return 2 * self.layers * self.chunk_bytes


TINY = KVShape(2, 4, 64, 16)
LLAMA3_8B = KVShape(32, 8, 128, 16)
LLAMA3_70B = KVShape(80, 8, 128, 32)


def ragged(seqs):
    """list of int32 arrays -> (tokens int32 [sum len], offsets int64 [R+1])"""
    offsets = np.zeros(len(seqs) + 1, dtype=np.int64)
    if len(seqs):
        offsets[1:] = np.cumsum([len(s) for s in seqs])
    tokens = np.concatenate(seqs).astype(np.int32) if len(seqs) and offsets[-1] > 0 else np.zeros(0, dtype=np.int32)
    return tokens, offsets


def max_blocks_of(seqs, block_tokens):
    return max(1, max((len(s) // block_tokens for s in seqs), default=1))


def zipf_probs(n, s):
    p = 1.0 / np.arange(1, n + 1, dtype=np.float64) ** s
    return p / p.sum()


# ---------------------------------------------------------------------------------------------------
# payload: counter-based bytes for a block identified by a 64-bit tag
# ---------------------------------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def payload_words(tags, words_per_block, xp=np):
    """int32 words [len(tags), words_per_block] of the K/V payload of blocks with the given tags.

    A splitmix-style counter generator: word i of block t depends only on (t, i), so any block (or any
    chunk of it) can be regenerated anywhere.  Every 16-bit half has bit 14 cleared, so read as bf16
    the values are finite and smaller than 2 in magnitude.  Works with numpy (xp=np) or torch (xp=torch,
    tags an int64 tensor on any device).
    """
    if xp is np:
        t = np.asarray(tags).astype(np.uint64).reshape(-1, 1)
        i = np.arange(words_per_block, dtype=np.uint64).reshape(1, -1)
        with np.errstate(over="ignore"):
            x = t * np.uint64(0xD6E8FEB86659FD93) + i * np.uint64(0x9E3779B97F4A7C15)
            x ^= x >> np.uint64(31)
            x *= np.uint64(0xBF58476D1CE4E5B9)
            x ^= x >> np.uint64(29)
        w = (x & np.uint64(0xBFFFBFFF)).astype(np.uint32)
        return w.view(np.int32)
    torch = xp
    t = tags.to(torch.int64).reshape(-1, 1)
    i = torch.arange(words_per_block, dtype=torch.int64, device=t.device).reshape(1, -1)

    def s64(v):  # python int -> the int64 with the same bit pattern
        return v - (1 << 64) if v >= (1 << 63) else v

    x = t * s64(0xD6E8FEB86659FD93) + i * s64(0x9E3779B97F4A7C15)
    x = x ^ ((x >> 31) & ((1 << 33) - 1))
    x = x * s64(0xBF58476D1CE4E5B9)
    x = x ^ ((x >> 29) & ((1 << 35) - 1))
    return (x & 0xBFFFBFFF).to(torch.int32)  # values above 2^31 wrap to the same 32 bits


# ---------------------------------------------------------------------------------------------------
# config 1: tiny branching store
# ---------------------------------------------------------------------------------------------------
@dataclass
class TinyWorkload:
    shape: KVShape
    store_seqs: list
    queries: list
    pool_blocks: int
    vocab: int
    seed: int


def tiny(seed=BASE_SEED, n_store=64, store_len=512, n_query=8, query_len=1024, vocab=32000, shape=TINY,
         pool_blocks=None):
    """Stored sequence i>0 copies the first L~U{0..store_len} tokens (not block aligned) of a uniformly
    chosen earlier sequence; queries are a random-length prefix of a stored sequence + fresh tokens."""
    rng = np.random.Generator(np.random.PCG64(seed))
    store = []
    for i in range(n_store):
        s = rng.integers(0, vocab, size=store_len, dtype=np.int32)
        if i > 0:
            src = store[int(rng.integers(0, i))]
            L = int(rng.integers(0, store_len + 1))
            s[:L] = src[:L]
        store.append(s)
    queries = []
    for _ in range(n_query):
        q = rng.integers(0, vocab, size=query_len, dtype=np.int32)
        src = store[int(rng.integers(0, n_store))]
        L = int(rng.integers(0, store_len + 1))
        q[:L] = src[:L]
        queries.append(q)
    if pool_blocks is None:
        pool_blocks = n_store * (store_len // shape.block_tokens)
    return TinyWorkload(shape, store, queries, pool_blocks, vocab, seed)


def random_kv_cache(seed, shape, num_blocks):
    """Per-layer paged cache [2, num_blocks, chunk_bytes] uint8 holding bf16 bit patterns of N(0,1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n_el = shape.chunk_bytes // 2
    out = []
    for _ in range(shape.layers):
        x = rng.standard_normal(size=(2, num_blocks, n_el), dtype=np.float32)
        bits = x.view(np.uint32)
        bf16 = ((bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
        out.append(np.ascontiguousarray(bf16).view(np.uint8).reshape(2, num_blocks, shape.chunk_bytes))
    return out


def shuffled_block_tables(rng, seqs, block_tokens, max_blocks, num_cache_blocks):
    """Give every full block of every request a distinct cache block, in shuffled order; -1 elsewhere."""
    R = len(seqs)
    bt = np.full((R, max_blocks), -1, dtype=np.int32)
    need = sum(min(len(s) // block_tokens, max_blocks) for s in seqs)
    assert need <= num_cache_blocks, (need, num_cache_blocks)
    perm = rng.permutation(num_cache_blocks)[:need].astype(np.int32)
    k = 0
    for r, s in enumerate(seqs):
        nb = min(len(s) // block_tokens, max_blocks)
        bt[r, :nb] = perm[k:k + nb]
        k += nb
    return bt


# ---------------------------------------------------------------------------------------------------
# configs 2, 4, 5: document + question streams with Zipf popularity
# ---------------------------------------------------------------------------------------------------
@dataclass
class DocStream:
    shape: KVShape
    docs: list                 # token arrays
    probs: np.ndarray          # popularity of doc i
    vocab: int
    suffix_range: tuple
    seed: int
    rng: np.random.Generator = field(repr=False, default=None)
    next_uid: int = 0

    @property
    def max_blocks(self):
        longest = max(len(d) for d in self.docs) + self.suffix_range[1]
        return -(-longest // self.shape.block_tokens)

    def batch(self, n_requests):
        """-> (seqs, tags): prompts = document + unique question; tags[r][j] identifies the payload of
        block j of request r (equal for equal token prefixes, distinct otherwise)."""
        B = self.shape.block_tokens
        seqs, tags = [], []
        for _ in range(n_requests):
            d = int(self.rng.choice(len(self.docs), p=self.probs))
            lo, hi = self.suffix_range
            sl = int(self.rng.integers(lo, hi + 1)) if hi > 0 else 0
            suffix = self.rng.integers(0, self.vocab, size=sl, dtype=np.int32)
            seq = np.concatenate([self.docs[d], suffix])
            nb = len(seq) // B
            doc_full = len(self.docs[d]) // B          # blocks made of document tokens only
            t = np.empty(nb, dtype=np.uint64)
            j = np.arange(nb, dtype=np.uint64)
            t[:] = (np.uint64(d + 1) << np.uint64(24)) | j
            uid = np.uint64((1 << 30) + self.next_uid)
            t[doc_full:] = (uid << np.uint64(24)) | j[doc_full:]
            self.next_uid += 1
            seqs.append(seq)
            tags.append(t)
        return seqs, tags


def doc_stream(seed, shape, n_docs, len_range, zipf_s, vocab, suffix_range):
    rng = np.random.Generator(np.random.PCG64(seed))
    docs = [rng.integers(0, vocab, size=int(rng.integers(len_range[0], len_range[1] + 1)), dtype=np.int32)
            for _ in range(n_docs)]
    probs = zipf_probs(n_docs, zipf_s)[rng.permutation(n_docs)]      # ranks assigned by a seeded shuffle
    return DocStream(shape, docs, probs, vocab, suffix_range, seed, rng)


def llama8b_stream(seed=BASE_SEED + 1, n_docs=500, len_range=(2000, 6000), shape=LLAMA3_8B):
    """config 2: 500 documents of 2k-6k tokens, Zipf(1.1), question suffix of 64-256 tokens."""
    return doc_stream(seed, shape, n_docs, len_range, 1.1, 128256, (64, 256))


def llama70b_stream(seed=BASE_SEED + 3, n_docs=18, doc_tokens=16384, shape=LLAMA3_70B):
    """config 4: 16k-token documents, Zipf(1.2); the prompt is the document itself plus a short question."""
    return doc_stream(seed, shape, n_docs, (doc_tokens, doc_tokens), 1.2, 128256, (32, 32))


def churn_stream(seed=BASE_SEED + 4, n_docs=5000, len_range=(1000, 8000), shape=LLAMA3_8B):
    """config 5: 5000 documents of 1k-8k tokens, Zipf(1.0), question suffix of 64-256 tokens."""
    return doc_stream(seed, shape, n_docs, len_range, 1.0, 128256, (64, 256))


def tags_matrix(tags, max_blocks):
    out = np.zeros((len(tags), max_blocks), dtype=np.uint64)
    for r, t in enumerate(tags):
        n = min(len(t), max_blocks)
        out[r, :n] = t[:n]
    return out


# ---------------------------------------------------------------------------------------------------
# config 3: lookup stress
# ---------------------------------------------------------------------------------------------------
@dataclass
class LookupStress:
    block_tokens: int
    store_seqs: list           # 3 per root: trunk, and two branches forking off the trunk
    queries: list
    hit_depth: np.ndarray      # intended matched blocks per query
    n_nodes: int
    table_slots: int
    vocab: int


def lookup_stress(seed=BASE_SEED + 2, n_roots=50000, trunk=12, branch=4, n_queries=16384, query_blocks=64,
                  block_tokens=16, vocab=128000, load=0.7, p_continue=0.9, all_hit=False):
    """Trie of n_roots*(trunk+2*branch) nodes; queries follow a random root-to-leaf path for a
    geometric(p_continue) number of blocks (truncated by the path), then fresh tokens."""
    rng = np.random.Generator(np.random.PCG64(seed))
    B = block_tokens
    store, paths = [], []
    for _ in range(n_roots):
        t = rng.integers(0, vocab, size=trunk * B, dtype=np.int32)
        store.append(t)
        root_paths = [t]
        for _b in range(2):
            f = int(rng.integers(1, trunk + 1))               # fork after f trunk blocks
            br = np.concatenate([t[:f * B], rng.integers(0, vocab, size=branch * B, dtype=np.int32)])
            store.append(br)
            root_paths.append(br)
        paths.append(root_paths)
    queries, depth = [], np.zeros(n_queries, dtype=np.int32)
    for q in range(n_queries):
        path = paths[int(rng.integers(0, n_roots))][int(rng.integers(0, 3))]
        pb = len(path) // B
        if all_hit:
            d = pb
            seq = path.copy()
        else:
            d = 0
            while d < pb and rng.random() < p_continue:
                d += 1
            seq = rng.integers(0, vocab, size=query_blocks * B, dtype=np.int32)
            seq[:d * B] = path[:d * B]
        queries.append(seq)
        depth[q] = d
    n_nodes = n_roots * (trunk + 2 * branch)
    return LookupStress(B, store, queries, depth, n_nodes, int(np.ceil(n_nodes / load)), vocab)


# ---------------------------------------------------------------------------------------------------
# multi-turn conversations: growing chains, deep tries, small increments
# ---------------------------------------------------------------------------------------------------
@dataclass
class ConversationStream:
    """Each conversation is an append-only token sequence; a request is the whole history plus a new turn, so
    all earlier full blocks are a stored prefix and every step adds only a few blocks per conversation."""
    shape: KVShape
    n_conversations: int
    turn_range: tuple
    max_tokens: int
    vocab: int
    seed: int
    rng: np.random.Generator = field(repr=False, default=None)
    history: list = field(repr=False, default_factory=list)

    @property
    def max_blocks(self):
        return -(-self.max_tokens // self.shape.block_tokens)

    def batch(self, n_requests):
        """-> (seqs, tags) for n_requests distinct conversations, each extended by one turn (a conversation that
        would outgrow max_tokens starts over with a fresh id)."""
        B = self.shape.block_tokens
        pick = self.rng.choice(self.n_conversations, size=min(n_requests, self.n_conversations), replace=False)
        seqs, tags = [], []
        for c in pick:
            uid, toks = self.history[c]
            turn = self.rng.integers(0, self.vocab, size=int(self.rng.integers(self.turn_range[0], self.turn_range[1] + 1)),
                                     dtype=np.int32)
            if len(toks) + len(turn) > self.max_tokens:
                uid, toks = self._fresh_uid(), np.zeros(0, dtype=np.int32)
            toks = np.concatenate([toks, turn])
            self.history[c] = (uid, toks)
            nb = len(toks) // B
            seqs.append(toks)
            tags.append((np.uint64(uid) << np.uint64(24)) | np.arange(nb, dtype=np.uint64))
        return seqs, tags

    def _fresh_uid(self):
        self._next = getattr(self, "_next", 0) + 1
        return (1 << 28) + self._next


def conversation_stream(seed=BASE_SEED + 5, shape=LLAMA3_8B, n_conversations=256, turn_range=(50, 400), max_tokens=8192,
                        vocab=128256):
    st = ConversationStream(shape, n_conversations, turn_range, max_tokens, vocab, seed,
                            np.random.Generator(np.random.PCG64(seed)))
    st.history = [(st._fresh_uid(), np.zeros(0, dtype=np.int32)) for _ in range(n_conversations)]
    return st
