"""Seeded call histories shared by the oracle pins and the GPU parity tests (inputs only, no store arithmetic)."""
import numpy as np


def small_request_gdsf_history(steps, seed=10):
    """One request per call on a tiny store under GDSF, long enough for priorities to outgrow the call count.
    Yields after every call so that a second implementation can be driven in lock step."""
    rng = np.random.default_rng(seed)
    seqs = [rng.integers(0, 3, size=int(rng.integers(1, 4)), dtype=np.int32) for _ in range(6)]
    for step in range(steps):
        s = seqs[int(rng.integers(0, 6))]
        if rng.random() < 0.5:
            yield ("lookup", s)
        else:
            yield ("insert", s)
        if rng.random() < 0.6:
            yield ("evict", int(rng.integers(1, 3)))
