"""Random-k sparsifier for the oracle — TEST INFRASTRUCTURE ONLY.

The paper's appendix on other compressors uses Random-k ("random k% of entries") in place of
Top-k.  Reading taken here (the paper does not say how the k entries are drawn): for worker i
at iteration t every index j gets a pseudo-random priority and the k largest priorities are
kept, equal priorities by increasing index.  That is a uniform draw without replacement of
exactly k indices.  The priorities come from the counter-based generator Philox-4x32-10
(Salmon, Moraes, Dror, Shaw, SC'11), implemented below from its published definition:

    priority(j) = Philox4x32_10(key = (seed_lo, seed_hi),
                                counter = (j // 4, t_lo, i, t_hi ^ 0x52414E44))[j % 4] >> 9
"""
import numpy as np

M0, M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Vectorised Philox-4x32 with 10 rounds.  Counters: uint32 arrays (broadcastable);
    key: two Python ints.  Returns four uint32 arrays."""
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & MASK for c in (c0, c1, c2, c3))
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    for r in range(10):
        p0 = M0 * c0                                     # 64-bit products of 32-bit words
        p1 = M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & MASK
        kk0 = np.uint64((k0 + r * W0) & 0xFFFFFFFF)      # key bumped by the Weyl constants
        kk1 = np.uint64((k1 + r * W1) & 0xFFFFFFFF)
        c0, c1, c2, c3 = hi1 ^ c1 ^ kk0, lo1, hi0 ^ c3 ^ kk1, lo0
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def priorities(d, seed, step, worker):
    """23-bit priority of every index 0..d-1 for (seed, step, worker)."""
    groups = np.arange((d + 3) // 4, dtype=np.uint64)
    out = philox4x32_10(groups, step & 0xFFFFFFFF, worker, ((step >> 32) & 0xFFFFFFFF) ^ 0x52414E44,
                        seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    return (np.stack(out, axis=1).reshape(-1)[:d] >> np.uint32(9)).astype(np.uint32)


def randk_select(d, k, seed, step, worker):
    """Indices (ascending) of the k largest priorities; equal priorities -> lower index."""
    pr = priorities(d, seed, step, worker).astype(np.uint64)
    idx = np.arange(d, dtype=np.uint64)
    word = (pr << np.uint64(32)) | (np.uint64(0xFFFFFFFF) - idx)
    word.sort()
    top = word[d - k:]
    sel = (np.uint64(0xFFFFFFFF) - (top & np.uint64(0xFFFFFFFF))).astype(np.uint32)
    sel.sort()
    return sel
