"""Minibatch sampling xi_k^(i) ~ D_i and the non-IID partition table.

The paper only says that worker i draws a random minibatch from its own data
distribution D_i at every iteration (Section 2, the sentence after Eq. 2) and
that the stochastic gradient is unbiased (Section 4, assumption 2).  The
reading taken here: B indices drawn independently and uniformly WITH
replacement from worker i's n samples, a pure function of
(seed, worker i, iteration k, slot j).

Rule.  Slot j sits in Philox block q = j // 4, lane r = j % 4.  The block is
Philox4x32-10 with counter (q, k, i, 1) and key (seed mod 2^32, seed >> 32).
The index is floor(word_r * n / 2^32), i.e. the high 32 bits of the 64-bit
product, which lies in [0, n).

Partition table (stand-in for the paper's skewed non-IID split, Section 4,
"non-IID" paragraph).  Each worker holds samples of exactly two of the ten
classes.  Class slots are the concatenation of seeded Fisher-Yates
permutations of 0..9; worker i takes slots 2i and 2i+1 (distinct, because ten
is even).  Permutation t is shuffled from the identity for p = 9 down to 1 by
swapping entries p and floor(w * (p+1) / 2^32), where w is word 0 of the Philox
block with counter (p, t, 0, 2) and the same key.

This is test infrastructure (see the package docstring).
"""
import numpy as np

from .philox import philox4x32_10

STREAM_MINIBATCH = 1
STREAM_PARTITION = 2
N_CLASSES = 10


def _key(seed):
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    return seed & 0xFFFFFFFF, seed >> 32


def minibatch_indices(seed, m, k, batch, n):
    """int32 array [m][batch]: sample indices of every worker at iteration k."""
    k0, k1 = _key(seed)
    i = np.arange(m, dtype=np.uint64)[:, None]
    j = np.arange(batch, dtype=np.uint64)[None, :]
    words = philox4x32_10(j // np.uint64(4), np.uint64(k), i,
                          np.uint64(STREAM_MINIBATCH), k0, k1)
    lane = (j % np.uint64(4)) + np.zeros_like(i)
    w = np.choose(lane.astype(np.int64), words)
    idx = (w * np.uint64(n)) >> np.uint64(32)
    return idx.astype(np.int32)


def class_pairs(seed, m):
    """int32 array [m][2]: the two classes worker i samples from."""
    k0, k1 = _key(seed)
    n_perm = (2 * m + N_CLASSES - 1) // N_CLASSES
    slots = []
    for t in range(n_perm):
        perm = list(range(N_CLASSES))
        for p in range(N_CLASSES - 1, 0, -1):
            w = int(philox4x32_10(p, t, 0, STREAM_PARTITION, k0, k1)[0])
            q = (w * (p + 1)) >> 32
            perm[p], perm[q] = perm[q], perm[p]
        slots.extend(perm)
    return np.asarray(slots[:2 * m], dtype=np.int32).reshape(m, 2)
