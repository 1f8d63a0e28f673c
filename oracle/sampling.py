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
STREAM_EPOCH = 3
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


# ---------------------------------------------------------------------------
# Second sampling rule: one pass over D_i per epoch, without replacement.
#
# The paper's runs go through each node's partition epoch by epoch (Section 4: the data
# "is evenly partitioned across all nodes and not shuffled" between nodes).  Reading: worker
# i's draws are numbered t = k * B + j; draw t belongs to epoch e = t // n and takes sample
# pi_{i,e}(t mod n), where pi_{i,e} is a permutation of 0..n-1 that is a pure function of
# (seed, i, e), so no state is carried from step to step.
#
# pi is a balanced Feistel network with cycle walking (Black and Rogaway, "Ciphers with
# arbitrary finite domains", CT-RSA 2002): with h = ceil(ceil(log2 n) / 2) the value is split
# into two h-bit halves (L, R); four rounds (L, R) <- (R, L xor F_r(R)) permute 0..2^(2h)-1;
# the network is applied again until the result is below n.  F_r(R) is the low h bits of word
# 0 of the Philox4x32-10 block with counter (R, 4 * e + r, i, 3) and key (seed lo, seed hi).


def _half_bits(n):
    bits = max(1, int(n - 1).bit_length())
    return (bits + 1) // 2


def epoch_permutation(seed, i, e, o, n):
    """pi_{i,e}(o) for 0 <= o < n, as a Python int."""
    k0, k1 = _key(seed)
    h = _half_bits(n)
    mask = (1 << h) - 1
    v = int(o)
    while True:
        left, right = v >> h, v & mask
        for r in range(4):
            f = int(philox4x32_10(right, (4 * int(e) + r) & 0xFFFFFFFF, i, STREAM_EPOCH,
                                  k0, k1)[0]) & mask
            left, right = right, left ^ f
        v = (left << h) | right
        if v < n:
            return v


def minibatch_indices_epoch(seed, m, k, batch, n, worker_offset=0):
    """int32 [m][batch]: the epoch rule's indices of every worker at iteration k."""
    out = np.empty((m, batch), dtype=np.int32)
    for i in range(m):
        for j in range(batch):
            t = int(k) * batch + j
            out[i, j] = epoch_permutation(seed, i + worker_offset, t // n, t % n, n)
    return out
