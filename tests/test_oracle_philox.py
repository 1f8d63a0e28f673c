"""Pins for oracle.philox and oracle.sampling."""
import os

import numpy as np

from oracle import philox, sampling
from conftest import GOLDEN


def _kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers_scalar_and_vector():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert list(philox.philox_scalar(ctr, key)) == want
        got = philox.philox4x32_10(*ctr, *key)
        assert [int(g) for g in got] == want


def test_philox_vector_matches_scalar_on_random_counters():
    rng = np.random.default_rng(5)
    c = rng.integers(0, 2**32, size=(4, 64), dtype=np.uint64)
    k = rng.integers(0, 2**32, size=(2, 64), dtype=np.uint64)
    out = philox.philox4x32_10(c[0], c[1], c[2], c[3], k[0], k[1])
    for t in range(64):
        want = philox.philox_scalar(c[:, t], k[:, t])
        assert tuple(int(o[t]) for o in out) == want


def test_philox_output_bits_are_balanced():
    # a dropped round or a wrong multiplier shows up as biased bits long
    # before it shows up in the KAT rows' neighbours
    n = 1 << 14
    out = philox.philox4x32_10(np.arange(n), 0, 0, 0, 7, 9)
    words = np.concatenate([o for o in out])
    for b in range(32):
        frac = float(((words >> np.uint64(b)) & np.uint64(1)).mean())
        assert abs(frac - 0.5) < 0.01, (b, frac)


def test_indices_range_shape_determinism():
    a = sampling.minibatch_indices(0, 16, 3, 128, 5000)
    b = sampling.minibatch_indices(0, 16, 3, 128, 5000)
    assert a.dtype == np.int32 and a.shape == (16, 128)
    assert np.array_equal(a, b)
    assert a.min() >= 0 and a.max() < 5000
    assert not np.array_equal(a[0], a[1])                     # workers differ
    assert not np.array_equal(a, sampling.minibatch_indices(0, 16, 4, 128, 5000))
    assert not np.array_equal(a, sampling.minibatch_indices(1, 16, 3, 128, 5000))


def test_indices_follow_the_stated_rule_by_brute_force():
    seed, m, k, B, n = 0x1234567890ABCDEF, 3, 77, 10, 1000
    got = sampling.minibatch_indices(seed, m, k, B, n)
    for i in range(m):
        for j in range(B):
            words = philox.philox_scalar((j // 4, k, i, 1),
                                         (seed & 0xFFFFFFFF, seed >> 32))
            assert got[i, j] == (words[j % 4] * n) >> 32


def test_indices_are_uniform_chi_square():
    n, B = 50, 128
    counts = np.zeros(n)
    for k in range(400):
        idx = sampling.minibatch_indices(11, 4, k, B, n)
        counts += np.bincount(idx.ravel(), minlength=n)
    expect = counts.sum() / n
    chi2 = ((counts - expect) ** 2 / expect).sum()
    # 49 degrees of freedom: mean 49, sd ~9.9; 110 is > 6 sd
    assert chi2 < 110, chi2


def test_indices_prefix_property_and_ragged_batch():
    # slot j depends only on (seed, i, k, j): a shorter batch is a prefix
    a = sampling.minibatch_indices(3, 2, 5, 7, 999)
    b = sampling.minibatch_indices(3, 2, 5, 64, 999)
    assert np.array_equal(a, b[:, :7])


def test_class_pairs_are_permutation_slots():
    for seed in (0, 1, 99):
        for m in (1, 4, 5, 64):
            cp = sampling.class_pairs(seed, m)
            assert cp.shape == (m, 2) and cp.dtype == np.int32
            assert (cp[:, 0] != cp[:, 1]).all()
            flat = cp.ravel()
            for t in range(len(flat) // 10):
                assert sorted(flat[10 * t:10 * t + 10]) == list(range(10))
    assert not np.array_equal(sampling.class_pairs(0, 64), sampling.class_pairs(1, 64))


def test_class_pairs_shuffle_is_uniform():
    # Fisher-Yates must leave every class equally likely in every slot
    counts = np.zeros((10, 10))
    for seed in range(3000):
        perm = sampling.class_pairs(seed, 5).ravel()
        counts[np.arange(10), perm] += 1
    chi2 = ((counts - 300.0) ** 2 / 300.0).sum()
    # 81 degrees of freedom, sd ~12.7
    assert chi2 < 160, chi2


# ------------------------------------------------------------ epoch rule

def test_epoch_permutation_is_a_bijection_for_awkward_sizes():
    for n in (1, 2, 3, 5, 16, 17, 100, 1000, 1024, 1025):
        for seed, i, e in ((0, 0, 0), (9, 3, 7)):
            vals = [sampling.epoch_permutation(seed, i, e, o, n) for o in range(n)]
            assert sorted(vals) == list(range(n)), (n, seed, i, e)


def test_epoch_permutation_inverts_round_by_round():
    # structural pin: undo the four Feistel rounds (and the cycle walk) with the inverse
    # network written here; a wrong half swap or round index would not invert
    n, seed, i, e = 777, 5, 2, 3
    k0, k1 = seed & 0xFFFFFFFF, seed >> 32
    h = ((n - 1).bit_length() + 1) // 2
    mask = (1 << h) - 1

    def inverse(v):
        while True:
            left, right = v >> h, v & mask
            for r in (3, 2, 1, 0):
                f = int(philox.philox4x32_10(left, 4 * e + r, i, 3, k0, k1)[0]) & mask
                left, right = right ^ f, left
            v = (left << h) | right
            if v < n:
                return v

    for o in range(0, n, 7):
        assert inverse(sampling.epoch_permutation(seed, i, e, o, n)) == o


def test_epoch_rule_visits_every_sample_once_per_epoch():
    seed, m, B, n = 4, 3, 8, 40               # 5 iterations per epoch
    seen = np.concatenate([sampling.minibatch_indices_epoch(seed, m, k, B, n) for k in range(5)], axis=1)
    for i in range(m):
        assert sorted(seen[i]) == list(range(n))
    nxt = np.concatenate([sampling.minibatch_indices_epoch(seed, m, k, B, n) for k in range(5, 10)], axis=1)
    for i in range(m):
        assert sorted(nxt[i]) == list(range(n)) and not np.array_equal(nxt[i], seen[i])
    assert not np.array_equal(seen[0], seen[1])


def test_epoch_rule_straddles_epochs_and_respects_worker_offset():
    seed, B, n = 6, 16, 40                    # iteration 2 takes draws 32..47: epochs 0 and 1
    a = sampling.minibatch_indices_epoch(seed, 4, 2, B, n)
    for j in range(B):
        t = 2 * B + j
        assert a[1, j] == sampling.epoch_permutation(seed, 1, t // n, t % n, n)
    b = sampling.minibatch_indices_epoch(seed, 2, 2, B, n, worker_offset=2)
    assert np.array_equal(b, a[2:])


def test_epoch_permutation_first_position_is_uniform():
    n = 20
    counts = np.zeros(n)
    for seed in range(2000):
        counts[sampling.epoch_permutation(seed, 0, 0, 0, n)] += 1
    chi2 = ((counts - 100.0) ** 2 / 100.0).sum()
    assert chi2 < 60, chi2                      # 19 degrees of freedom
