"""Pins for the checker's counter-based random numbers, fold split and minibatch order."""
import os

import numpy as np
import pytest

import oracle

M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
MASK = 0xFFFFFFFF


def philox_int(ctr, key, rounds=10):
    """Philox-4x32 restated with Python big integers (independent of the C++)."""
    c = list(ctr)
    k = list(key)
    for _ in range(rounds):
        p0, p1 = M0 * c[0], M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & MASK, (p0 >> 32) ^ c[3] ^ k[1], p0 & MASK]
        k = [(k[0] + W0) & MASK, (k[1] + W1) & MASK]
    return c


def philox_inverse(out, key, rounds=10):
    """The inverse bijection: recovers the counter from the output."""
    inv0, inv1 = pow(M0, -1, 1 << 32), pow(M1, -1, 1 << 32)
    ks = [list(key)]
    for _ in range(rounds - 1):
        ks.append([(ks[-1][0] + W0) & MASK, (ks[-1][1] + W1) & MASK])
    c = list(out)
    for r in reversed(range(rounds)):
        x2 = (c[1] * inv1) & MASK
        x0 = (c[3] * inv0) & MASK
        x1 = c[0] ^ ((M1 * x2) >> 32) ^ ks[r][0]
        x3 = c[2] ^ ((M0 * x0) >> 32) ^ ks[r][1]
        c = [x0, x1, x2, x3]
    return c


def test_published_known_answers(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) if l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        got = oracle.philox_raw(v[0:4], v[4:6])
        assert [int(x) for x in got] == v[6:10]
        assert philox_int(v[0:4], v[4:6]) == v[6:10]


def test_matches_bigint_restatement_and_edges():
    rng = np.random.default_rng(5)
    cases = [(0, 1, 0, 0, 0, 0), (2**64 - 1, 3, MASK, MASK, 2**28 - 1, MASK), (7, 2, 0, MASK, 0, 1)]
    for _ in range(3000):
        cases.append((int(rng.integers(0, 2**64, dtype=np.uint64)), int(rng.integers(0, 16)),
                      int(rng.integers(0, 2**32)), int(rng.integers(0, 2**32)),
                      int(rng.integers(0, 2**28)), int(rng.integers(0, 2**32))))
    for seed, stream, a, b, c, blk in cases:
        got = [int(x) for x in oracle.rng_block(seed, stream, a, b, c, blk)]
        ctr = [blk, a, b, (stream << 28) | c]
        key = [seed & MASK, seed >> 32]
        want = philox_int(ctr, key)
        assert got == want
        assert philox_inverse(got, key) == ctr  # a bijection of the counter


def test_streams_do_not_collide_and_look_uniform():
    seen = set()
    words = []
    for stream in (1, 2, 3):
        for a in range(4):
            for blk in range(64):
                w = tuple(int(x) for x in oracle.rng_block(0, stream, a, 1, 2, blk))
                assert w not in seen
                seen.add(w)
                words.extend(w)
    u = (np.array(words, np.uint64) >> 8).astype(np.float64) * 2.0**-24
    assert abs(u.mean() - 0.5) < 0.02
    assert abs(u.var() - 1.0 / 12.0) < 0.01
    byte = np.array(words, np.uint64) & 0xFF
    counts = np.bincount(byte.astype(np.int64), minlength=256)
    chi2 = ((counts - len(words) / 256.0) ** 2 / (len(words) / 256.0)).sum()
    assert chi2 < 400.0  # 255 dof: mean 255, sd ~22.6


@pytest.mark.parametrize("N", [1, 2, 5, 120, 1438, 2048, 5000])
def test_perm_is_sort_of_keys(N):
    p = oracle.perm(N, 42, oracle.STREAM_PERM, 3, 4, 5)
    assert sorted(p.tolist()) == list(range(N))
    # brute force from the definition: key_i = word_i << 32 | i, ascending
    words = []
    for blk in range((N + 3) // 4):
        words.extend(philox_int([blk, 3, 4, (3 << 28) | 5], [42, 0]))
    keys = sorted((words[i] << 32) | i for i in range(N))
    assert [k & MASK for k in keys] == p.tolist()


@pytest.mark.parametrize("n,K", [(150, 5), (569, 5), (1797, 5), (442, 5), (11, 3), (7, 7), (10, 2)])
def test_fold_split_partition(n, K):
    pi, fo = oracle.fold_split(n, K, 0)
    assert sorted(pi.tolist()) == list(range(n))
    sizes = np.bincount(fo, minlength=K)
    assert sizes.sum() == n and fo.min() == 0 and fo.max() == K - 1
    rem = n % K
    assert sizes.tolist() == [n // K + (1 if f < rem else 0) for f in range(K)]
    # folds are contiguous segments of pi
    off = 0
    for f in range(K):
        assert set(pi[off:off + sizes[f]].tolist()) == set(np.nonzero(fo == f)[0].tolist())
        off += sizes[f]
    # the split depends on the seed
    assert not np.array_equal(oracle.fold_split(n, K, 1)[0], pi) or n < 4


def test_epoch_order_is_permutation_of_train_rows():
    n, K = 569, 5
    pi, fo = oracle.fold_split(n, K, 9)
    for fold in (0, 4):
        train_rows = set(np.nonzero(fo != fold)[0].tolist())
        o0 = oracle.epoch_order(n, K, 9, 2, fold, 0)
        o1 = oracle.epoch_order(n, K, 9, 2, fold, 1)
        o2 = oracle.epoch_order(n, K, 9, 3, fold, 0)
        for o in (o0, o1, o2):
            assert len(o) == len(train_rows) and set(o.tolist()) == train_rows
        assert not np.array_equal(o0, o1) and not np.array_equal(o0, o2)
    # train list keeps pi order with the held-out segment removed
    sig = oracle.perm(len(o0), 9, oracle.STREAM_PERM, 2, 4, 0)
    tlist = np.array([r for r in pi.tolist() if fo[r] != 4])
    assert np.array_equal(tlist[sig], oracle.epoch_order(n, K, 9, 2, 4, 0))


def test_glorot_init_bounds_and_moments():
    d, H, C = 64, 200, 10
    th = oracle.init_params(d, H, C, 0, 7, 3)
    b1 = np.sqrt(np.float32(6.0) / np.float32(d + H))
    b2 = np.sqrt(np.float32(6.0) / np.float32(H + C))
    W1 = th[: d * H]
    rest = th[d * H + H: d * H + H + H * C]
    assert np.all(np.abs(W1) <= b1) and np.all(np.abs(rest) <= b2)
    assert np.all(np.abs(th[d * H: d * H + H]) <= b1) and np.all(np.abs(th[-C:]) <= b2)
    assert abs(W1.mean()) < 4 * b1 / np.sqrt(3 * W1.size)
    assert abs(W1.var() / (float(b1) ** 2 / 3.0) - 1.0) < 0.05
    assert abs(rest.var() / (float(b2) ** 2 / 3.0) - 1.0) < 0.1
    # every value is bound * (2u-1) with u a multiple of 2^-24, from the INIT stream
    w = philox_int([0, 7, 3, (2 << 28) | 0], [0, 0])
    u = np.float32(w[1] >> 8) * np.float32(2.0**-24)
    assert th[1] == float(b1 * (np.float32(2.0) * u - np.float32(1.0)))

    # one hand-recomputed element of every other block of the parameter vector: the layer tag
    # (1 = b1, 2 = W2, 3 = b2) sits in the low bits of the last counter word, element i is word
    # i & 3 of block i >> 2, W2 is indexed j * C + o, and each layer uses its own bound
    def draw(layer, idx, bound):
        w = philox_int([idx >> 2, 7, 3, (2 << 28) | layer], [0, 0])[idx & 3]
        return float(bound * (np.float32(2.0) * (np.float32(w >> 8) * np.float32(2.0**-24)) - np.float32(1.0)))

    assert th[d * H + 5] == draw(1, 5, b1)                                   # b1[5]
    assert th[d * H + H + 37 * C + 4] == draw(2, 37 * C + 4, b2)             # W2[37][4]
    assert th[d * H + H + H * C + 9] == draw(3, 9, b2)                       # b2[9]
    assert th[3 * H + 130] == draw(0, 3 * H + 130, b1)                       # W1[3][130]
    assert len({draw(t, 9, b2) for t in (1, 2, 3)}) == 3                     # swapping two tags would show
    # different (config, fold) -> different draw; all values float32-representable
    assert not np.array_equal(th, oracle.init_params(d, H, C, 0, 7, 4))
    assert np.array_equal(th, th.astype(np.float32).astype(np.float64))
