"""Pins for the oracle's Philox4x32-10 and the dropout keep mask built on it."""
import os

import numpy as np

from oracle import cnn

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def _philox_bigint(ctr, key):
    """Independent restatement with Python integers (no fixed-width types)."""
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k[0]) & 0xFFFFFFFF, p1 & 0xFFFFFFFF,
             ((p0 >> 32) ^ c[3] ^ k[1]) & 0xFFFFFFFF, p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert list(cnn.philox4x32_10(ctr, key)) == out
        assert _philox_bigint(ctr, key) == out


def test_matches_bigint_on_random_counters():
    rng = np.random.default_rng(11)
    for _ in range(2000):
        ctr = [int(v) for v in rng.integers(0, 2**32, 4, dtype=np.uint64)]
        key = [int(v) for v in rng.integers(0, 2**32, 2, dtype=np.uint64)]
        assert list(cnn.philox4x32_10(ctr, key)) == _philox_bigint(ctr, key)


def test_bijective_on_small_counter_range():
    seen = set()
    for c0 in range(4096):
        seen.add(tuple(cnn.philox4x32_10([c0, 0, 0, 0], [1, 2])))
    assert len(seen) == 4096


def test_keep_mask_matches_definition():
    seed, worker, step, b, p = 0x1234567890ABCDEF, 5, (3 << 32) + 9, 3, 0.25
    keep = cnn.dropout_keep(seed, worker, step, b, p).reshape(-1)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for e in range(b * 512):
        word = _philox_bigint([e // 4, worker, step & 0xFFFFFFFF, step >> 32], key)[e % 4]
        assert keep[e] == (1 if word >= 0x40000000 else 0)


def test_keep_fraction_and_keying():
    b = 4096
    k0 = cnn.dropout_keep(0x5EED, 0, 0, b, 0.25)
    n = k0.size
    sigma = np.sqrt(0.75 * 0.25 / n)
    assert abs(k0.mean() - 0.75) < 4 * sigma
    # worker, step and seed all change the mask; same key reproduces it
    assert (cnn.dropout_keep(0x5EED, 0, 0, b, 0.25) == k0).all()
    for other in (cnn.dropout_keep(0x5EED, 1, 0, b, 0.25), cnn.dropout_keep(0x5EED, 0, 1, b, 0.25),
                  cnn.dropout_keep(0x5EEE, 0, 0, b, 0.25), cnn.dropout_keep(0x5EED, 0, 1 << 32, b, 0.25)):
        assert 0.3 < (other != k0).mean() < 0.45      # two independent 3/4-masks differ w.p. 3/8
    assert cnn.dropout_keep(1, 0, 0, 64, 0.0).all()
    assert abs(cnn.dropout_keep(1, 0, 0, 4096, 0.5).mean() - 0.5) < 0.01
