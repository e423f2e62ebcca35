"""Pins of the oracle's Philox4x32-10 and of the uniforms derived from it."""
import os

import numpy as np

from oracle import oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))


def _kat():
    rows = []
    with open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(x, 16) for x in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def py_philox(key, ctr):
    """Second implementation, straight from the published round function, in Python integers."""
    M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
    c = list(ctr)
    k = list(key)
    mask = 0xFFFFFFFF
    for _ in range(10):
        hi0, lo0 = divmod(M0 * c[0], 1 << 32)
        hi1, lo1 = divmod(M1 * c[2], 1 << 32)
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + W0) & mask, (k[1] + W1) & mask]
    return tuple(c)


def test_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert list(O.philox(key, ctr)) == out
        assert list(py_philox(key, ctr)) == out


def test_two_implementations_agree():
    rng = np.random.default_rng(7)
    for _ in range(20000):
        key = [int(x) for x in rng.integers(0, 2**32, 2)]
        ctr = [int(x) for x in rng.integers(0, 2**32, 4)]
        assert O.philox(key, ctr) == py_philox(key, ctr)


def test_uniform_keying():
    # key = seed halves, counter = (ctx lo, ctx hi, position, 0); word 0 >> 8 and word 1
    seed, ctx, pos = 0x1234567890ABCDEF, 0xFEDCBA9876543210, 77
    w = py_philox((seed & 0xFFFFFFFF, seed >> 32), (ctx & 0xFFFFFFFF, ctx >> 32, pos, 0))
    assert O.uniforms(seed, ctx, pos) == (w[0] >> 8, w[1])


def test_uniformity():
    n = 200000
    ua = np.empty(n)
    us = np.empty(n)
    for i in range(n):
        a, s = O.uniforms(5, i % 1000, i // 1000)
        ua[i], us[i] = a / 2**24, s / 2**32
    for u in (ua, us):
        assert abs(u.mean() - 0.5) < 4 * (1 / 12 / n) ** 0.5
        assert abs(u.var() - 1 / 12) < 1e-3
        # Kolmogorov-Smirnov against U(0,1), alpha ~ 1e-3
        s = np.sort(u)
        d = max(np.max(np.arange(1, n + 1) / n - s), np.max(s - np.arange(n) / n))
        assert d < 1.95 / n ** 0.5
    assert abs(np.corrcoef(ua, us)[0, 1]) < 0.01
    assert ua.max() < 1.0 and us.max() < 1.0
