"""Pins for the oracle's counter-based Rademacher generator (CPU only)."""
import os

import numpy as np

from oracle import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert orc.philox4x32_10(v[0:4], v[4:6]) == tuple(v[6:10])


def _philox_py(ctr, key):
    # independent restatement of the published round function, in Python integers
    c, k = list(ctr), list(key)
    for _ in range(10):
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_bit_to_element_mapping():
    # element i of block b: row r=(i%4096)//128, slot=(i//4)%32, comp=i%4 -> bit 4*row+comp of
    # Philox(counter=(32*b+slot, t, p), key=seed)
    rng = np.random.default_rng(5)
    for _ in range(300):
        seed = int(rng.integers(0, 2 ** 63))
        t = int(rng.integers(0, 2 ** 32))
        p = int(rng.integers(0, 8))
        i = int(rng.integers(0, 2 ** 40))
        b, r = divmod(i, 4096)
        row, slot, comp = r // 128, (r // 4) % 32, r % 4
        q = 32 * b + slot
        out = _philox_py([q & 0xFFFFFFFF, q >> 32, t, p], [seed & 0xFFFFFFFF, seed >> 32])
        bit = 4 * row + comp
        assert orc.rademacher_bit(seed, t, p, i) == (out[bit // 32] >> (bit % 32)) & 1


def test_probe_matches_single_bits_and_is_pm_one():
    z = orc.probe(7, 3, 1, 4000, 9000)
    assert set(np.unique(z)) == {-1.0, 1.0}
    for j in [0, 1, 95, 96, 97, 4095, 4096, 8999]:
        assert z[j] == (-1.0 if orc.rademacher_bit(7, 3, 1, 4000 + j) else 1.0)
    # a window of the same stream does not depend on where the window starts
    assert np.array_equal(orc.probe(7, 3, 1, 5000, 100), z[1000:1100])


def test_balance_and_decorrelation():
    n = 1 << 18
    base = orc.probe(0, 1, 0, 0, n)
    assert abs(base.sum()) <= 4 * np.sqrt(n)
    # per "segment" balance on ragged windows
    for off, m in [(0, 1000), (37, 4096), (5000, 33333), (100001, 65536)]:
        assert abs(base[off:off + m].sum()) <= 4 * np.sqrt(m)
    others = {
        "probe": orc.probe(0, 1, 1, 0, n),
        "step": orc.probe(0, 2, 0, 0, n),
        "seed": orc.probe(1, 1, 0, 0, n),
        "shifted": orc.probe(0, 1, 0, 4096, n),
    }
    for name, z in others.items():
        assert abs(float((base * z).mean())) <= 4 / np.sqrt(n), name
    # neighbouring indices: lags that stay in a row, cross rows, cross the 4096 block
    for lag in [1, 2, 3, 4, 5, 31, 32, 127, 128, 129, 4095, 4096]:
        c = float((base[:-lag] * base[lag:]).mean())
        assert abs(c) <= 4 / np.sqrt(n - lag), lag
