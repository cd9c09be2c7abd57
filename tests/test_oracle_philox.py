"""Pins for the oracle's random-number generator (Philox4x32-10, SC'11) and its keying."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_known_answer_vectors(oracle):
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        got = oracle.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == out


def test_keying_maps_to_counter_and_key(oracle):
    """random_word(seed, step, worker, e) = word (e mod 4) of the block with
    counter (lo(e/4), hi(e/4), worker, hi(seed)) and key (lo(seed), step)."""
    seed = 0x0123456789ABCDEF
    for e in (0, 1, 2, 3, 4, 7, 1 << 20, (1 << 34) + 5):
        for worker in (0, 3):
            for step in (0, 9):
                q = e >> 2
                blk = oracle.philox4x32_10([q & 0xFFFFFFFF, q >> 32, worker, seed >> 32],
                                           [seed & 0xFFFFFFFF, step])
                assert oracle.random_word(seed, step, worker, e) == int(blk[e & 3])


def test_streams_differ_across_seed_step_worker(oracle):
    base = [oracle.random_word(0, 0, 0, e) for e in range(64)]
    for seed, step, worker in [(1, 0, 0), (0, 1, 0), (0, 0, 1), (1 << 32, 0, 0)]:
        other = [oracle.random_word(seed, step, worker, e) for e in range(64)]
        assert sum(a == b for a, b in zip(base, other)) == 0


def test_uniform_grid_and_range(oracle):
    """uniform12 = 1 + u, u = (low 23 bits) / 2^23: exact, in [1, 2)."""
    assert oracle.uniform12(0) == 1.0
    assert oracle.uniform12(0xFF800000) == 1.0              # high 9 bits are dropped
    assert oracle.uniform12(1) == 1.0 + 2.0 ** -23
    assert oracle.uniform12(0xFFFFFFFF) == 2.0 - 2.0 ** -23
    assert oracle.uniform12(0x00400000) == 1.5
    for w in (0x12345678, 0x9ABCDEF0, 0x007FFFFF):
        assert oracle.uniform12(w) == 1.0 + (w & 0x7FFFFF) / 2.0 ** 23


def test_uniform_moments(oracle):
    n = 20000
    u = np.array([oracle.uniform12(oracle.random_word(7, 3, 1, e)) for e in range(n)]) - 1.0
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 5 * (1 / 12 ** 0.5) / n ** 0.5
    assert abs(u.var() - 1 / 12) < 0.004
    # bits look balanced
    w = np.array([oracle.random_word(7, 3, 1, e) for e in range(4096)], dtype=np.uint64)
    for bit in range(32):
        frac = ((w >> np.uint64(bit)) & np.uint64(1)).mean()
        assert abs(frac - 0.5) < 5 * 0.5 / 4096 ** 0.5


def test_uniform_at_23_bits_is_the_word_uniform(oracle):
    for e in (0, 1, 5, 1023, (1 << 33) + 3):
        assert oracle.uniform12_at(9, 4, 2, e, 23) == oracle.uniform12(oracle.random_word(9, 4, 2, e))


def test_uniform_at_16_bits_keying(oracle):
    """16-bit resolution: one block per eight elements, counter (lo(e/8), hi(e/8), worker, hi(seed)),
    key (lo(seed), step); element e takes word (e/2) mod 4, low half if e is even, high half if
    odd; 1 + half / 2^16.  Checked against the block function, which the known-answer vectors pin."""
    seed = 0x0123456789ABCDEF
    for e in (0, 1, 2, 3, 6, 7, 8, 9, 15, 16, (1 << 20) + 5, (1 << 35) + 6):
        for worker in (0, 3):
            for step in (0, 9):
                q = e >> 3
                blk = oracle.philox4x32_10([q & 0xFFFFFFFF, q >> 32, worker, seed >> 32],
                                           [seed & 0xFFFFFFFF, step])
                w = int(blk[(e >> 1) & 3])
                half = (w >> 16) if (e & 1) else (w & 0xFFFF)
                got = oracle.uniform12_at(seed, step, worker, e, 16)
                assert got == 1.0 + half / 65536.0
                assert 1.0 <= got < 2.0


def test_uniform_at_16_bits_moments(oracle):
    n = 40000
    u = np.array([oracle.uniform12_at(7, 3, 1, e, 16) for e in range(n)]) - 1.0
    assert u.min() >= 0.0 and u.max() < 1.0
    assert np.all(u * 65536 == np.round(u * 65536))          # on the 2^-16 grid
    assert abs(u.mean() - 0.5) < 5 * (1 / 12 ** 0.5) / n ** 0.5
    assert abs(u.var() - 1 / 12) < 0.003
    # neighbours (the two halves of a word, the words of a block) are uncorrelated
    for lag in (1, 2, 8):
        c = np.corrcoef(u[:-lag], u[lag:])[0, 1]
        assert abs(c) < 5 / n ** 0.5
