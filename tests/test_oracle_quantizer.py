"""Pins for the oracle's randomized quantizer (Eq. rand_q, Eq. xi) and the message format."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quantizer_hand_case.txt")


def _offs(*sizes):
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)


def _norms_scales(oracle, offs, grads, mode=0):
    nrm = oracle.worker_norms(offs, grads)
    return nrm, oracle.scales(nrm, mode)


def test_worker_norms_match_float64_norm(oracle):
    rng = np.random.RandomState(0)
    offs = _offs(5, 1000, 33, 1)
    grads = [(rng.randn(offs[-1]) * 10.0 ** rng.uniform(-5, 1)).astype(np.float32) for _ in range(3)]
    nrm = oracle.worker_norms(offs, grads)
    for i in range(3):
        for l in range(4):
            ref = np.float32(np.sqrt(np.sum(grads[i][offs[l]:offs[l + 1]].astype(np.float64) ** 2)))
            assert abs(nrm[i, l] - ref) <= np.spacing(ref)
    sc = oracle.scales(nrm, oracle.SCALE_SHARED_MAX)
    assert np.array_equal(sc, nrm.max(axis=0))
    assert np.array_equal(oracle.scales(nrm, oracle.SCALE_PER_WORKER), nrm)


def test_hand_case_b2(oracle, rng_bits):
    rows = [list(map(float, l.split())) for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    g = np.array([r[0] for r in rows], dtype=np.float32)
    offs = _offs(len(g))
    nrm, sc = _norms_scales(oracle, offs, [g])
    assert sc[0] == np.float32(rows[0][1])
    ups = np.zeros(len(g))
    n_seeds = 4000
    acc = np.zeros(len(g))
    for seed in range(n_seeds):
        level, neg = oracle.quantize(offs, [g], 2, seed, 0, sc, rng_bits=rng_bits)
        for k, r in enumerate(rows):
            fl = int(r[3])
            assert level[0, k] in ((fl, fl + 1) if r[4] > 0 else (fl,))
            assert neg[0, k] == int(r[5])
            ups[k] += level[0, k] == fl + 1
        acc += np.where(neg[0] == 1, -1.0, 1.0) * level[0] * (5.0 / 3.0)
    for k, r in enumerate(rows):
        p = r[4]
        assert abs(ups[k] / n_seeds - p) <= 5 * np.sqrt(max(p * (1 - p), 1e-12) / n_seeds) + 1e-6
    # E[Q(g)] = g
    assert np.allclose(acc / n_seeds, g, atol=5 * (5.0 / 3.0) * 0.5 / np.sqrt(n_seeds))


@pytest.mark.parametrize("bits", [1, 2, 4, 8, 16])
def test_level_is_a_neighbouring_grid_point(oracle, bits, rng_bits):
    """xi takes one of the two grid points around |g|/||g|| (Eq. xi); levels fit in b bits."""
    rng = np.random.RandomState(bits)
    offs = _offs(257, 64, 1023)
    grads = [(rng.standard_t(3, offs[-1]) * 0.01).astype(np.float32) for _ in range(2)]
    nrm, sc = _norms_scales(oracle, offs, grads)
    level, neg = oracle.quantize(offs, grads, bits, 11, 5, sc, rng_bits=rng_bits)
    S = 2 ** bits - 1
    assert level.max() <= S
    for i in range(2):
        for l in range(3):
            sl = slice(offs[l], offs[l + 1])
            x = np.abs(grads[i][sl].astype(np.float64)) * S / np.float64(sc[l])
            fl = np.floor(x)
            lv = level[i, sl].astype(np.float64)
            tol = 1e-6 * max(S, 1)              # fp32 evaluation of x near an integer
            ok = (lv == fl) | (lv == fl + 1) | ((np.abs(x - np.round(x)) < tol) & (np.abs(lv - np.round(x)) <= 1))
            assert ok.all()
            assert np.array_equal(neg[i, sl], (grads[i][sl] < 0).astype(np.uint8))


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_exact_cases(oracle, bits, rng_bits):
    S = 2 ** bits - 1
    # (a) one non-zero element, a power of two: x = S exactly, Q(g) = g for every seed
    g = np.zeros(37, dtype=np.float32)
    g[5] = -0.125
    offs = _offs(37)
    nrm, sc = _norms_scales(oracle, offs, [g])
    assert sc[0] == np.float32(0.125)
    for seed in range(20):
        level, neg = oracle.quantize(offs, [g], bits, seed, 0, sc, rng_bits=rng_bits)
        assert level[0, 5] == S and neg[0, 5] == 1 and level[0].sum() == S
    # (b) S^2 elements all +-c, c a power of two: ||g|| = S*c, x = 1 exactly, every level is 1
    n = S * S
    rng = np.random.RandomState(1)
    g = (0.25 * rng.choice([-1.0, 1.0], size=n)).astype(np.float32)
    offs = _offs(n)
    nrm, sc = _norms_scales(oracle, offs, [g])
    assert sc[0] == np.float32(S * 0.25)
    for seed in range(3):
        level, neg = oracle.quantize(offs, [g], bits, seed, 1, sc, rng_bits=rng_bits)
        assert (level[0] == 1).all()
        q = np.where(neg[0] == 1, -1.0, 1.0) * level[0] * (float(sc[0]) / S)
        assert np.array_equal(q.astype(np.float32), g)


def test_unbiased_and_variance_bound(oracle, rng_bits):
    """E[Q(g)] = g and E||Q(g)-g||^2 <= min{n/S^2, sqrt(n)/S} ||g||^2 (QSGD Lemma 3.1, cited
    under assumption A4), by Monte Carlo over seeds."""
    rng = np.random.RandomState(3)
    n, bits, n_seeds = 1000, 4, 2048
    S = 2 ** bits - 1
    g = (rng.randn(n) * 0.03).astype(np.float32)
    offs = _offs(n)
    nrm, sc = _norms_scales(oracle, offs, [g])
    nu = float(sc[0])
    mean = np.zeros(n)
    err2 = 0.0
    for seed in range(n_seeds):
        level, neg = oracle.quantize(offs, [g], bits, seed, 0, sc, rng_bits=rng_bits)
        q = np.where(neg[0] == 1, -1.0, 1.0) * level[0] * (nu / S)
        mean += q
        err2 += np.sum((q - g) ** 2)
    mean /= n_seeds
    err2 /= n_seeds
    # each coordinate: a two-point variable with spacing nu/S => std <= (nu/S)/2
    assert np.max(np.abs(mean - g)) <= 5.5 * (nu / S) / 2 / np.sqrt(n_seeds)
    assert err2 <= min(n / S ** 2, np.sqrt(n) / S) * nu ** 2
    # and the variance is not degenerate (the quantizer is actually random)
    assert err2 > 0.01 * min(n / S ** 2, np.sqrt(n) / S) * nu ** 2


def test_up_probability_is_fraction(oracle, rng_bits):
    """P(level = floor(x)+1) = x - floor(x) for a fixed x, across element positions."""
    n, bits = 40000, 8
    S = 255
    g = np.full(n, 0.3, dtype=np.float32)
    g[0] = 64.0                                   # dominates the norm
    offs = _offs(n)
    nrm, sc = _norms_scales(oracle, offs, [g])
    x = 0.3 * S / float(sc[0])
    level, _ = oracle.quantize(offs, [g], bits, 5, 2, sc, rng_bits=rng_bits)
    p = (level[0, 1:] == np.floor(x) + 1).mean()
    frac = x - np.floor(x)
    assert abs(p - frac) < 5 * np.sqrt(frac * (1 - frac) / n)


def test_scale_invariance_power_of_two(oracle, rng_bits):
    rng = np.random.RandomState(4)
    offs = _offs(100, 333)
    grads = [(rng.randn(offs[-1]) * 1e-3).astype(np.float32) for _ in range(3)]
    nrm, sc = _norms_scales(oracle, offs, grads)
    l1, n1 = oracle.quantize(offs, grads, 8, 1, 1, sc, rng_bits=rng_bits)
    grads2 = [g * np.float32(2.0 ** 7) for g in grads]
    nrm2, sc2 = _norms_scales(oracle, offs, grads2)
    assert np.array_equal(sc2, sc * np.float32(128.0))
    l2, n2 = oracle.quantize(offs, grads2, 8, 1, 1, sc2, rng_bits=rng_bits)
    assert np.array_equal(l1, l2) and np.array_equal(n1, n2)


def test_zero_norm_layer_gives_zero_levels(oracle, rng_bits):
    offs = _offs(10, 20)
    g = np.zeros(30, dtype=np.float32)
    g[10:] = 1.0
    nrm, sc = _norms_scales(oracle, offs, [g])
    assert sc[0] == 0.0
    level, neg = oracle.quantize(offs, [g], 8, 0, 0, sc, rng_bits=rng_bits)
    assert (level[0, :10] == 0).all() and (neg == 0).all()


def test_random_stream_independent_of_layer_partition(oracle, rng_bits):
    rng = np.random.RandomState(5)
    g = rng.randn(64).astype(np.float32)
    a = oracle.quantize(_offs(64), [g], 8, 3, 3, np.array([10.0], np.float32), rng_bits=rng_bits)
    b = oracle.quantize(_offs(10, 54), [g], 8, 3, 3, np.array([10.0, 10.0], np.float32), rng_bits=rng_bits)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("bits", [1, 2, 4, 8, 16])
def test_bit_budget_and_pack_roundtrip(oracle, bits):
    """Message size: 32 bits per norm + d sign bits + b*d level bits ("(32 + d + b d) bits"),
    up to 16-byte padding; planes agree with numpy's little-endian bit packing."""
    rng = np.random.RandomState(bits)
    d = 1003
    level = rng.randint(0, 2 ** bits, size=d).astype(np.uint32)
    neg = rng.randint(0, 2, size=d).astype(np.uint8)
    lp, sp = oracle.pack(level, neg, bits)
    assert 0 <= lp.size * 8 - bits * d < 128 + 8 and lp.size % 16 == 0
    assert 0 <= sp.size * 8 - d < 128 + 8 and sp.size % 16 == 0
    ref_sign = np.packbits(neg, bitorder="little")
    assert np.array_equal(sp[:ref_sign.size], ref_sign) and not sp[ref_sign.size:].any()
    bitmat = ((level[:, None] >> np.arange(bits, dtype=np.uint32)[None, :]) & 1).astype(np.uint8)
    ref_level = np.packbits(bitmat.reshape(-1), bitorder="little")
    assert np.array_equal(lp[:ref_level.size], ref_level) and not lp[ref_level.size:].any()
    l2, n2 = oracle.unpack(lp, sp, d, bits)
    assert np.array_equal(l2, level) and np.array_equal(n2, neg)
