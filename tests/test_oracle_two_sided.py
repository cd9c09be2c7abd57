"""Pins for the oracle's Step 10 of Algorithm A1 (two-sided quantisation: the server quantizes the
aggregate once more before sending it back, g_hat <- Q(g_hat))."""
import numpy as np
import pytest


def _offs(*sizes):
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)


def _problem(seed, sizes=(7, 300, 1, 64)):
    rng = np.random.RandomState(seed)
    offs = _offs(*sizes)
    sig = np.repeat(10.0 ** rng.uniform(-4, 0, size=len(sizes)), sizes)
    return offs, (rng.randn(int(offs[-1])) * sig).astype(np.float32)


@pytest.mark.parametrize("bits", [1, 2, 4, 8, 16])
def test_is_the_quantizer_of_eq_xi_applied_to_one_vector(oracle, bits, rng_bits):
    """Grid points, signs, norm and the receiver's value, each against a float64 evaluation."""
    offs, g = _problem(bits)
    S = 2 ** bits - 1
    out, sc, level, neg = oracle.requantize(offs, g, bits, 11, 3, stream=4, rng_bits=rng_bits)
    for l in range(len(offs) - 1):
        sl = slice(int(offs[l]), int(offs[l + 1]))
        g64 = g[sl].astype(np.float64)
        nu = np.float32(np.sqrt(np.sum(g64 * g64)))
        assert abs(sc[l] - nu) <= np.spacing(nu)
        x = np.abs(g64) * (S / np.float64(sc[l]))
        fl = np.floor(x)
        lev = level[sl].astype(np.float64)
        near_int = np.abs(x - np.round(x)) < 1e-4 * np.maximum(x, 1.0)      # fp32 product may land on either side
        assert np.all((lev == fl) | (lev == fl + 1) | (near_int & (np.abs(lev - x) <= 1.0 + 1e-3)))
        assert lev.max() <= S
        assert np.array_equal(neg[sl], (g[sl] < 0).astype(np.uint8))
        val = np.float64(sc[l]) * np.where(neg[sl] == 1, -lev, lev) / S
        assert np.all(np.abs(out[sl] - val) <= 2 * np.spacing(np.abs(val).astype(np.float32)) + 1e-45)


def test_reduces_to_the_workers_quantizer_on_the_same_stream(oracle, rng_bits):
    """Q(g_hat) on stream s = what worker s of an (s+1)-worker problem would send for the same vector."""
    offs, g = _problem(5)
    s = 3
    out, sc, level, neg = oracle.requantize(offs, g, 8, 2, 9, stream=s, rng_bits=rng_bits)
    grads = [np.zeros_like(g) for _ in range(s)] + [g]
    nrm = oracle.worker_norms(offs, grads)
    sc_pw = oracle.scales(nrm, oracle.SCALE_PER_WORKER)
    lev_w, neg_w = oracle.quantize(offs, grads, 8, 2, 9, sc_pw, oracle.SCALE_PER_WORKER, rng_bits=rng_bits)
    assert np.array_equal(sc, sc_pw[s])
    assert np.array_equal(level, lev_w[s]) and np.array_equal(neg, neg_w[s])
    # and the receiver's value is the one-worker aggregate of that message
    _, gh = oracle.aggregate(offs, lev_w[s:s + 1], neg_w[s:s + 1], sc, 8)
    assert np.array_equal(out.view(np.uint32), gh.view(np.uint32))


def test_server_stream_differs_from_every_workers(oracle, rng_bits):
    offs, g = _problem(6, sizes=(4000,))
    M = 4
    _, _, lev_srv, _ = oracle.requantize(offs, g, 8, 0, 0, stream=M, rng_bits=rng_bits)
    for i in range(M):
        _, _, lev_i, _ = oracle.requantize(offs, g, 8, 0, 0, stream=i, rng_bits=rng_bits)
        assert (lev_i != lev_srv).mean() > 0.2


def test_unbiased_and_variance_bound(oracle, rng_bits):
    """E[Q(g_hat)] = g_hat and E||Q(g_hat) - g_hat||^2 <= min{n/S^2, sqrt(n)/S} ||g_hat||^2."""
    offs, g = _problem(7, sizes=(500,))
    bits, S, n = 4, 15, 500
    N = 1500
    acc = np.zeros(n)
    err2 = 0.0
    for seed in range(N):
        out, sc, _, _ = oracle.requantize(offs, g, bits, seed, 1, stream=8, rng_bits=rng_bits)
        acc += out
        err2 += float(np.sum((out.astype(np.float64) - g) ** 2))
    nu = float(sc[0])
    assert np.all(np.abs(acc / N - g) <= 5 * (nu / S) * 0.5 / np.sqrt(N) + 1e-7 * nu)
    assert err2 / N <= min(n / S ** 2, np.sqrt(n) / S) * nu * nu


def test_exact_and_zero_cases(oracle, rng_bits):
    offs = _offs(6, 9, 4)
    g = np.zeros(19, dtype=np.float32)
    g[2] = -0.25                      # a lone power of two: x = S exactly, Q(g) = g for every seed
    g[6:15] = [0.5, -0.5, 0.5, 0.5, -0.5, -0.5, 0.5, 0.5, -0.5]   # S^2 equal magnitudes at b = 2: every level is 1
    for seed in range(20):
        out, sc, level, neg = oracle.requantize(offs, g, 2, seed, 0, stream=3, rng_bits=rng_bits)
        assert np.array_equal(out, g)
        assert sc[0] == 0.25 and sc[1] == 1.5 and sc[2] == 0.0
        assert np.all(level[6:15] == 1) and level[2] == 3 and np.all(level[15:] == 0)


def test_scales_in_replace_the_norm(oracle, rng_bits):
    offs, g = _problem(8, sizes=(50, 60))
    sc_in = np.array([3.0, 0.125], dtype=np.float32)
    out, sc, level, neg = oracle.requantize(offs, g, 8, 1, 1, stream=2, rng_bits=rng_bits, scales_in=sc_in)
    assert np.array_equal(sc, sc_in)
    val = np.repeat(sc_in.astype(np.float64), [50, 60]) * np.where(neg == 1, -1.0, 1.0) * level / 255.0
    assert np.allclose(out, val, rtol=3e-7, atol=0)
