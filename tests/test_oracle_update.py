"""Pins for the oracle's aggregation (Eq. grad_agg), LALR update (Eq. 3) and the whole step."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "lalr_hand_cases.txt")


def _offs(*sizes):
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)


def _problem(rng, sizes, M, sigma=1e-2):
    offs = _offs(*sizes)
    d = int(offs[-1])
    grads = [(rng.randn(d) * sigma).astype(np.float32) for _ in range(M)]
    theta = (rng.randn(d) * 0.05).astype(np.float32)
    mom = (rng.randn(d) * 1e-3).astype(np.float32)
    return offs, grads, theta, mom


# ------------------------------------------------------------------ aggregation

def test_aggregate_is_mean_of_dequantized_messages(oracle, rng_bits):
    """g_hat = (1/M) sum_i ||g||*sign*level/S, evaluated independently in float64."""
    rng = np.random.RandomState(0)
    offs, grads, _, _ = _problem(rng, [100, 7, 300], 5)
    bits, S, M = 4, 15, 5
    nrm = oracle.worker_norms(offs, grads)
    for mode in (oracle.SCALE_SHARED_MAX, oracle.SCALE_PER_WORKER):
        sc = oracle.scales(nrm, mode)
        level, neg = oracle.quantize(offs, grads, bits, 2, 0, sc, mode, rng_bits=rng_bits)
        code_sum, g_hat = oracle.aggregate(offs, level, neg, sc, bits, mode)
        signed = np.where(neg == 1, -1.0, 1.0) * level.astype(np.float64)
        ref = np.zeros(offs[-1])
        for l in range(3):
            sl = slice(offs[l], offs[l + 1])
            for i in range(M):
                nu = float(sc[i, l]) if mode == oracle.SCALE_PER_WORKER else float(sc[l])
                ref[sl] += nu * signed[i, sl] / S
        ref /= M
        # fp32 accumulation of M terms of size <= nu: absolute error ~ M * 2^-24 * nu
        assert np.allclose(g_hat, ref, rtol=2e-6, atol=M * 6e-8 * float(sc.max()))
        if mode == oracle.SCALE_SHARED_MAX:
            assert np.array_equal(code_sum, signed.sum(axis=0).astype(np.int32))
            assert np.abs(code_sum).max() <= M * S
        else:
            assert code_sum is None


def test_per_worker_formula_with_equal_scales_matches_shared(oracle, rng_bits):
    rng = np.random.RandomState(1)
    offs, grads, _, _ = _problem(rng, [64, 200], 4)
    nrm = oracle.worker_norms(offs, grads)
    sc = oracle.scales(nrm, oracle.SCALE_SHARED_MAX)
    level, neg = oracle.quantize(offs, grads, 8, 0, 0, sc, rng_bits=rng_bits)
    _, g_shared = oracle.aggregate(offs, level, neg, sc, 8)
    sc_pw = np.tile(sc, (4, 1))
    _, g_pw = oracle.aggregate(offs, level, neg, sc_pw, 8, oracle.SCALE_PER_WORKER)
    assert np.allclose(g_shared, g_pw, rtol=1e-6, atol=4 * 6e-8 * float(sc.max()))


def test_m1_aggregate_is_the_signed_code(oracle, rng_bits):
    rng = np.random.RandomState(2)
    offs, grads, _, _ = _problem(rng, [50, 50], 1)
    nrm = oracle.worker_norms(offs, grads)
    sc = oracle.scales(nrm)
    level, neg = oracle.quantize(offs, grads, 8, 0, 0, sc, rng_bits=rng_bits)
    code_sum, g_hat = oracle.aggregate(offs, level, neg, sc, 8)
    assert np.array_equal(code_sum, np.where(neg[0] == 1, -1, 1) * level[0].astype(np.int64))


def test_bits32_is_exact_worker_average(oracle):
    rng = np.random.RandomState(3)
    offs, grads, _, _ = _problem(rng, [33, 1000], 8)
    g_hat = oracle.average(offs, grads)
    ref = np.mean(np.stack(grads).astype(np.float64), axis=0)
    gmax = max(float(np.abs(g).max()) for g in grads)
    assert np.allclose(g_hat, ref, rtol=1e-6, atol=8 * 6e-8 * gmax)
    # integers: every partial sum and the division by M = 8 are exact
    ints = [rng.randint(-1000, 1000, size=offs[-1]).astype(np.float32) for _ in range(8)]
    assert np.array_equal(oracle.average(offs, ints), np.mean(np.stack(ints).astype(np.float64), axis=0))
    # M = 1: identity
    assert np.array_equal(oracle.average(offs, grads[:1]), grads[0])


# ------------------------------------------------------------------ LALR

def _cases():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = [np.array(p.split(), dtype=np.float64) for p in line.split("|")]
        out.append(parts)
    return out


def test_lalr_hand_cases(oracle):
    cases = _cases()
    assert len(cases) == 6
    for theta, m, g, hp, theta_new, m_new in cases:
        offs = _offs(len(theta))
        th, mo, norms = oracle.lalr(offs, theta.astype(np.float32), m.astype(np.float32), g.astype(np.float32),
                                    float(hp[0]), float(hp[1]), float(hp[2]), 0.0, 10.0)
        assert np.allclose(th, theta_new, rtol=1e-6, atol=1e-7), (theta, th, theta_new)
        assert np.allclose(mo, m_new, rtol=1e-6, atol=1e-7)
        assert np.isclose(norms[0, 0], np.linalg.norm(theta))
        assert np.isclose(norms[0, 1], np.linalg.norm(m_new))


def test_lalr_step_length_invariant(oracle):
    """||theta' - theta||_2 = eta * min{max{||theta||, c_l}, c_u} whenever ||u|| != 0,
    whatever the gradient magnitude (direct consequence of Eq. 3)."""
    rng = np.random.RandomState(4)
    sizes = [10, 500, 3, 2000]
    offs = _offs(*sizes)
    d = offs[-1]
    theta = rng.randn(d).astype(np.float32)
    theta[offs[1]:offs[2]] *= 3.0                        # ||theta_1|| ~ 67 > c_u
    mom = (rng.randn(d) * 0.1).astype(np.float32)
    for gscale in (1e-6, 1.0, 1e4):
        g = (rng.randn(d) * gscale).astype(np.float32)
        for c_l, c_u in ((0.0, 10.0), (5.0, 10.0)):
            th, mo, norms = oracle.lalr(offs, theta, mom, g, 0.05, 0.9, 1e-4, c_l, c_u)
            for l in range(4):
                sl = slice(offs[l], offs[l + 1])
                step = np.linalg.norm(th[sl].astype(np.float64) - theta[sl])
                tau = min(max(np.linalg.norm(theta[sl].astype(np.float64)), c_l), c_u)
                assert np.isclose(step, 0.05 * tau, rtol=2e-5)
                # direction is -u
                u = mo[sl].astype(np.float64)
                assert np.allclose((theta[sl] - th[sl]) / step, u / np.linalg.norm(u), atol=2e-4)


def test_lalr_matches_float64_formula(oracle):
    rng = np.random.RandomState(5)
    offs, grads, theta, mom = _problem(rng, [77, 1234, 5], 1)
    g = grads[0]
    lr, mu, wd = 0.1, 0.9, 5e-4
    th, mo, norms = oracle.lalr(offs, theta, mom, g, lr, mu, wd)
    for l in range(3):
        sl = slice(offs[l], offs[l + 1])
        t64, m64, g64 = (a[sl].astype(np.float64) for a in (theta, mom, g))
        u = mu * m64 + g64 + wd * t64
        ref = t64 - min(max(np.linalg.norm(t64), 0.0), 10.0) * lr / np.linalg.norm(u) * u
        assert np.allclose(mo[sl], u, rtol=1e-6, atol=1e-9)
        assert np.allclose(th[sl], ref, rtol=1e-6, atol=1e-8)


def test_zero_norm_conventions(oracle):
    offs = _offs(4, 4, 4)
    theta = np.array([0, 0, 0, 0, 1, 2, 3, 4, 1, 1, 1, 1], dtype=np.float32)
    mom = np.array([1, -1, 2, 0, 0, 0, 0, 0, 0.5, 0.5, 0.5, 0.5], dtype=np.float32)
    g = np.array([1, 1, 1, 1, 0, 0, 0, 0, 0, 0, 0, 0], dtype=np.float32)
    th, mo, norms = oracle.lalr(offs, theta, mom, g, 0.1, 0.5, 0.0)
    # layer 0: all-zero parameters, c_l = 0: do not move; momentum updates
    assert np.array_equal(th[:4], np.zeros(4)) and np.allclose(mo[:4], 0.5 * mom[:4] + g[:4])
    # layer 1: u = 0 (no momentum, no gradient, no decay): unchanged, no NaN
    assert np.array_equal(th[4:8], theta[4:8]) and np.array_equal(mo[4:8], np.zeros(4))
    # layer 2: zero gradient: u = mu*m
    assert np.allclose(mo[8:], 0.25) and np.isfinite(th).all()
    # with c_l > 0 the zero tensor does move, by exactly eta*c_l
    th2, _, _ = oracle.lalr(offs, theta, mom, g, 0.1, 0.5, 0.0, 2.0, 10.0)
    assert np.isclose(np.linalg.norm(th2[:4]), 0.1 * 2.0, rtol=1e-5)


# ------------------------------------------------------------------ whole step

def test_step_equals_composition(oracle, rng_bits):
    rng = np.random.RandomState(6)
    offs, grads, theta, mom = _problem(rng, [40, 1000, 9, 513], 3)
    hp = dict(lr=0.1, momentum=0.9, weight_decay=5e-4)
    for mode in (oracle.SCALE_SHARED_MAX, oracle.SCALE_PER_WORKER):
        out = oracle.step(offs, theta, mom, grads, 8, 42, 7, scale_mode=mode, **hp, rng_bits=rng_bits)
        nrm = oracle.worker_norms(offs, grads)
        sc = oracle.scales(nrm, mode)
        level, neg = oracle.quantize(offs, grads, 8, 42, 7, sc, mode, rng_bits=rng_bits)
        cs, g_hat = oracle.aggregate(offs, level, neg, sc, 8, mode)
        th, mo, norms = oracle.lalr(offs, theta, mom, g_hat, hp["lr"], hp["momentum"], hp["weight_decay"])
        assert np.array_equal(out["theta"], th) and np.array_equal(out["mom"], mo)
        assert np.array_equal(out["layer_norms"], norms)
        assert np.array_equal(out["scales"], sc.reshape(-1))
        if mode == oracle.SCALE_SHARED_MAX:
            assert np.array_equal(out["code_sum"], cs)


def test_step_window_equals_full(oracle, rng_bits):
    rng = np.random.RandomState(7)
    offs, grads, theta, mom = _problem(rng, [40, 1000, 9, 513], 2)
    hp = dict(lr=0.1, momentum=0.9, weight_decay=5e-4)
    full = oracle.step(offs, theta, mom, grads, 4, 1, 2, **hp, rng_bits=rng_bits)
    a, b = int(offs[1]), int(offs[3])
    win = oracle.step(offs, theta[a:b].copy(), mom[a:b].copy(), [g[a:b].copy() for g in grads], 4, 1, 2,
                      l0=1, l1=3, window=True, **hp, rng_bits=rng_bits)
    assert np.array_equal(win["theta"], full["theta"][a:b])
    assert np.array_equal(win["mom"], full["mom"][a:b])
    assert np.array_equal(win["code_sum"], full["code_sum"][a:b])


def test_m1_b32_step_is_plain_lalr(oracle, rng_bits):
    """M = 1 reduces DAT to AT (Sec. 3); with b = 32 nothing is quantized."""
    rng = np.random.RandomState(8)
    offs, grads, theta, mom = _problem(rng, [100, 50], 1)
    out = oracle.step(offs, theta, mom, grads, 32, 0, 0, 0.1, 0.9, 1e-4, rng_bits=rng_bits)
    th, mo, _ = oracle.lalr(offs, theta, mom, grads[0], 0.1, 0.9, 1e-4)
    assert np.array_equal(out["theta"], th) and np.array_equal(out["mom"], mo)


def test_step_with_many_bits_approaches_unquantized_step(oracle, rng_bits):
    """As b grows Q -> identity: the 16-bit step is close to the 32-bit (exact average) step."""
    rng = np.random.RandomState(9)
    offs, grads, theta, mom = _problem(rng, [300, 700], 4)
    hp = dict(lr=0.1, momentum=0.9, weight_decay=5e-4)
    exact = oracle.step(offs, theta, mom, grads, 32, 0, 0, **hp, rng_bits=rng_bits)
    q16 = oracle.step(offs, theta, mom, grads, 16, 0, 0, **hp, rng_bits=rng_bits)
    q2 = oracle.step(offs, theta, mom, grads, 2, 0, 0, **hp, rng_bits=rng_bits)
    e16 = np.abs(q16["mom"] - exact["mom"]).max()
    e2 = np.abs(q2["mom"] - exact["mom"]).max()
    nu = oracle.scales(oracle.worker_norms(offs, grads)).max()
    assert e16 <= nu / 65535 + 1e-9 and e2 > 50 * e16


def test_resume_is_exact(oracle, rng_bits):
    """The random stream is a pure function of (seed, step, worker, element): 4 straight
    steps equal 2 steps + copy of (theta, m) + 2 steps, bit for bit."""
    rng = np.random.RandomState(10)
    offs, _, theta, mom = _problem(rng, [64, 640], 2)
    gs = [[(rng.randn(offs[-1]) * 0.01).astype(np.float32) for _ in range(2)] for _ in range(4)]
    hp = dict(lr=0.05, momentum=0.9, weight_decay=1e-4)
    th, mo = theta, mom
    for t in range(4):
        o = oracle.step(offs, th, mo, gs[t], 8, 5, t, **hp, rng_bits=rng_bits)
        th, mo = o["theta"], o["mom"]
    th2, mo2 = theta, mom
    for t in range(2):
        o = oracle.step(offs, th2, mo2, gs[t], 8, 5, t, **hp, rng_bits=rng_bits)
        th2, mo2 = o["theta"], o["mom"]
    th2, mo2 = th2.copy(), mo2.copy()
    for t in range(2, 4):
        o = oracle.step(offs, th2, mo2, gs[t], 8, 5, t, **hp, rng_bits=rng_bits)
        th2, mo2 = o["theta"], o["mom"]
    assert np.array_equal(th, th2) and np.array_equal(mo, mo2)
    # and the step index matters
    o_same = oracle.step(offs, theta, mom, gs[0], 8, 5, 0, **hp, rng_bits=rng_bits)
    o_other = oracle.step(offs, theta, mom, gs[0], 8, 5, 1, **hp, rng_bits=rng_bits)
    assert not np.array_equal(o_same["code_sum"], o_other["code_sum"])


def test_tiny_mlp_config_runs(oracle, rng_bits):
    from paper_2206_06257_b200 import synth
    cfg = synth.config("tiny_mlp")
    theta, mom = synth.make_params(cfg)
    grads = synth.make_grads(cfg, 0)
    out = oracle.step(cfg.offsets, theta.numpy(), mom.numpy(), [g.numpy() for g in grads], cfg.bits, 0, 0,
                      cfg.lr, cfg.momentum, cfg.weight_decay, cfg.c_l, cfg.c_u, rng_bits=rng_bits)
    assert np.isfinite(out["theta"]).all() and np.abs(out["code_sum"]).max() <= cfg.M * 255
    for l in range(cfg.h):
        sl = slice(cfg.offsets[l], cfg.offsets[l + 1])
        step = np.linalg.norm(out["theta"][sl].astype(np.float64) - theta.numpy()[sl])
        tau = min(np.linalg.norm(theta.numpy()[sl].astype(np.float64)), cfg.c_u)
        assert np.isclose(step, cfg.lr * tau, rtol=2e-5)
