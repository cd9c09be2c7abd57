"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bit-exact: packed level and sign planes, integer code sums, g_hat and m' (given equal scales).
Scales: within 1 fp32 ulp of the oracle's (both accumulate exact squares in fp64; only the
summation order differs); the oracle is then given the GPU's scale bits so that everything
downstream is comparable bit for bit.  theta', m' end to end: 1e-5 relative.
"""
import numpy as np
import pytest
import torch

from helpers import (REL_TOL, GpuPlan, assert_close_per_layer, hp_tuple, np_of, oracle_planes, to_dev,
                     ulp_diff)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    assert torch.cuda.is_available()
    from paper_2206_06257_b200 import api as _api
    return _api


def _offs(sizes):
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)


def _random_problem(seed, sizes, M, sigma_lo=-5, sigma_hi=-1, dist="normal"):
    rng = np.random.RandomState(seed)
    offs = _offs(sizes)
    d = int(offs[-1])
    sig = np.repeat(10.0 ** rng.uniform(sigma_lo, sigma_hi, size=len(sizes)), sizes)
    grads = []
    for _ in range(M):
        z = rng.standard_t(3, d) if dist == "t3" else rng.randn(d)
        grads.append((z * sig).astype(np.float32))
    theta = (rng.randn(d) * 0.05).astype(np.float32)
    mom = (rng.randn(d) * 1e-3).astype(np.float32)
    return offs, grads, theta, mom


def _check_unfused(api, oracle, offs, grads, theta, mom, bits, hp, seed=3, step=5, rng_bits=16):
    M = len(grads)
    d = int(offs[-1])
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, M, bits, rng_bits) as P:
        lv, sg, sc = P.alloc_message()
        api.dat_quantize(P.plan, g_dev, seed, step, lv, sg, sc)
        torch.cuda.synchronize()
        sc_gpu = np_of(sc)
        # S1: scales within 1 ulp
        sc_ref = oracle.scales(oracle.worker_norms(offs, grads))
        assert ulp_diff(sc_gpu, sc_ref).max() <= 1
        n_scale_mismatch = int((sc_gpu != sc_ref).sum())
        # S2+S3: planes bit-exact given the GPU's scales
        level, neg = oracle.quantize(offs, grads, bits, seed, step, sc_gpu, rng_bits=rng_bits)
        lp_ref, sp_ref = oracle_planes(oracle, level, neg, bits)
        assert np.array_equal(np_of(lv).reshape(M, -1), lp_ref)
        assert np.array_equal(np_of(sg).reshape(M, -1), sp_ref)
        # S4+S5
        cs = torch.full((d + 8,), 12345, dtype=torch.int32, device="cuda")[:d]
        gh = torch.zeros(d, dtype=torch.float32, device="cuda")
        api.dat_aggregate(P.plan, lv, sg, sc, cs, gh)
        cs_ref, gh_ref = oracle.aggregate(offs, level, neg, sc_gpu, bits)
        assert np.array_equal(np_of(cs), cs_ref)
        assert np.array_equal(np_of(gh).view(np.uint32), gh_ref.view(np.uint32))
        # S6-S8
        th_d, mo_d = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        norms = torch.zeros(2 * P.h, dtype=torch.float32, device="cuda")
        api.dat_lalr_step(P.plan, th_d, mo_d, gh, hp, norms)
        th_ref, mo_ref, norms_ref = oracle.lalr(offs, theta, mom, gh_ref, *hp)
        assert np.array_equal(np_of(mo_d).view(np.uint32), mo_ref.view(np.uint32))
        assert ulp_diff(np_of(norms).reshape(-1, 2), norms_ref).max() <= 1
        assert_close_per_layer(np_of(th_d), th_ref, offs, "theta (unfused)")
        assert P.status() == 0
        return n_scale_mismatch


def _check_fused(api, oracle, offs, grads, theta, mom, bits, hp, seed=3, step=5, rng_bits=16, entry="dat_step"):
    M = len(grads)
    dat_step = getattr(api, entry)
    d = int(offs[-1])
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, M, bits, rng_bits) as P:
        th_d, mo_d = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        cs = torch.full((d,), 777, dtype=torch.int32, device="cuda")
        norms = torch.zeros(2 * P.h, dtype=torch.float32, device="cuda")
        sc = torch.zeros(P.h, dtype=torch.float32, device="cuda")
        dat_step(P.plan, th_d, mo_d, g_dev, seed, step, hp, cs, norms, sc)
        torch.cuda.synchronize()
        assert P.status() == 0
        ref = oracle.step(offs, theta, mom, grads, bits, seed, step, *hp, rng_bits=rng_bits)
        if bits != 32:
            sc_gpu = np_of(sc)
            assert ulp_diff(sc_gpu, ref["scales"]).max() <= 1
            if not np.array_equal(sc_gpu, ref["scales"]):        # conditional protocol: same scale bits
                ref = oracle.step(offs, theta, mom, grads, bits, seed, step, *hp, scales_in=sc_gpu, rng_bits=rng_bits)
            assert np.array_equal(np_of(cs), ref["code_sum"])
        assert np.array_equal(np_of(mo_d).view(np.uint32), ref["mom"].view(np.uint32))
        assert ulp_diff(np_of(norms).reshape(-1, 2), ref["layer_norms"]).max() <= 1
        assert_close_per_layer(np_of(th_d), ref["theta"], offs, "theta (fused)")
        assert_close_per_layer(np_of(mo_d), ref["mom"], offs, "mom (fused)")
        # a second call on fresh copies gives bit-identical results (run-to-run determinism)
        th2, mo2 = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        dat_step(P.plan, th2, mo2, g_dev, seed, step, hp)
        torch.cuda.synchronize()
        assert torch.equal(th2, th_d) and torch.equal(mo2, mo_d)
        return np_of(th_d), np_of(mo_d)


HP = (0.1, 0.9, 5e-4, 0.0, 10.0)

# several tiles + ragged tails + tiny and odd-sized layers (offsets not multiples of 4)
SIZES_RAGGED = [1, 2, 3, 5, 31, 32, 33, 4096, 4097, 10, 12289, 7, 20001, 64, 8191]


@pytest.mark.parametrize("bits", [1, 2, 4, 8, 16])
def test_unfused_parity_ragged(api, oracle, bits, rng_bits):
    offs, grads, theta, mom = _random_problem(bits, SIZES_RAGGED, 3)
    _check_unfused(api, oracle, offs, grads, theta, mom, bits, HP, rng_bits=rng_bits)


def _check_unfused_per_worker(api, oracle, offs, grads, theta, mom, bits, hp, seed=3, step=5, rng_bits=16):
    """The paper-literal quantizer (one norm per worker, Eq. rand_q) and Eq. grad_agg summed in fp32."""
    M = len(grads)
    d = int(offs[-1])
    h = len(offs) - 1
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, M, bits, rng_bits, scale_mode=api.DAT_SCALE_PER_WORKER) as P:
        assert P.num_scales == M * h
        lv, sg, sc = P.alloc_message()
        api.dat_quantize(P.plan, g_dev, seed, step, lv, sg, sc)
        torch.cuda.synchronize()
        sc_gpu = np_of(sc).reshape(M, h)
        sc_ref = oracle.scales(oracle.worker_norms(offs, grads), oracle.SCALE_PER_WORKER)
        assert ulp_diff(sc_gpu, sc_ref).max() <= 1
        level, neg = oracle.quantize(offs, grads, bits, seed, step, sc_gpu, oracle.SCALE_PER_WORKER, rng_bits=rng_bits)
        lp_ref, sp_ref = oracle_planes(oracle, level, neg, bits)
        assert np.array_equal(np_of(lv).reshape(M, -1), lp_ref)
        assert np.array_equal(np_of(sg).reshape(M, -1), sp_ref)
        gh = torch.zeros(d, dtype=torch.float32, device="cuda")
        api.dat_aggregate(P.plan, lv, sg, sc, None, gh)
        _, gh_ref = oracle.aggregate(offs, level, neg, sc_gpu, bits, oracle.SCALE_PER_WORKER)
        assert np.array_equal(np_of(gh).view(np.uint32), gh_ref.view(np.uint32))
        th_d, mo_d = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        api.dat_lalr_step(P.plan, th_d, mo_d, gh, hp)
        th_ref, mo_ref, _ = oracle.lalr(offs, theta, mom, gh_ref, *hp)
        assert np.array_equal(np_of(mo_d).view(np.uint32), mo_ref.view(np.uint32))
        assert_close_per_layer(np_of(th_d), th_ref, offs, "theta (per-worker scales)")
        assert P.status() == 0
        # what this mode does not offer is refused on the host
        cs = torch.zeros(d, dtype=torch.int32, device="cuda")
        with pytest.raises(api.DatError) as e:
            api.dat_aggregate(P.plan, lv, sg, sc, cs, gh)
        assert e.value.code == api.DAT_ERR_ARG
        # the same in one call: dat_step on a per-worker plan (M*h norms out, no integer code sums)
        th_s, mo_s = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        sc_s = torch.zeros(M * h, dtype=torch.float32, device="cuda")
        norms = torch.zeros(2 * h, dtype=torch.float32, device="cuda")
        api.dat_step(P.plan, th_s, mo_s, g_dev, seed, step, hp, None, norms, sc_s)
        torch.cuda.synchronize()
        assert P.status() == 0
        sc_step = np_of(sc_s).reshape(M, h)
        assert ulp_diff(sc_step, sc_ref).max() <= 1
        ref = oracle.step(offs, theta, mom, grads, bits, seed, step, *hp, scale_mode=oracle.SCALE_PER_WORKER,
                          scales_in=sc_step, rng_bits=rng_bits)
        assert np.array_equal(np_of(mo_s).view(np.uint32), ref["mom"].view(np.uint32))
        assert ulp_diff(np_of(norms).reshape(-1, 2), ref["layer_norms"]).max() <= 1
        assert_close_per_layer(np_of(th_s), ref["theta"], offs, "theta (dat_step, per-worker scales)")


@pytest.mark.parametrize("bits", [1, 4, 8, 16])
def test_unfused_parity_per_worker_scales(api, oracle, bits, rng_bits):
    offs, grads, theta, mom = _random_problem(40 + bits, SIZES_RAGGED, 5)
    grads[2] *= np.float32(37.0)                 # workers with very different norms
    grads[4][int(offs[7]):int(offs[8])] = 0.0    # one worker's layer all zero: its norm is 0
    _check_unfused_per_worker(api, oracle, offs, grads, theta, mom, bits, HP, rng_bits=rng_bits)


@pytest.mark.parametrize("bits", [1, 2, 8, 16])
def test_two_sided_requantize_parity(api, oracle, bits, rng_bits):
    """Algorithm A1 Step 10 on the GPU against the oracle: norms within 1 ulp, then (given the GPU's
    norm bits) the server's packed message and the receiver's value bit for bit."""
    offs, grads, theta, mom = _random_problem(70 + bits, SIZES_RAGGED, 3)
    d, M = int(offs[-1]), 3
    g = grads[0].copy()
    g[int(offs[9]):int(offs[10])] = 0.0          # a layer whose aggregate is zero
    with GpuPlan(api, offs, M, bits, rng_bits) as P:
        gh = torch.from_numpy(g).cuda()
        lv = torch.full((P.level_bytes,), 0xAB, dtype=torch.uint8, device="cuda")
        sg = torch.full((P.sign_bytes,), 0xCD, dtype=torch.uint8, device="cuda")
        sc = torch.zeros(P.h, dtype=torch.float32, device="cuda")
        api.dat_requantize(P.plan, gh, 5, 2, lv, sg, sc)
        torch.cuda.synchronize()
        _, sc_ref, _, _ = oracle.requantize(offs, g, bits, 5, 2, stream=M, rng_bits=rng_bits)
        sc_gpu = np_of(sc)
        assert ulp_diff(sc_gpu, sc_ref).max() <= 1
        out_ref, _, level, neg = oracle.requantize(offs, g, bits, 5, 2, stream=M, rng_bits=rng_bits, scales_in=sc_gpu)
        lp_ref, sp_ref = oracle.pack(level, neg, bits)
        assert np.array_equal(np_of(lv), lp_ref) and np.array_equal(np_of(sg), sp_ref)
        assert np.array_equal(np_of(gh).view(np.uint32), out_ref.view(np.uint32))
        # caller-supplied norms, in place
        gh2 = torch.from_numpy(g).cuda()
        api.dat_requantize(P.plan, gh2, 5, 2, lv, sg, sc, scales_in=sc)
        torch.cuda.synchronize()
        assert torch.equal(gh2, gh)
        assert P.status() == 0


LAMB_HP = (0.2, 0.9, 0.999, 1e-6, 1e-4, 0.0, 10.0)      # lr, beta1, beta2, zeta, weight decay, c_l, c_u


def test_lamb_step_parity_three_steps(api, oracle):
    """Algorithm A2 + Eq. upth on the GPU against the oracle over t = 1, 2, 3: the moments bit for bit (both
    sides are fed the same g_hat and the same theta history), theta' within the tolerance, norms within 1 ulp."""
    offs, grads, theta, mom = _random_problem(91, SIZES_RAGGED + [0 + 50000], 3)
    d = int(offs[-1])
    theta[int(offs[4]):int(offs[5])] = 0.0                     # an all-zero parameter tensor
    var = np.zeros(d, dtype=np.float32)
    mom = np.zeros(d, dtype=np.float32)
    with GpuPlan(api, offs, 3, 8) as P:
        th_d, mo_d, va_d = (torch.from_numpy(x.copy()).cuda() for x in (theta, mom, var))
        norms = torch.zeros(2 * P.h, dtype=torch.float32, device="cuda")
        th_ref, mo_ref, va_ref = theta, mom, var
        for t in (1, 2, 3):
            g = grads[t - 1]
            if t == 2:
                g = g.copy()
                g[int(offs[10]):int(offs[11])] = 0.0           # a layer with zero gradient
            th_in = np_of(th_d).copy()                         # the oracle continues from the GPU's theta: moments stay comparable
            api.dat_lamb_step(P.plan, th_d, mo_d, va_d, torch.from_numpy(g).cuda(), LAMB_HP, t, norms)
            torch.cuda.synchronize()
            th_ref, mo_ref, va_ref, n_ref = oracle.lamb(offs, th_in, mo_ref, va_ref, g, t, *LAMB_HP)
            assert np.array_equal(np_of(mo_d).view(np.uint32), mo_ref.view(np.uint32))
            assert np.array_equal(np_of(va_d).view(np.uint32), va_ref.view(np.uint32))
            assert ulp_diff(np_of(norms).reshape(-1, 2), n_ref).max() <= 1
            assert_close_per_layer(np_of(th_d), th_ref, offs, "theta (LAMB, t = %d)" % t)
        assert P.status() == 0
        with pytest.raises(api.DatError) as e:
            api.dat_lamb_step(P.plan, th_d, mo_d, va_d, th_d, LAMB_HP, 0)
        assert e.value.code == api.DAT_ERR_ARG


@pytest.mark.parametrize("mode", ["shared", "per_worker", "b32"])
def test_step_lamb_parity_three_steps(api, oracle, mode):
    """dat_step_lamb: Steps 7 and 9 followed by Algorithm A2 and Eq. upth in the one launch, over t = 1, 2, 3
    with fresh gradients and an advancing step counter.  The oracle gets the GPU's quantizer norms and the
    GPU's theta history; then g_hat is its own, and m', v' must agree bit for bit, theta' within the tolerance."""
    M, bits = 4, (32 if mode == "b32" else 8)
    sm = oracle.SCALE_PER_WORKER if mode == "per_worker" else oracle.SCALE_SHARED_MAX
    offs, _, theta, _ = _random_problem(93, SIZES_RAGGED + [50000], M)
    d, h = int(offs[-1]), len(offs) - 1
    theta[int(offs[4]):int(offs[5])] = 0.0                     # an all-zero parameter tensor
    mom, var = np.zeros(d, dtype=np.float32), np.zeros(d, dtype=np.float32)
    with GpuPlan(api, offs, M, bits, 16, scale_mode=api.DAT_SCALE_PER_WORKER if mode == "per_worker" else 0) as P:
        th_d, mo_d, va_d = (torch.from_numpy(x.copy()).cuda() for x in (theta, mom, var))
        norms = torch.zeros(2 * h, dtype=torch.float32, device="cuda")
        sc = torch.zeros(P.num_scales, dtype=torch.float32, device="cuda")
        mo_ref, va_ref = mom, var
        for t in (1, 2, 3):
            _, grads, _, _ = _random_problem(200 + t, SIZES_RAGGED + [50000], M)
            if t == 2:
                for g in grads:
                    g[int(offs[10]):int(offs[11])] = 0.0       # a layer with zero gradient
            th_in = np_of(th_d).copy()
            api.dat_step_lamb(P.plan, th_d, mo_d, va_d, [torch.from_numpy(g).cuda() for g in grads], 7, t, LAMB_HP, t, None, norms, sc)
            torch.cuda.synchronize()
            assert P.status() == 0
            if bits == 32:
                gh = oracle.average(offs, grads)
            else:
                sc_gpu = np_of(sc)
                sc_ref = oracle.scales(oracle.worker_norms(offs, grads), sm)
                assert ulp_diff(sc_gpu.reshape(sc_ref.shape), sc_ref).max() <= 1
                level, neg = oracle.quantize(offs, grads, bits, 7, t, sc_gpu, sm, rng_bits=16)
                _, gh = oracle.aggregate(offs, level, neg, sc_gpu, bits, sm)
            th_ref, mo_ref, va_ref, n_ref = oracle.lamb(offs, th_in, mo_ref, va_ref, gh, t, *LAMB_HP)
            assert np.array_equal(np_of(mo_d).view(np.uint32), mo_ref.view(np.uint32))
            assert np.array_equal(np_of(va_d).view(np.uint32), va_ref.view(np.uint32))
            assert ulp_diff(np_of(norms).reshape(-1, 2), n_ref).max() <= 1
            assert_close_per_layer(np_of(th_d), th_ref, offs, "theta (dat_step_lamb, t = %d)" % t)
        with pytest.raises(api.DatError) as e:
            api.dat_step_lamb(P.plan, th_d, mo_d, va_d, [torch.from_numpy(g).cuda() for g in grads], 7, 4, LAMB_HP, 0)
        assert e.value.code == api.DAT_ERR_ARG


@pytest.mark.parametrize("mode", ["shared", "per_worker"])
@pytest.mark.parametrize("bits", [1, 2, 4, 8, 16])
def test_aggregate_gather_equals_aggregate(api, oracle, bits, mode):
    """dat_aggregate_gather: every worker's planes in a buffer of its own (as a peer would hold them); the
    result is dat_aggregate's bit for bit, and the oracle's."""
    M = 5
    sm = oracle.SCALE_PER_WORKER if mode == "per_worker" else oracle.SCALE_SHARED_MAX
    offs, grads, _, _ = _random_problem(60 + bits, SIZES_RAGGED, M)
    d = int(offs[-1])
    with GpuPlan(api, offs, M, bits, 16, scale_mode=api.DAT_SCALE_PER_WORKER if mode == "per_worker" else 0) as P:
        lv, sg, sc = P.alloc_message()
        api.dat_quantize(P.plan, [torch.from_numpy(g).cuda() for g in grads], 3, 5, lv, sg, sc)
        lb, sb, _, _ = api.dat_plan_sizes(P.plan)
        pad = torch.empty(48, dtype=torch.uint8, device="cuda")          # (separate allocations, in scrambled order)
        lvs = [lv[i * lb:(i + 1) * lb].clone() for i in reversed(range(M))][::-1]
        sgs = [sg[i * sb:(i + 1) * sb].clone() for i in range(M)]
        cs1 = None if mode == "per_worker" else torch.zeros(d, dtype=torch.int32, device="cuda")
        cs2 = None if mode == "per_worker" else torch.zeros(d, dtype=torch.int32, device="cuda")
        g1, g2 = torch.zeros(d, device="cuda"), torch.zeros(d, device="cuda")
        api.dat_aggregate(P.plan, lv, sg, sc, cs1, g1)
        api.dat_aggregate_gather(P.plan, lvs, sgs, sc, cs2, g2)
        torch.cuda.synchronize()
        assert torch.equal(g1, g2) and (cs1 is None or torch.equal(cs1, cs2))
        level, neg = oracle.quantize(offs, grads, bits, 3, 5, np_of(sc), sm, rng_bits=16)
        _, gh = oracle.aggregate(offs, level, neg, np_of(sc), bits, sm)
        assert np.array_equal(np_of(g2).view(np.uint32), gh.view(np.uint32))
        with pytest.raises(api.DatError) as e:                           # a worker without planes
            api.dat_aggregate_gather(P.plan, lvs[:-1] + [None], sgs, sc, None, g2)
        assert e.value.code == api.DAT_ERR_ARG
        with pytest.raises(api.DatError) as e:                           # a plane that is not 16-byte aligned
            api.dat_aggregate_gather(P.plan, [lvs[0].data_ptr() + 4] + lvs[1:], sgs, sc, None, g2)
        assert e.value.code == api.DAT_ERR_ALIGN
        del pad


class _Guarded:
    """Buffers cut out of larger ones whose margins hold a pattern: nothing may write outside what it was given."""
    MARGIN = 256                                                    # bytes on either side (keeps 16-byte alignment)

    def __init__(self):
        self.items = []

    def make(self, n, dtype, fill=0):
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        whole = torch.full((nbytes + 2 * self.MARGIN,), 0x5A, dtype=torch.uint8, device="cuda")
        body = whole[self.MARGIN:self.MARGIN + nbytes]
        body.fill_(0)
        view = body.view(dtype)
        if fill:
            view.fill_(fill)
        self.items.append(whole)
        return view

    def check(self):
        torch.cuda.synchronize()
        for whole in self.items:
            assert bool((whole[:self.MARGIN] == 0x5A).all()) and bool((whole[-self.MARGIN:] == 0x5A).all()), "a write outside a buffer"


@pytest.mark.parametrize("bits", [1, 4, 8])
def test_nothing_is_written_outside_the_callers_buffers(api, bits, rng_bits):
    """Every output of every entry point sits between two margins of a known pattern; ragged layers, M = 3."""
    M = 3
    offs, grads, theta, mom = _random_problem(70 + bits, SIZES_RAGGED, M)
    d, h = int(offs[-1]), len(offs) - 1
    gs = [torch.from_numpy(g).cuda() for g in grads]
    for scale_mode in (0, api.DAT_SCALE_PER_WORKER):
        with GpuPlan(api, offs, M, bits, rng_bits, scale_mode=scale_mode) as P:
            lb, sb, ns, _ = api.dat_plan_sizes(P.plan)
            G = _Guarded()
            lv, sg, sc = G.make(M * lb, torch.uint8), G.make(M * sb, torch.uint8), G.make(ns, torch.float32)
            wn = G.make(M * h, torch.float32)
            cs = None if scale_mode else G.make(d, torch.int32)
            gh, gh2 = G.make(d, torch.float32), G.make(d, torch.float32)
            th, mo, va = G.make(d, torch.float32), G.make(d, torch.float32), G.make(d, torch.float32)
            th.copy_(torch.from_numpy(theta)); mo.copy_(torch.from_numpy(mom))
            norms, sc_out, sc2 = G.make(2 * h, torch.float32), G.make(ns, torch.float32), G.make(h, torch.float32)
            slv, ssg, ssc = G.make(lb, torch.uint8), G.make(sb, torch.uint8), G.make(h, torch.float32)
            api.dat_worker_norms(P.plan, gs, wn)
            api.dat_quantize(P.plan, gs, 3, 0, lv, sg, sc)
            api.dat_aggregate(P.plan, lv, sg, sc, cs, gh)
            api.dat_aggregate_gather(P.plan, [lv[i * lb:(i + 1) * lb] for i in range(M)], [sg[i * sb:(i + 1) * sb] for i in range(M)], sc, cs, gh)
            api.dat_requantize(P.plan, gh, 3, 0, slv, ssg, ssc)
            api.dat_lalr_step(P.plan, th, mo, gh, HP, norms)
            api.dat_lamb_step(P.plan, th, mo, va, gh, LAMB_HP, 1, norms)
            api.dat_step(P.plan, th, mo, gs, 3, 1, HP, cs, norms, sc_out)
            api.dat_step_lamb(P.plan, th, mo, va, gs, 3, 2, LAMB_HP, 2, cs, norms, sc_out)
            api.dat_step_two_sided(P.plan, th, mo, gs, 3, 3, HP, gh2, cs, norms, sc_out, sc2)
            api.dat_step_lamb_two_sided(P.plan, th, mo, va, gs, 3, 4, LAMB_HP, 3, gh2, cs, norms, sc_out, sc2)
            if not scale_mode:
                api.dat_step_passes(P.plan, th, mo, gs, 3, 5, HP, cs, norms, sc_out)
            assert P.status() == 0
            G.check()


def test_step_refuses_stream_capture(api):
    """The one-launch step carries its epoch and its Philox key as launch parameters: it must not end up in a graph."""
    offs, grads, theta, mom = _random_problem(5, [1000, 5000], 2)
    with GpuPlan(api, offs, 2, 8, 16) as P:
        th, mo = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        gs = [torch.from_numpy(g).cuda() for g in grads]
        api.dat_step(P.plan, th, mo, gs, 1, 0, HP)
        torch.cuda.synchronize()
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            g.capture_begin()
            try:
                th.add_(0.0)                                        # something to capture
                with pytest.raises(api.DatError) as e:
                    api.dat_step(P.plan, th, mo, gs, 1, 1, HP, stream=s)
                assert e.value.code == api.DAT_ERR_UNSUPPORTED
            finally:
                g.capture_end()
        torch.cuda.synchronize()
        th2, mo2 = th.clone(), mo.clone()
        api.dat_step(P.plan, th, mo, gs, 1, 1, HP)                  # the plan is as it was
        with GpuPlan(api, offs, 2, 8, 16) as P2:
            api.dat_step(P2.plan, th2, mo2, gs, 1, 1, HP)
            torch.cuda.synchronize()
        assert torch.equal(th, th2) and torch.equal(mo, mo2)


def _two_sided_reference(oracle, offs, grads, bits, seed, step, M, sm, rng_bits, sc_gpu, sc2_gpu):
    """Steps 7, 9 and 10 from the oracle's own operations: the workers' levels with the GPU's quantizer norms,
    the aggregate, the server's Q(g_hat) with the GPU's server norms (each norm checked to the last place first)."""
    sc_ref = oracle.scales(oracle.worker_norms(offs, grads), sm)
    assert ulp_diff(sc_gpu.reshape(sc_ref.shape), sc_ref).max() <= 1
    level, neg = oracle.quantize(offs, grads, bits, seed, step, sc_gpu, sm, rng_bits=rng_bits)
    cs, gh = oracle.aggregate(offs, level, neg, sc_gpu, bits, sm)
    _, sc2_ref, _, _ = oracle.requantize(offs, gh, bits, seed, step, stream=M, rng_bits=rng_bits)
    assert ulp_diff(sc2_gpu, sc2_ref).max() <= 1
    out, _, _, _ = oracle.requantize(offs, gh, bits, seed, step, stream=M, rng_bits=rng_bits, scales_in=sc2_gpu)
    return cs, out


@pytest.mark.parametrize("mode", ["shared", "per_worker"])
@pytest.mark.parametrize("bits", [1, 2, 8, 16])
def test_step_two_sided_parity(api, oracle, bits, mode, rng_bits):
    """dat_step_two_sided: Steps 7, 9, 10 and 12 in the one launch, twice in a row on the same plan (fresh
    gradients, advancing step counter).  The receiver's value and m' bit for bit, theta' within the tolerance."""
    M = 5
    sm = oracle.SCALE_PER_WORKER if mode == "per_worker" else oracle.SCALE_SHARED_MAX
    sizes = SIZES_RAGGED + [50000]
    offs, _, theta, mom = _random_problem(300 + bits, sizes, M)
    d, h = int(offs[-1]), len(offs) - 1
    theta[int(offs[4]):int(offs[5])] = 0.0                     # an all-zero parameter tensor
    with GpuPlan(api, offs, M, bits, rng_bits, scale_mode=api.DAT_SCALE_PER_WORKER if mode == "per_worker" else 0) as P:
        th_d, mo_d = torch.from_numpy(theta.copy()).cuda(), torch.from_numpy(mom.copy()).cuda()
        gh_d = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
        cs_d = torch.zeros(d, dtype=torch.int32, device="cuda")
        norms = torch.zeros(2 * h, dtype=torch.float32, device="cuda")
        sc = torch.zeros(P.num_scales, dtype=torch.float32, device="cuda")
        sc2 = torch.zeros(h, dtype=torch.float32, device="cuda")
        mo_ref = mom
        for step in (0, 1):
            _, grads, _, _ = _random_problem(400 + bits + step, sizes, M, dist="t3" if step else "normal")
            if step == 1:
                for g in grads:
                    g[int(offs[10]):int(offs[11])] = 0.0       # a layer with zero gradient: nu = nu^ = 0
            th_in = np_of(th_d).copy()
            api.dat_step_two_sided(P.plan, th_d, mo_d, [torch.from_numpy(g).cuda() for g in grads], 9, step, HP, gh_d,
                                   cs_d, norms, sc, sc2)
            torch.cuda.synchronize()
            assert P.status() == 0
            cs_ref, out = _two_sided_reference(oracle, offs, grads, bits, 9, step, M, sm, rng_bits, np_of(sc), np_of(sc2))
            if mode == "shared":
                assert np.array_equal(np_of(cs_d), cs_ref)
            assert np.array_equal(np_of(gh_d).view(np.uint32), out.view(np.uint32)), "the receiver's value"
            th_ref, mo_ref, n_ref = oracle.lalr(offs, th_in, mo_ref, out, *HP)
            assert np.array_equal(np_of(mo_d).view(np.uint32), mo_ref.view(np.uint32))
            assert ulp_diff(np_of(norms).reshape(-1, 2), n_ref).max() <= 1
            assert_close_per_layer(np_of(th_d), th_ref, offs, "theta (dat_step_two_sided, step %d)" % step)
        # the one-sided step on the same plan afterwards is the ordinary one
        th1, mo1 = torch.from_numpy(theta.copy()).cuda(), torch.from_numpy(mom.copy()).cuda()
        th2, mo2 = th1.clone(), mo1.clone()
        gs = [torch.from_numpy(g).cuda() for g in grads]
        api.dat_step(P.plan, th1, mo1, gs, 9, 5, HP)
        with GpuPlan(api, offs, M, bits, rng_bits, scale_mode=api.DAT_SCALE_PER_WORKER if mode == "per_worker" else 0) as P2:
            api.dat_step(P2.plan, th2, mo2, gs, 9, 5, HP)
            torch.cuda.synchronize()
        assert torch.equal(th1, th2) and torch.equal(mo1, mo2)


def test_step_lamb_two_sided_parity(api, oracle):
    M, bits = 4, 4
    sizes = SIZES_RAGGED + [50000]
    offs, grads, theta, _ = _random_problem(95, sizes, M)
    d, h = int(offs[-1]), len(offs) - 1
    mom, var = np.zeros(d, dtype=np.float32), np.zeros(d, dtype=np.float32)
    with GpuPlan(api, offs, M, bits, 16) as P:
        th_d, mo_d, va_d = (torch.from_numpy(x.copy()).cuda() for x in (theta, mom, var))
        gh_d = torch.zeros(d, dtype=torch.float32, device="cuda")
        norms = torch.zeros(2 * h, dtype=torch.float32, device="cuda")
        sc = torch.zeros(P.num_scales, dtype=torch.float32, device="cuda")
        sc2 = torch.zeros(h, dtype=torch.float32, device="cuda")
        mo_ref, va_ref = mom, var
        for t in (1, 2):
            th_in = np_of(th_d).copy()
            api.dat_step_lamb_two_sided(P.plan, th_d, mo_d, va_d, [torch.from_numpy(g).cuda() for g in grads], 7, t, LAMB_HP, t,
                                        gh_d, None, norms, sc, sc2)
            torch.cuda.synchronize()
            assert P.status() == 0
            _, out = _two_sided_reference(oracle, offs, grads, bits, 7, t, M, oracle.SCALE_SHARED_MAX, 16, np_of(sc), np_of(sc2))
            th_ref, mo_ref, va_ref, n_ref = oracle.lamb(offs, th_in, mo_ref, va_ref, out, t, *LAMB_HP)
            assert np.array_equal(np_of(mo_d).view(np.uint32), mo_ref.view(np.uint32))
            assert np.array_equal(np_of(va_d).view(np.uint32), va_ref.view(np.uint32))
            assert ulp_diff(np_of(norms).reshape(-1, 2), n_ref).max() <= 1
            assert_close_per_layer(np_of(th_d), th_ref, offs, "theta (dat_step_lamb_two_sided, t = %d)" % t)
    with GpuPlan(api, offs, M, 32, 16) as P:                    # b = 32: nothing to quantize with
        with pytest.raises(api.DatError) as e:
            api.dat_step_two_sided(P.plan, th_d, mo_d, [torch.from_numpy(g).cuda() for g in grads], 7, 0, HP, gh_d)
        assert e.value.code == api.DAT_ERR_BITS


@pytest.mark.parametrize("bits", [1, 2, 4, 8, 16, 32])
def test_fused_parity_ragged(api, oracle, bits, rng_bits):
    offs, grads, theta, mom = _random_problem(100 + bits, SIZES_RAGGED, 3)
    _check_fused(api, oracle, offs, grads, theta, mom, bits, HP, rng_bits=rng_bits)


@pytest.mark.parametrize("M", [1, 2, 5, 8, 13, 32, 64])
def test_fused_parity_worker_counts(api, oracle, M, rng_bits):
    offs, grads, theta, mom = _random_problem(M, [1000, 5000, 3, 9000], M, dist="t3")
    _check_fused(api, oracle, offs, grads, theta, mom, 4, HP, rng_bits=rng_bits)


@pytest.mark.parametrize("bits", [1, 2, 4, 8, 16])
def test_step_passes_parity_ragged(api, oracle, bits, rng_bits):
    """The three-pass form of the step against the oracle, under the same protocol as the fused kernel."""
    offs, grads, theta, mom = _random_problem(100 + bits, SIZES_RAGGED, 3)
    _check_fused(api, oracle, offs, grads, theta, mom, bits, HP, rng_bits=rng_bits, entry="dat_step_passes")


@pytest.mark.parametrize("M", [1, 5, 13, 64])
def test_step_passes_worker_counts_and_extreme_scales(api, oracle, M, rng_bits):
    offs, grads, theta, mom = _random_problem(M, [1000, 5000, 3, 9000], M, dist="t3")
    grads = [g.copy() for g in grads]
    for g in grads:
        g[int(offs[1]):int(offs[2])] *= np.float32(1e30)      # a huge layer norm: the plain form takes over
        g[int(offs[3]):] *= np.float32(1e-30)                 # a tiny one
        g[int(offs[2]):int(offs[3])] = 0.0                    # a zero one
    _check_fused(api, oracle, offs, grads, theta, mom, 8, HP, rng_bits=rng_bits, entry="dat_step_passes")


def test_bounded_wait_runs_out_and_plan_recovers(api, oracle):
    """The wait of a work item for a layer's norm is bounded.  With the test hook the limit is set to about a
    millisecond and one layer's tile counter is pre-set so that the layer never completes: the call must
    return, the status word must carry DAT_STATUS_TIMEOUT, and after dat_get_status the next ordinary call
    on the same plan must give what a fresh plan gives, bit for bit."""
    import time
    offs, grads, theta, mom = _random_problem(77, [5000, 300, 9000, 40], 3)
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, 3, 8) as P:
        api.dat_plan_test_stall(P.plan, 2_000_000, 2)
        th, mo = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        t0 = time.time()
        api.dat_step(P.plan, th, mo, g_dev, 5, 9, HP)
        torch.cuda.synchronize()
        assert time.time() - t0 < 10.0
        assert P.status() & api.DAT_STATUS_TIMEOUT
        assert P.status() == 0                                  # read and cleared
        api.dat_plan_test_stall(P.plan, 0, -1)                  # the default limit again
        th1, mo1 = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        api.dat_step(P.plan, th1, mo1, g_dev, 5, 9, HP)
        torch.cuda.synchronize()
        assert P.status() == 0
        with GpuPlan(api, offs, 3, 8) as P2:
            th2, mo2 = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
            api.dat_step(P2.plan, th2, mo2, g_dev, 5, 9, HP)
            torch.cuda.synchronize()
        assert torch.equal(th1, th2) and torch.equal(mo1, mo2)
        ref = oracle.step(offs, theta, mom, grads, 8, 5, 9, *HP)
        assert_close_per_layer(np_of(th1), ref["theta"], offs, "theta after recovery")


def test_self_checking_build_runs_the_ragged_cases():
    """The build with -DDAT_SELFCHECK (DAT_DEBUG=1: every tile an item names is checked before use, a
    violation sets DAT_STATUS_BOUNDS instead of faulting) passes the ragged parity cases with a clean status."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, DAT_DEBUG="1")
    subprocess.check_call([sys.executable, "-m", "paper_2206_06257_b200.build"], cwd=root, env=env)   # no-op when up to date
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", os.path.join(root, "tests", "test_gpu_parity.py"),
                        "-k", "test_fused_parity_ragged and rng16"], env=env,
                       cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def test_step_passes_equals_fused_on_resnet18(api, oracle):
    from paper_2206_06257_b200 import synth
    cfg = synth.config("resnet18")
    theta, mom = synth.make_params(cfg, "cuda")
    grads = synth.make_grads(cfg, 0, "cuda")
    hp = hp_tuple(cfg)
    plan = api.dat_plan_create(cfg.offsets, cfg.M, cfg.bits, rng_bits=cfg.rng_bits)
    try:
        th1, mo1, th2, mo2 = theta.clone(), mom.clone(), theta.clone(), mom.clone()
        cs1 = torch.zeros(cfg.d, dtype=torch.int32, device="cuda")
        cs2 = torch.zeros(cfg.d, dtype=torch.int32, device="cuda")
        sc1 = torch.zeros(cfg.h, device="cuda")
        sc2 = torch.zeros(cfg.h, device="cuda")
        api.dat_step(plan, th1, mo1, grads, 0, 4, hp, cs1, None, sc1)
        api.dat_step_passes(plan, th2, mo2, grads, 0, 4, hp, cs2, None, sc2)
        torch.cuda.synchronize()
        assert ulp_diff(np_of(sc1), np_of(sc2)).max() <= 1
        if torch.equal(sc1, sc2):                              # same norm bits: everything downstream is comparable bit for bit
            assert torch.equal(cs1, cs2) and torch.equal(mo1, mo2)
        assert_close_per_layer(np_of(th2), np_of(th1), cfg.offsets, "theta (passes vs fused)")
        assert api.dat_get_status(plan) == 0
    finally:
        api.dat_plan_destroy(plan)


@pytest.mark.parametrize("M", [9, 13, 64])
def test_fused_b32_more_than_eight_workers(api, oracle, M):
    """No quantisation (b = 32) with more gradient rows than one batch holds: the ordered fp32 average of all M."""
    offs, grads, theta, mom = _random_problem(300 + M, [1000, 5000, 3, 9000], M)
    _check_fused(api, oracle, offs, grads, theta, mom, 32, HP)


@pytest.mark.parametrize("bits", [2, 8, 16])
def test_fused_parity_extreme_scales(api, oracle, bits, rng_bits):
    """Layers whose norms sit at the ends of the fp32 range (the scaled form of the level
    computation does not apply there), a layer with a single non-zero element (|g| = nu: the
    clamp of the level is live), subnormal gradients, and ordinary layers around them."""
    sizes = [3000, 2500, 4099, 2048, 2600, 777]
    offs, grads, theta, mom = _random_problem(7 + bits, sizes, 3)
    o = offs
    def rescale(x, norm):
        x64 = x.astype(np.float64)
        return (x64 / np.sqrt(np.sum(x64 * x64)) * norm).astype(np.float32)
    for i, g in enumerate(grads):
        g[o[0]:o[1]] = rescale(g[o[0]:o[1]], 2e38 if i == 1 else 3e37)      # S / nu * 2^-b is subnormal
        g[o[1]:o[2]] = rescale(g[o[1]:o[2]], 3e-40)                         # subnormal gradients and norm
        g[o[2]:o[3]] = 0.0
        g[o[2] + 1234 + i] = np.float32(-0.37 if i else 0.37)               # one element: |g| = nu
        g[o[4]:o[5]] = rescale(g[o[4]:o[5]], 1e-29)                         # tiny but normal
    _check_fused(api, oracle, offs, grads, theta, mom, bits, HP, rng_bits=rng_bits)
    _check_unfused(api, oracle, offs, grads, theta, mom, bits, HP, rng_bits=rng_bits)


def test_fused_equals_unfused_on_gpu(api, oracle, rng_bits):
    offs, grads, theta, mom = _random_problem(7, SIZES_RAGGED, 4)
    M, d = 4, int(offs[-1])
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, M, 8, rng_bits) as P:
        lv, sg, sc = P.alloc_message()
        gh = torch.zeros(d, dtype=torch.float32, device="cuda")
        th1, mo1 = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        api.dat_quantize(P.plan, g_dev, 1, 2, lv, sg, sc)
        api.dat_aggregate(P.plan, lv, sg, sc, None, gh)
        api.dat_lalr_step(P.plan, th1, mo1, gh, HP)
        th2, mo2 = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        api.dat_step(P.plan, th2, mo2, g_dev, 1, 2, HP)
        torch.cuda.synchronize()
        assert torch.equal(th1, th2) and torch.equal(mo1, mo2)


def test_b32_unfused_average(api, oracle):
    offs, grads, theta, mom = _random_problem(8, [100, 4099, 3], 5)
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, 5, 32) as P:
        gh = torch.zeros(int(offs[-1]), dtype=torch.float32, device="cuda")
        api.dat_average(P.plan, g_dev, gh)
        assert np.array_equal(np_of(gh).view(np.uint32), oracle.average(offs, grads).view(np.uint32))
        with pytest.raises(api.DatError) as e:
            api.dat_quantize(P.plan, g_dev, 0, 0, gh, gh, gh)
        assert e.value.code == api.DAT_ERR_BITS


def test_m1_b32_is_plain_lalr(api, oracle):
    offs, grads, theta, mom = _random_problem(9, [300, 5000], 1)
    th, mo = _check_fused(api, oracle, offs, grads, theta, mom, 32, HP)
    th_ref, mo_ref, _ = oracle.lalr(offs, theta, mom, grads[0], *HP)
    assert np.array_equal(mo, mo_ref)
    assert_close_per_layer(th, th_ref, offs, "theta")


def test_zero_norm_conventions(api, oracle):
    offs, grads, theta, mom = _random_problem(10, [500, 700, 900, 64], 3)
    for g in grads:
        g[offs[1]:offs[2]] = 0.0            # a layer whose gradient is zero for every worker
    theta[offs[2]:offs[3]] = 0.0            # an all-zero parameter tensor (momentum non-zero)
    theta[offs[3]:] = 0.0
    mom[offs[3]:] = 0.0                     # zero parameters, zero momentum: u = g_hat only
    th, mo = _check_fused(api, oracle, offs, grads, theta, mom, 8, HP)
    assert np.isfinite(th).all() and np.isfinite(mo).all()
    assert not th[offs[2]:offs[3]].any()    # tau(0) = c_l = 0: does not move
    assert mo[offs[2]:offs[3]].any()
    _check_unfused(api, oracle, offs, grads, theta, mom, 8, HP)


def test_all_zero_everything(api, oracle):
    offs = _offs([10, 5000])
    z = np.zeros(int(offs[-1]), dtype=np.float32)
    th, mo = _check_fused(api, oracle, offs, [z, z.copy()], z.copy(), z.copy(), 8, HP)
    assert not th.any() and not mo.any()


def test_scales_in_is_used(api, oracle):
    offs, grads, theta, mom = _random_problem(11, [1000, 3000], 2)
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, 2, 8) as P:
        lv, sg, sc = P.alloc_message()
        mine = np.array([0.5, 2.0], dtype=np.float32)      # larger and (for layer 0 maybe) smaller than max|g|
        mine[0] = np.abs(np.stack(grads)[:, :1000]).max() * 0.5   # forces the clamp to S
        sin = torch.from_numpy(mine).cuda()
        api.dat_quantize(P.plan, g_dev, 0, 0, lv, sg, sc, sin)
        assert np.array_equal(np_of(sc), mine)
        level, neg = oracle.quantize(offs, grads, 8, 0, 0, mine)
        assert level.max() == 255
        lp, sp = oracle_planes(oracle, level, neg, 8)
        assert np.array_equal(np_of(lv).reshape(2, -1), lp) and np.array_equal(np_of(sg).reshape(2, -1), sp)


@pytest.mark.parametrize("name", ["tiny_mlp", "flat_small"])
def test_config_small(api, oracle, name):
    from paper_2206_06257_b200 import synth
    cfg = synth.config(name)
    theta, mom = synth.make_params(cfg)
    grads = [g.numpy() for g in synth.make_grads(cfg, 0)]
    _check_unfused(api, oracle, cfg.offsets, grads, theta.numpy(), mom.numpy(), cfg.bits, hp_tuple(cfg), 0, 0)
    _check_fused(api, oracle, cfg.offsets, grads, theta.numpy(), mom.numpy(), cfg.bits, hp_tuple(cfg), 0, 0)


def test_resnet18_ten_steps_and_resume(api, oracle):
    """Ten consecutive steps, the step counter advancing the random key; state compared with the
    oracle after every step; then resume exactness (5 + copy + 5 == 10 straight)."""
    from paper_2206_06257_b200 import synth
    cfg = synth.config("resnet18")
    theta, mom = synth.make_params(cfg)
    hp = hp_tuple(cfg)
    th_ref, mo_ref = theta.numpy().copy(), mom.numpy().copy()
    sigma = synth._per_element(cfg, synth.layer_sigmas(cfg), "cpu")
    with GpuPlan(api, cfg.offsets, cfg.M, cfg.bits) as P:
        th_d, mo_d = theta.cuda(), mom.cuda()
        th_r, mo_r = theta.cuda(), mom.cuda()            # the resumed run
        sc = torch.zeros(cfg.h, dtype=torch.float32, device="cuda")
        for t in range(cfg.steps):
            grads = synth.make_grads(cfg, t, sigma_elem=sigma)
            g_dev = to_dev(grads)
            api.dat_step(P.plan, th_d, mo_d, g_dev, cfg.seed, t, hp, None, None, sc)
            if t == 5:                                   # "checkpoint": copy the state out and back
                th_r, mo_r = th_r.cpu().cuda(), mo_r.cpu().cuda()
            api.dat_step(P.plan, th_r, mo_r, g_dev, cfg.seed, t, hp)
            if t < 3 or t == cfg.steps - 1:
                # the oracle continues from the GPU's previous state, so that one step is compared
                ref = oracle.step(cfg.offsets, th_ref, mo_ref, [g.numpy() for g in grads], cfg.bits, cfg.seed, t,
                                  *hp, scales_in=np_of(sc), want_code_sum=False)
                assert np.array_equal(np_of(mo_d).view(np.uint32), ref["mom"].view(np.uint32))
                assert_close_per_layer(np_of(th_d), ref["theta"], cfg.offsets, "theta step %d" % t)
            th_ref, mo_ref = np_of(th_d).copy(), np_of(mo_d).copy()
        assert torch.equal(th_d, th_r) and torch.equal(mo_d, mo_r)
        assert P.status() == 0


def test_step_counter_changes_codes(api):
    offs, grads, theta, mom = _random_problem(12, [5000], 2)
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, 2, 8) as P:
        outs = []
        for seed, step in [(0, 0), (0, 1), (1, 0), (0, 0)]:
            cs = torch.zeros(5000, dtype=torch.int32, device="cuda")
            api.dat_step(P.plan, torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda(), g_dev, seed, step,
                         HP, cs)
            outs.append(cs.cpu())
        assert not torch.equal(outs[0], outs[1]) and not torch.equal(outs[0], outs[2])
        assert torch.equal(outs[0], outs[3])


def test_host_detected_errors(api):
    offs = _offs([100, 200])
    with pytest.raises(api.DatError) as e:
        api.dat_plan_create([0, 5, 5], 2, 8)
    assert e.value.code == api.DAT_ERR_LAYOUT
    with pytest.raises(api.DatError) as e:
        api.dat_plan_create(offs, 2, 3)
    assert e.value.code == api.DAT_ERR_BITS
    with pytest.raises(api.DatError) as e:
        api.dat_plan_create(offs, 0, 8)
    assert e.value.code == api.DAT_ERR_ARG
    with pytest.raises(api.DatError) as e:
        api.dat_plan_create(offs, 65, 8)
    assert e.value.code == api.DAT_ERR_ARG
    with GpuPlan(api, offs, 2, 8) as P:
        buf = torch.zeros(400, dtype=torch.float32, device="cuda")
        th, mo = torch.zeros(300, device="cuda"), torch.zeros(300, device="cuda")
        g = [torch.zeros(300, device="cuda"), torch.zeros(300, device="cuda")]
        before = api.dat_plan_launch_count(P.plan)
        with pytest.raises(api.DatError) as e:                 # misaligned gradient pointer
            api.dat_step(P.plan, th, mo, [g[0], buf[1:301]], 0, 0, HP)
        assert e.value.code == api.DAT_ERR_ALIGN
        with pytest.raises(api.DatError) as e:                 # step does not fit 32 bits
            api.dat_step(P.plan, th, mo, g, 0, 1 << 32, HP)
        assert e.value.code == api.DAT_ERR_ARG
        with pytest.raises(api.DatError) as e:                 # null pointer
            api.dat_step(P.plan, None, mo, g, 0, 0, HP)
        assert e.value.code == api.DAT_ERR_ARG
        with pytest.raises(api.DatError) as e:
            api.dat_lalr_step(P.plan, th, mo, buf[1:301], HP)
        assert e.value.code == api.DAT_ERR_ALIGN
        assert api.dat_plan_launch_count(P.plan) == before     # nothing was launched
        api.dat_step(P.plan, th, mo, g, 0, 0, HP)              # and the plan still works
        torch.cuda.synchronize()
        assert api.dat_plan_launch_count(P.plan) > before
        assert P.status() == 0


def test_nonfinite_input_sets_status_bit(api):
    offs = _offs([1000, 1000])
    g = [torch.randn(2000, device="cuda") * 0.01 for _ in range(2)]
    g[1][1500] = float("inf")
    with GpuPlan(api, offs, 2, 8) as P:
        th, mo = torch.randn(2000, device="cuda"), torch.zeros(2000, device="cuda")
        api.dat_step(P.plan, th, mo, g, 0, 0, HP)
        assert P.status() & api.DAT_STATUS_NONFINITE
        assert P.status() == 0                                   # reading clears it
        assert torch.isfinite(th[:1000]).all()                   # the finite layer is untouched by it
        g[1][1500] = 0.0
        api.dat_step(P.plan, torch.randn(2000, device="cuda"), mo.zero_(), g, 0, 1, HP)
        assert P.status() == 0


def test_step_host_matches_device_call(api):
    offs, grads, theta, mom = _random_problem(13, [3000, 50, 9001], 3)
    g_dev = [torch.from_numpy(g).cuda() for g in grads]
    with GpuPlan(api, offs, 3, 8) as P:
        th_d, mo_d = torch.from_numpy(theta).cuda(), torch.from_numpy(mom).cuda()
        api.dat_step(P.plan, th_d, mo_d, g_dev, 4, 4, HP)
        th_h = torch.from_numpy(theta.copy()).pin_memory()
        mo_h = torch.from_numpy(mom.copy()).pin_memory()
        g_h = [torch.from_numpy(g).pin_memory() for g in grads]
        api.dat_step_host(P.plan, th_h, mo_h, g_h, 4, 4, HP)
        assert torch.equal(th_h, th_d.cpu()) and torch.equal(mo_h, mo_d.cpu())
