"""Parity at the full sizes of the workloads, in the launch configuration bench.py times (dat_step;
inputs generated on the device).  The oracle recomputes sampled layers one by one (its window mode
keeps the global element index, hence the same random stream); properties that hold at any size are
checked on everything."""
import numpy as np
import pytest
import torch

from helpers import assert_close_per_layer, hp_tuple, np_of, ulp_diff

pytestmark = pytest.mark.gpu


ENTRIES = ["dat_step", "dat_step_passes"]


def _run_and_check(oracle, cfg, sample_layers, step=0, entry="dat_step"):
    from paper_2206_06257_b200 import api, synth
    dev = "cuda"
    theta, mom = synth.make_params(cfg, device=dev)
    grads = synth.make_grads(cfg, step, device=dev)
    hp = hp_tuple(cfg)
    th0, mo0 = theta.clone(), mom.clone()
    plan = api.dat_plan_create(cfg.offsets, cfg.M, cfg.bits, rng_bits=cfg.rng_bits)
    try:
        cs = torch.zeros(cfg.d, dtype=torch.int32, device=dev)
        sc = torch.zeros(cfg.h, dtype=torch.float32, device=dev)
        norms = torch.zeros(2 * cfg.h, dtype=torch.float32, device=dev)
        getattr(api, entry)(plan, theta, mom, grads, cfg.seed, step, hp, cs, norms, sc)
        torch.cuda.synchronize()
        assert api.dat_get_status(plan) == 0
    finally:
        api.dat_plan_destroy(plan)
    offs = cfg.offsets
    S = 2 ** cfg.bits - 1
    # properties at any size
    assert torch.isfinite(theta).all() and torch.isfinite(mom).all()
    assert int(cs.abs().max()) <= cfg.M * S
    norms_h = np_of(norms).reshape(-1, 2)
    d64 = (theta.double() - th0.double()) ** 2
    csum = torch.cat([torch.zeros(1, dtype=torch.float64, device=dev), torch.cumsum(d64, 0)])
    idx = torch.from_numpy(offs).to(dev)
    step_len = torch.sqrt((csum[idx[1:]] - csum[idx[:-1]]).clamp_min(0)).cpu().numpy()
    del d64, csum
    for l in range(cfg.h):
        tau = min(max(float(norms_h[l, 0]), cfg.c_l), cfg.c_u)
        expect = cfg.lr * tau if norms_h[l, 1] != 0 else 0.0
        # (the prefix-sum difference leaves ~1e-7 of cancellation noise on zero-step layers)
        assert abs(step_len[l] - expect) <= 1e-4 * expect + 1e-6, (l, step_len[l], expect)
    # sampled layers, element by element
    sc_h = np_of(sc)
    for l in sample_layers:
        a, b = int(offs[l]), int(offs[l + 1])
        g_l = [np_of(g[a:b]) for g in grads]
        ref = oracle.step(offs, np_of(th0[a:b]), np_of(mo0[a:b]), g_l, cfg.bits, cfg.seed, step, *hp,
                          l0=l, l1=l + 1, window=True, rng_bits=cfg.rng_bits)
        assert ulp_diff(sc_h[l:l + 1], ref["scales"][l:l + 1]).max() <= 1
        if sc_h[l] != ref["scales"][l]:
            ref = oracle.step(offs, np_of(th0[a:b]), np_of(mo0[a:b]), g_l, cfg.bits, cfg.seed, step, *hp,
                              l0=l, l1=l + 1, window=True, scales_in=sc_h, rng_bits=cfg.rng_bits)
        assert np.array_equal(np_of(cs[a:b]), ref["code_sum"]), "layer %d code sums" % l
        assert np.array_equal(np_of(mom[a:b]).view(np.uint32), ref["mom"].view(np.uint32)), "layer %d momentum" % l
        assert_close_per_layer(np_of(theta[a:b]), ref["theta"], np.array([0, b - a]), "theta layer %d" % l)
    return theta, mom


@pytest.mark.parametrize("entry", ENTRIES)
def test_resnet50_bench_configuration_every_layer(oracle, entry):
    from paper_2206_06257_b200 import synth
    cfg = synth.config("resnet50")
    _run_and_check(oracle, cfg, range(cfg.h), entry=entry)


def test_resnet50_every_layer_23_bit_uniform(oracle):
    """The bench workload once more at the other resolution of the quantizer's uniform number."""
    from paper_2206_06257_b200 import synth
    cfg = synth.config("resnet50")
    cfg.rng_bits = 23
    _run_and_check(oracle, cfg, range(cfg.h), step=3)


@pytest.mark.parametrize("entry", ENTRIES)
def test_resnet50_m32_b4_student_t_with_zero_layers(oracle, entry):
    """M = 32: a large layer's gradients (302 MB) do not fit the L2 cache.  One of the largest layers
    (2.36 M elements) is among those compared element by element."""
    from paper_2206_06257_b200 import synth
    cfg = synth.config("resnet50_m32")
    zg, zp = cfg.zero_grad_layers[0], cfg.zero_param_layers[0]
    sizes = np.diff(cfg.offsets)
    sample = sorted(set(list(range(0, cfg.h, 7)) + [zg, zp, 159, 160]))
    sample = [l for l in sample if sizes[l] <= 1_100_000] + [int(np.argmax(sizes))]
    theta, mom = _run_and_check(oracle, cfg, sample, entry=entry)
    a, b = int(cfg.offsets[zp]), int(cfg.offsets[zp + 1])
    assert not theta[a:b].any() and mom[a:b].any()          # all-zero tensor does not move (c_l = 0)


@pytest.mark.parametrize("entry", ENTRIES)
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_flat_1b_sampled_layers(oracle, bits, entry):
    """The 1B-parameter model at every bit width of its sweep.  Compared element by element: the two
    smallest layers, layers near the median and the lower third, the first and the last layer, one of
    about 300 k elements, one between 0.42 M and 2 M elements (several tiles of one layer per thread
    block row), and the largest layer (about 16 M elements)."""
    from paper_2206_06257_b200 import synth
    if torch.cuda.get_device_properties(0).total_memory < 80e9:
        pytest.skip("needs about 60 GB of device memory")
    cfg = synth.config("flat1b", bits=bits)
    sizes = np.diff(cfg.offsets)
    order = np.argsort(sizes)
    mid = [int(l) for l in order if 420_000 <= sizes[l] <= 2_000_000]
    sample = sorted(set([int(order[0]), int(order[1]), int(order[len(order) // 2]), int(order[len(order) // 3]),
                         0, cfg.h - 1, int(np.argmin(np.abs(sizes - 300_000))), mid[len(mid) // 2], int(order[-1])]))
    if entry != "dat_step":                                  # the large layers once per bit width are enough
        sample = [l for l in sample if sizes[l] <= 2_000_000]
    _run_and_check(oracle, cfg, sample, entry=entry)
    torch.cuda.empty_cache()


def test_resnet50_two_sided_sampled_layers(oracle):
    """dat_step_two_sided on the bench workload.  The oracle's own operations, layer by layer on windows that
    keep the global element index: the workers' levels, the aggregate, then -- on the full vector, with the
    sampled layers filled in -- the server's Q(g_hat), and the update of each sampled layer."""
    from paper_2206_06257_b200 import api, synth
    cfg = synth.config("resnet50")
    dev, step = "cuda", 2
    theta, mom = synth.make_params(cfg, device=dev)
    grads = synth.make_grads(cfg, step, device=dev)
    hp = hp_tuple(cfg)
    th0, mo0 = theta.clone(), mom.clone()
    gh = torch.zeros(cfg.d, dtype=torch.float32, device=dev)
    sc = torch.zeros(cfg.h, dtype=torch.float32, device=dev)
    sc2 = torch.zeros(cfg.h, dtype=torch.float32, device=dev)
    norms = torch.zeros(2 * cfg.h, dtype=torch.float32, device=dev)
    plan = api.dat_plan_create(cfg.offsets, cfg.M, cfg.bits, rng_bits=cfg.rng_bits)
    try:
        api.dat_step_two_sided(plan, theta, mom, grads, cfg.seed, step, hp, gh, None, norms, sc, sc2)
        torch.cuda.synchronize()
        assert api.dat_get_status(plan) == 0
    finally:
        api.dat_plan_destroy(plan)
    offs = cfg.offsets
    sizes = np.diff(offs)
    sample = sorted(set(list(range(0, cfg.h, 9)) + [int(np.argmax(sizes)), int(np.argmin(sizes)), cfg.h - 2, cfg.h - 1]))
    sc_h, sc2_h = np_of(sc), np_of(sc2)
    gh_full = np.zeros(cfg.d, dtype=np.float32)
    for l in sample:
        a, b = int(offs[l]), int(offs[l + 1])
        g_l = [np_of(g[a:b]) for g in grads]
        nu = oracle.scales(oracle.worker_norms(offs, g_l, l0=l, l1=l + 1, window=True))
        assert ulp_diff(sc_h[l:l + 1], nu[l:l + 1]).max() <= 1
        level, neg = oracle.quantize(offs, g_l, cfg.bits, cfg.seed, step, sc_h, l0=l, l1=l + 1, window=True, rng_bits=cfg.rng_bits)
        _, gh_full[a:b] = oracle.aggregate(offs, level, neg, sc_h, cfg.bits, l0=l, l1=l + 1, window=True)
    _, sc2_ref, _, _ = oracle.requantize(offs, gh_full, cfg.bits, cfg.seed, step, stream=cfg.M, rng_bits=cfg.rng_bits)
    out, _, _, _ = oracle.requantize(offs, gh_full, cfg.bits, cfg.seed, step, stream=cfg.M, rng_bits=cfg.rng_bits, scales_in=sc2_h)
    gh_h, th_h, mo_h = np_of(gh), np_of(theta), np_of(mom)
    norms_h = np_of(norms).reshape(-1, 2)
    for l in sample:
        a, b = int(offs[l]), int(offs[l + 1])
        assert ulp_diff(sc2_h[l:l + 1], sc2_ref[l:l + 1]).max() <= 1
        assert np.array_equal(gh_h[a:b].view(np.uint32), out[a:b].view(np.uint32)), "layer %d: the receiver's value" % l
        th_ref, mo_ref, n_ref = oracle.lalr(offs, np_of(th0[a:b]), np_of(mo0[a:b]), out[a:b], *hp, l0=l, l1=l + 1, window=True)
        assert np.array_equal(mo_h[a:b].view(np.uint32), mo_ref.view(np.uint32)), "layer %d momentum" % l
        assert ulp_diff(norms_h[l], n_ref[l]).max() <= 1
        assert_close_per_layer(th_h[a:b], th_ref, np.array([0, b - a]), "theta layer %d" % l)


def _sample_layers(cfg):
    sizes = np.diff(cfg.offsets)
    return sorted(set(list(range(0, cfg.h, 9)) + [int(np.argmax(sizes)), int(np.argmin(sizes)), cfg.h - 2, cfg.h - 1]))


def test_resnet50_per_worker_norms_sampled_layers(oracle):
    """dat_step on a plan with one quantizer norm per worker (Eq. grad_agg as written) at the bench size."""
    from paper_2206_06257_b200 import api, synth
    cfg = synth.config("resnet50")
    dev, step = "cuda", 1
    theta, mom = synth.make_params(cfg, device=dev)
    grads = synth.make_grads(cfg, step, device=dev)
    hp = hp_tuple(cfg)
    th0, mo0 = theta.clone(), mom.clone()
    sc = torch.zeros(cfg.M * cfg.h, dtype=torch.float32, device=dev)
    norms = torch.zeros(2 * cfg.h, dtype=torch.float32, device=dev)
    plan = api.dat_plan_create(cfg.offsets, cfg.M, cfg.bits, rng_bits=cfg.rng_bits, scale_mode=api.DAT_SCALE_PER_WORKER)
    try:
        api.dat_step(plan, theta, mom, grads, cfg.seed, step, hp, None, norms, sc)
        torch.cuda.synchronize()
        assert api.dat_get_status(plan) == 0
    finally:
        api.dat_plan_destroy(plan)
    offs, sc_h = cfg.offsets, np_of(sc)
    for l in _sample_layers(cfg):
        a, b = int(offs[l]), int(offs[l + 1])
        g_l = [np_of(g[a:b]) for g in grads]
        nu = oracle.worker_norms(offs, g_l, l0=l, l1=l + 1, window=True)
        assert ulp_diff(sc_h.reshape(cfg.M, cfg.h)[:, l], nu[:, l]).max() <= 1
        ref = oracle.step(offs, np_of(th0[a:b]), np_of(mo0[a:b]), g_l, cfg.bits, cfg.seed, step, *hp, l0=l, l1=l + 1,
                          window=True, scale_mode=oracle.SCALE_PER_WORKER, scales_in=sc_h, rng_bits=cfg.rng_bits)
        assert np.array_equal(np_of(mom[a:b]).view(np.uint32), ref["mom"].view(np.uint32)), "layer %d momentum" % l
        assert_close_per_layer(np_of(theta[a:b]), ref["theta"], np.array([0, b - a]), "theta layer %d" % l)


def test_resnet50_lamb_sampled_layers(oracle):
    """dat_step_lamb (Algorithm A2 in the one launch) at the bench size, t = 1 and t = 2 on one plan."""
    from paper_2206_06257_b200 import api, synth
    cfg = synth.config("resnet50")
    dev = "cuda"
    theta, mom = synth.make_params(cfg, device=dev)
    var = torch.zeros_like(mom)
    lamb_hp = (cfg.lr, 0.9, 0.999, 1e-6, 1e-4, cfg.c_l, cfg.c_u)
    sc = torch.zeros(cfg.h, dtype=torch.float32, device=dev)
    norms = torch.zeros(2 * cfg.h, dtype=torch.float32, device=dev)
    offs = cfg.offsets
    plan = api.dat_plan_create(cfg.offsets, cfg.M, cfg.bits, rng_bits=cfg.rng_bits)
    try:
        for t in (1, 2):
            grads = synth.make_grads(cfg, t, device=dev)
            th0, mo0, va0 = theta.clone(), mom.clone(), var.clone()
            api.dat_step_lamb(plan, theta, mom, var, grads, cfg.seed, t, lamb_hp, t, None, norms, sc)
            torch.cuda.synchronize()
            assert api.dat_get_status(plan) == 0
            sc_h, norms_h = np_of(sc), np_of(norms).reshape(-1, 2)
            for l in _sample_layers(cfg):
                a, b = int(offs[l]), int(offs[l + 1])
                g_l = [np_of(g[a:b]) for g in grads]
                nu = oracle.scales(oracle.worker_norms(offs, g_l, l0=l, l1=l + 1, window=True))
                assert ulp_diff(sc_h[l:l + 1], nu[l:l + 1]).max() <= 1
                level, neg = oracle.quantize(offs, g_l, cfg.bits, cfg.seed, t, sc_h, l0=l, l1=l + 1, window=True, rng_bits=cfg.rng_bits)
                _, gh = oracle.aggregate(offs, level, neg, sc_h, cfg.bits, l0=l, l1=l + 1, window=True)
                th_ref, mo_ref, va_ref, n_ref = oracle.lamb(np.array([0, b - a]), np_of(th0[a:b]), np_of(mo0[a:b]), np_of(va0[a:b]), gh, t, *lamb_hp)
                assert np.array_equal(np_of(mom[a:b]).view(np.uint32), mo_ref.view(np.uint32)), "layer %d m', t = %d" % (l, t)
                assert np.array_equal(np_of(var[a:b]).view(np.uint32), va_ref.view(np.uint32)), "layer %d v', t = %d" % (l, t)
                assert ulp_diff(norms_h[l], n_ref[0]).max() <= 1
                assert_close_per_layer(np_of(theta[a:b]), th_ref, np.array([0, b - a]), "theta layer %d, t = %d" % (l, t))
    finally:
        api.dat_plan_destroy(plan)
