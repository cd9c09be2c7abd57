"""dat_lalr_step_static: the LALR update for callers that cannot allocate device memory.

Some callers of this library run where cudaMalloc is off limits: inside an allocator's own
callbacks, in a process that handed out all device memory at start-up, or in a serving thread
that must never wait on the driver's allocation lock.  For them the library offers one entry
point that needs no plan and allocates nothing: its scratch lives in a fixed array inside the
library.  This test calls it through the C ABI and checks it against the plan-based
dat_lalr_step on the same inputs -- twice in a row, the second time on a smaller problem, so
that whatever the first call left in the shared scratch array must not leak into the second.

(The file name makes pytest collect it last: a run that stops at the first failure has then
already run every other test.)
"""
import numpy as np
import pytest
import torch

from helpers import REL_TOL, GpuPlan, assert_close_per_layer, np_of

pytestmark = pytest.mark.gpu

HP = (0.1, 0.9, 5e-4, 0.0, 10.0)


def _case(seed, sizes):
    rng = np.random.RandomState(seed)
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    d = int(offs[-1])
    theta = torch.from_numpy((rng.randn(d) * 0.05).astype(np.float32))
    mom = torch.from_numpy((rng.randn(d) * 1e-3).astype(np.float32))
    g_hat = torch.from_numpy((rng.randn(d) * 1e-2).astype(np.float32))
    return offs, theta, mom, g_hat


def _run_both(api, offs, theta, mom, g_hat, oracle=None, check_free=False):
    h = len(offs) - 1
    # existing entry point (plan-based)
    th_ref, mo_ref = theta.cuda(), mom.cuda()
    g_dev = g_hat.cuda()
    n_ref = torch.zeros(2 * h, dtype=torch.float32, device="cuda")
    with GpuPlan(api, offs, 1, 8) as P:
        api.dat_lalr_step(P.plan, th_ref, mo_ref, g_dev, HP, n_ref)
        torch.cuda.synchronize()
    # the entry point that allocates nothing: every buffer it touches is made here, before the call
    th_new, mo_new = theta.cuda(), mom.cuda()
    n_new = torch.zeros(2 * h, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    api.dat_lalr_step_static(offs, th_new, mo_new, g_dev, HP, n_new)
    torch.cuda.synchronize()
    if check_free:      # (not on a device's first call, which may load the kernels' code)
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
    assert_close_per_layer(np_of(th_new), np_of(th_ref), offs, "theta (static scratch)", REL_TOL)
    assert_close_per_layer(np_of(mo_new), np_of(mo_ref), offs, "mom (static scratch)", REL_TOL)
    assert np.allclose(np_of(n_new), np_of(n_ref), rtol=REL_TOL, atol=0)
    # the two run the same kernels, so in fact they agree bit for bit
    assert torch.equal(th_new, th_ref) and torch.equal(mo_new, mo_ref)
    if oracle is not None:          # and directly against the CPU oracle of the update
        th_o, mo_o, n_o = oracle.lalr(offs, np_of(theta), np_of(mom), np_of(g_hat), *HP)
        assert np.array_equal(np_of(mo_new).view(np.uint32), mo_o.view(np.uint32))
        assert_close_per_layer(np_of(th_new), th_o, offs, "theta (static scratch vs oracle)", REL_TOL)
        assert np.allclose(np_of(n_new).reshape(-1, 2), n_o, rtol=REL_TOL, atol=0)


def test_static_scratch_matches_plan_based_update_twice(oracle):
    assert torch.cuda.is_available()
    from paper_2206_06257_b200 import api
    # first call: many tiles, ragged layers, offsets that are not multiples of 4
    _run_both(api, *_case(1, [5, 70001, 4096, 33, 250007, 12289, 1]), oracle=oracle)
    # second call right after it: fewer layers and tiles than the scratch still remembers; and the
    # amount of free device memory must be the same before and after the call
    _run_both(api, *_case(2, [3000, 17, 9001]), oracle=oracle, check_free=True)


def test_static_scratch_accepts_exactly_its_limits():
    """As many layers as the scratch holds (one element each), and a layer that fills every tile."""
    from paper_2206_06257_b200 import api
    _run_both(api, *_case(3, [1] * api.DAT_STATIC_MAX_LAYERS))
    n = 4096 * api.DAT_STATIC_MAX_TILES
    th = torch.zeros(n, device="cuda")
    mo = torch.zeros(n, device="cuda")
    g = torch.ones(n, device="cuda")
    api.dat_lalr_step_static([0, n], th, mo, g, HP)         # exactly DAT_STATIC_MAX_TILES tiles
    torch.cuda.synchronize()
    assert torch.equal(mo, g) and not th.any()              # m' = g_hat; ||theta|| = 0 with c_l = 0: no move


def test_static_scratch_refuses_stream_capture():
    """The call copies its tables from host memory every time, so it must not end up in a CUDA graph."""
    from paper_2206_06257_b200 import api
    th, mo, gh = torch.zeros(64, device="cuda"), torch.zeros(64, device="cuda"), torch.ones(64, device="cuda")
    api.dat_lalr_step_static([0, 64], th, mo, gh, HP)          # (the device's first call, outside capture)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        g.capture_begin()
        try:
            gh.add_(0.0)                                        # something to capture
            with pytest.raises(api.DatError) as e:
                api.dat_lalr_step_static([0, 64], th, mo, gh, HP, stream=s)
            assert e.value.code == api.DAT_ERR_UNSUPPORTED
        finally:
            g.capture_end()
    torch.cuda.synchronize()


def test_static_scratch_refuses_what_does_not_fit():
    from paper_2206_06257_b200 import api
    th = torch.zeros(64, device="cuda")
    with pytest.raises(api.DatError) as e:                       # too many layers
        api.dat_lalr_step_static(np.arange(api.DAT_STATIC_MAX_LAYERS + 2), th, th, th, HP)
    assert e.value.code == api.DAT_ERR_TOO_LARGE
    with pytest.raises(api.DatError) as e:                       # too many tiles (nothing is touched)
        api.dat_lalr_step_static([0, 4096 * (api.DAT_STATIC_MAX_TILES + 1)], th, th, th, HP)
    assert e.value.code == api.DAT_ERR_TOO_LARGE
    with pytest.raises(api.DatError) as e:
        api.dat_lalr_step_static([0, 10, 10], th, th, th, HP)
    assert e.value.code == api.DAT_ERR_LAYOUT
