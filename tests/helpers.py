"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding and the
oracle on the same seeded inputs, and compare."""
import numpy as np
import torch

REL_TOL = 1e-5      # tolerance on updated parameters and momentum (fp32)


def ulp_diff(a, b):
    """Distance in units in the last place between two float32 arrays of like sign."""
    ai = np.asarray(a, dtype=np.float32).view(np.int32).astype(np.int64)
    bi = np.asarray(b, dtype=np.float32).view(np.int32).astype(np.int64)
    return np.abs(ai - bi)


def assert_close_per_layer(got, ref, offsets, what, rel=REL_TOL):
    """|got - ref| <= rel*|ref| + rel*rms(ref_l) for every element of every layer."""
    got = np.asarray(got, dtype=np.float64)
    ref64 = np.asarray(ref, dtype=np.float64)
    assert np.isfinite(got).all(), what + ": non-finite values"
    for l in range(len(offsets) - 1):
        sl = slice(int(offsets[l]), int(offsets[l + 1]))
        r = ref64[sl]
        rms = np.sqrt(np.mean(r * r))
        bad = np.abs(got[sl] - r) > rel * np.abs(r) + rel * rms
        assert not bad.any(), "%s: layer %d: %d of %d elements off (max abs diff %.3e, rms %.3e)" % (
            what, l, int(bad.sum()), r.size, float(np.abs(got[sl] - r).max()), rms)


def hp_tuple(cfg):
    return (cfg.lr, cfg.momentum, cfg.weight_decay, cfg.c_l, cfg.c_u)


def to_dev(ts):
    return [t.cuda() for t in ts]


def np_of(t):
    return t.detach().cpu().numpy()


class GpuPlan:
    """Plan + the caller-owned buffers of the unfused calls."""

    def __init__(self, api, offsets, M, bits, rng_bits=16, scale_mode=0):
        self.api = api
        self.offsets = np.asarray(offsets, dtype=np.int64)
        self.M, self.bits = M, bits
        self.h = len(self.offsets) - 1
        self.d = int(self.offsets[-1])
        self.plan = api.dat_plan_create(self.offsets, M, bits, scale_mode=scale_mode, rng_bits=rng_bits)
        self.level_bytes, self.sign_bytes, self.num_scales, self.ws = api.dat_plan_sizes(self.plan)

    def close(self):
        if self.plan:
            self.api.dat_plan_destroy(self.plan)
            self.plan = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def alloc_message(self):
        lv = torch.full((self.M * self.level_bytes,), 0xAB, dtype=torch.uint8, device="cuda")
        sg = torch.full((self.M * self.sign_bytes,), 0xCD, dtype=torch.uint8, device="cuda")
        sc = torch.zeros(self.num_scales, dtype=torch.float32, device="cuda")
        return lv, sg, sc

    def status(self):
        return self.api.dat_get_status(self.plan)


def oracle_planes(oracle, level, neg, bits):
    """Pack the oracle's per-worker codes into (M, level_bytes) and (M, sign_bytes) uint8."""
    lps, sps = [], []
    for i in range(level.shape[0]):
        lp, sp = oracle.pack(level[i], neg[i], bits)
        lps.append(lp)
        sps.append(sp)
    return np.stack(lps), np.stack(sps)
