"""The three operations of the sharded step on the CPU oracle (test infrastructure): the same interface as
paper_2206_06257_b200.sharded.CudaOps, torch CPU tensors in and out."""
import numpy as np
import torch

import oracle


class OracleOps:
    def __init__(self, offsets, M, M_loc, rank, world, bits, rng_bits=16):
        self.offsets = np.asarray(offsets, dtype=np.int64)
        self.h = self.offsets.size - 1
        self.M, self.M_loc, self.rank, self.bits, self.rng_bits = M, M_loc, rank, bits, rng_bits

    def plane_bytes(self, rg):
        return oracle.level_plane_bytes(rg.n, self.bits), oracle.sign_plane_bytes(rg.n)

    def worker_norms(self, grads_local):
        return torch.from_numpy(oracle.worker_norms(self.offsets, [g.numpy() for g in grads_local])).view(self.M_loc, self.h)

    def quantize_range(self, q, rg, grads_local, scales, seed, step):
        nu = np.zeros(self.h, dtype=np.float32)
        nu[rg.l0:rg.l1] = scales.numpy()[-(rg.l1 - rg.l0):]
        lvs, sgs = [], []
        for i, g in enumerate(grads_local):
            # worker i of this rank is worker rank*M_loc + i of the whole problem: its random stream has that index
            _, _, level, neg = oracle.requantize(self.offsets, g.numpy(), self.bits, seed, step, self.rank * self.M_loc + i,
                                                 rng_bits=self.rng_bits, scales_in=nu)
            lev = np.zeros(rg.n, dtype=np.uint32)
            ng = np.zeros(rg.n, dtype=np.uint8)
            lev[rg.pad:], ng[rg.pad:] = level[rg.a:rg.b], neg[rg.a:rg.b]
            lp, sp = oracle.pack(lev, ng, self.bits)
            lvs.append(lp)
            sgs.append(sp)
        return torch.from_numpy(np.concatenate(lvs)), torch.from_numpy(np.concatenate(sgs))

    def aggregate_update(self, rg, lv_all, sg_all, scales, theta_own, mom_own, hp):
        lb, sb = self.plane_bytes(rg)
        level = np.zeros((self.M, rg.n), dtype=np.uint32)
        neg = np.zeros((self.M, rg.n), dtype=np.uint8)
        for i in range(self.M):
            level[i], neg[i] = oracle.unpack(lv_all.numpy()[i * lb:(i + 1) * lb], sg_all.numpy()[i * sb:(i + 1) * sb], rg.n, self.bits)
        _, g_hat = oracle.aggregate(rg.offsets, level, neg, scales.numpy(), self.bits)
        th, mo, _ = oracle.lalr(rg.offsets, theta_own.numpy(), mom_own.numpy(), g_hat, *hp)
        theta_own.copy_(torch.from_numpy(th))
        mom_own.copy_(torch.from_numpy(mo))
