"""The sharded step (paper_2206_06257_b200/sharded.py): layer ranges owned by ranks, the shared norm agreed
by an all-reduce, packed planes sent to the owners, the update on the owned range, theta broadcast.

On CPU: two and three gloo ranks on 127.0.0.1 run the orchestration on the oracle's operations and the
gathered parameters must equal the oracle's unsharded step bit for bit (momentum of every owned range too).
On a GPU: the CUDA operations with two and four ranks' objects driven in ONE process on one device (the
messages are handed over by the test; no kernel waits for another), against the oracle and against dat_step."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HP = (0.1, 0.9, 5e-4, 0.0, 10.0)
SIZES = [5, 70001, 4096, 33, 25007, 12289, 1, 9000, 64, 20011, 3]      # ranges that do not start on multiples of 8


def _problem(seed, M):
    rng = np.random.RandomState(seed)
    offs = np.concatenate([[0], np.cumsum(SIZES)]).astype(np.int64)
    d = int(offs[-1])
    sig = np.repeat(10.0 ** rng.uniform(-4, -1, size=len(SIZES)), SIZES)
    grads = [(rng.randn(d) * sig).astype(np.float32) for _ in range(M)]
    theta = (rng.randn(d) * 0.05).astype(np.float32)
    mom = (rng.randn(d) * 1e-3).astype(np.float32)
    return offs, grads, theta, mom


def test_partition_is_contiguous_balanced_and_complete():
    sys.path.insert(0, ROOT)
    from paper_2206_06257_b200.sharded import RangeLayout, partition_layers
    offs = np.concatenate([[0], np.cumsum(SIZES)]).astype(np.int64)
    for world in (1, 2, 3, 4, len(SIZES)):
        parts = partition_layers(offs, world)
        assert parts[0][0] == 0 and parts[-1][1] == len(SIZES)
        assert all(parts[r][1] == parts[r + 1][0] for r in range(world - 1))
        assert all(l1 > l0 for l0, l1 in parts)
        for l0, l1 in parts:
            rg = RangeLayout(offs, l0, l1)
            assert rg.a8 % 8 == 0 and 0 <= rg.pad < 8 and rg.offsets[0] == 0 and rg.offsets[-1] == rg.n
            assert np.all(np.diff(rg.offsets) > 0)
    big = partition_layers(offs, 2)
    assert abs(offs[big[0][1]] - offs[-1] / 2) <= max(SIZES)       # the cut is at the boundary nearest to the middle
    with pytest.raises(ValueError):
        partition_layers(offs, len(SIZES) + 1)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank(rank, world, port, M, bits, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from paper_2206_06257_b200.sharded import ShardedStep
    from sharded_oracle_ops import OracleOps
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    offs, grads, theta, mom = _problem(5, M)
    M_loc = M // world
    st = ShardedStep(OracleOps(offs, M, M_loc, rank, world, bits), offs, M, rank, world)
    own = st.own
    th = torch.from_numpy(theta.copy())
    mo_own = torch.from_numpy(mom[own.a8:own.b].copy())
    g_loc = [torch.from_numpy(grads[rank * M_loc + i]) for i in range(M_loc)]
    for t in range(2):                                  # two consecutive steps on the evolving state
        st.step(th, mo_own, g_loc, 11, t, HP)
    out.put((rank, th.numpy().copy(), own.a, own.b, mo_own.numpy()[own.pad:].copy()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,M,bits", [(2, 4, 8), (3, 6, 4)])
def test_sharded_step_on_gloo_ranks_equals_the_unsharded_oracle(oracle, world, M, bits):
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, world, port, M, bits, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((out.get(timeout=300) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    offs, grads, theta, mom = _problem(5, M)
    ref_th, ref_mo = theta, mom
    for t in range(2):
        ref = oracle.step(offs, ref_th, ref_mo, grads, bits, 11, t, *HP)
        ref_th, ref_mo = ref["theta"], ref["mom"]
    for rank, th, a, b, mo in res:
        assert np.array_equal(th.view(np.uint32), ref_th.view(np.uint32)), "rank %d: gathered parameters" % rank
        assert np.array_equal(mo.view(np.uint32), ref_mo[a:b].view(np.uint32)), "rank %d: momentum of its range" % rank


@pytest.mark.gpu
@pytest.mark.parametrize("exchange", ["sendrecv", "pull"])
@pytest.mark.parametrize("world,M,bits", [(2, 4, 8), (4, 8, 2)])
def test_sharded_step_cuda_ops_in_one_process(oracle, world, M, bits, exchange):
    """The CUDA operations of the sharded step: `world` ranks' objects on one device, driven phase by phase."""
    sys.path.insert(0, ROOT)
    from paper_2206_06257_b200 import api
    from paper_2206_06257_b200.sharded import CudaOps, ShardedStep
    from helpers import assert_close_per_layer, np_of
    offs, grads, theta, mom = _problem(6, M)
    M_loc = M // world
    ops = [CudaOps(api, offs, M, M_loc, r, world, bits) for r in range(world)]
    try:
        ranks = [ShardedStep(ops[r], offs, M, r, world) for r in range(world)]
        th = [torch.from_numpy(theta.copy()).cuda() for _ in range(world)]
        mo = [torch.from_numpy(mom[s.own.a8:s.own.b].copy()).cuda() for s in ranks]
        g = [[torch.from_numpy(grads[r * M_loc + i]).cuda() for i in range(M_loc)] for r in range(world)]
        nus = [s.local_norms(g[r]) for r, s in enumerate(ranks)]
        nu = torch.stack(nus).max(dim=0).values                          # the all-reduce(max)
        planes = [s.quantize(nu, g[r], 11, 3) for r, s in enumerate(ranks)]
        for r, s in enumerate(ranks):
            if exchange == "pull":      # the owner's kernel reads every rank's planes where that rank left them
                s.update_pull(nu, [planes[src][r] for src in range(world)], th[r], mo[r], HP)
                continue
            lv_all, sg_all = s.receive_buffers(nu.device)
            for src in range(world):                                     # the point-to-point exchange
                lv_dst, sg_dst = s.slot(lv_all, sg_all, src)
                lv_dst.copy_(planes[src][r][0])
                sg_dst.copy_(planes[src][r][1])
            s.update(nu, lv_all, sg_all, th[r], mo[r], HP)
        full = torch.from_numpy(theta.copy()).cuda()
        for r, s in enumerate(ranks):                                    # the broadcasts
            full[s.own.a:s.own.b] = th[r][s.own.a:s.own.b]
        torch.cuda.synchronize()
        nu_h = np_of(nu)
        ref = oracle.step(offs, theta, mom, grads, bits, 11, 3, *HP, scales_in=nu_h)
        assert np.abs(nu_h.view(np.int32).astype(np.int64) - oracle.scales(oracle.worker_norms(offs, grads)).view(np.int32)).max() <= 1
        for r, s in enumerate(ranks):
            assert np.array_equal(np_of(mo[r])[s.own.pad:].view(np.uint32), ref["mom"][s.own.a:s.own.b].view(np.uint32))
        assert_close_per_layer(np_of(full), ref["theta"], offs, "theta (sharded, CUDA operations)")
        # and the unsharded one-call step gives the same momentum bit for bit
        with __import__("helpers").GpuPlan(api, offs, M, bits) as P:
            th1, mo1 = torch.from_numpy(theta.copy()).cuda(), torch.from_numpy(mom.copy()).cuda()
            api.dat_step(P.plan, th1, mo1, [t for row in g for t in row], 11, 3, HP)
            torch.cuda.synchronize()
        for r, s in enumerate(ranks):
            assert torch.equal(mo[r][s.own.pad:], mo1[s.own.a:s.own.b])
        assert_close_per_layer(np_of(full), np_of(th1), offs, "theta (sharded vs dat_step)")
    finally:
        for o in ops:
            o.close()
