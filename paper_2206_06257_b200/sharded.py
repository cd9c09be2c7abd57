"""The step sharded over several GPUs of one node (one process per GPU, torch.distributed).

The paper's own deployment is data-parallel training with one-sided quantisation: every worker
quantizes its gradient (Algorithm A1 Step 7), the quantized messages are exchanged, summed and
de-quantised (Step 9), and every machine applies the update (Step 12).  Here:

  * rank r holds the gradients of the workers r*M/G .. (r+1)*M/G - 1 (the whole vector each) and OWNS a
    contiguous range of layers (ranges balanced by element count), with the momentum of that range;
  * the shared quantizer norm nu_l = max_i ||g_l^(i)||_2 is agreed by one all-reduce(max) of h floats;
  * every rank quantizes its workers' gradients range by range and sends the packed level and sign
    planes of range q to its owner (plain point-to-point sends into the owner's OWN buffers);
  * the owner sums the M workers' codes of its range as integers, de-quantises, and applies the
    layer-wise update to its range of theta and m (all layer norms are local to the owner);
  * the updated ranges of theta are broadcast by their owners.

Two forms of the exchange: "sendrecv" (above), and "pull": every rank leaves its planes in a buffer of its own
that the other ranks have mapped (symmetric memory), and the owner's aggregation kernel reads the M workers'
planes of its range from where they lie -- its own memory and the peers' -- with plain loads
(dat_aggregate_gather): exchange and Step 9 in one kernel, nothing is sent.

Only the orchestration lives here; the arithmetic is done by an `ops` object -- `CudaOps` below calls
the CUDA library through the C ABI (dat_worker_norms, dat_quantize with caller-supplied norms,
dat_aggregate, dat_lalr_step on plans that cover one range each, with dat_plan_set_origin giving the
range's place in the global random streams), so the result is the one the unsharded dat_step gives.
"""
import numpy as np
import torch
import torch.distributed as dist


def partition_layers(offsets, world):
    """Contiguous layer ranges [(l0, l1)] for `world` owners, balanced by element count; every owner gets
    at least one layer (h >= world is required)."""
    offs = np.asarray(offsets, dtype=np.int64)
    h = offs.size - 1
    if h < world:
        raise ValueError("fewer layers (%d) than ranks (%d)" % (h, world))
    d = int(offs[-1])
    cuts = [0]
    for r in range(1, world):
        target = d * r / world
        l = int(np.searchsorted(offs, target, side="left"))          # first layer boundary at or after the target
        if l > 0 and target - offs[l - 1] < offs[l] - target:
            l -= 1                                                      # (the nearer boundary)
        l = min(max(l, cuts[-1] + 1), h - (world - r))                  # at least one layer here and for every later owner
        cuts.append(l)
    cuts.append(h)
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


class RangeLayout:
    """One owner's range as a problem of its own: elements [a8, b) of the flat vector, where a8 is the
    range's first element rounded down to a multiple of 8 (the random streams are drawn in blocks of 4 or 8
    consecutive elements, so a slice must start on such a boundary).  If a8 < a, the elements in between
    form a pad layer in front (they belong to the previous owner; whatever is computed for them is dropped)."""

    def __init__(self, offsets, l0, l1):
        offs = np.asarray(offsets, dtype=np.int64)
        self.l0, self.l1 = l0, l1
        self.a, self.b = int(offs[l0]), int(offs[l1])
        self.a8 = self.a & ~7
        self.pad = self.a - self.a8
        local = offs[l0:l1 + 1] - self.a8
        self.offsets = np.concatenate([[0], local]).astype(np.int64) if self.pad else local.astype(np.int64)
        self.n = self.b - self.a8                     # elements of the sub-problem (pad included)
        self.h = self.offsets.size - 1

    def scales(self, nu):
        """The sub-problem's norms from the global per-layer norms (the pad layer gets 1)."""
        own = nu[self.l0:self.l1]
        return torch.cat([torch.ones(1, dtype=own.dtype, device=own.device), own]) if self.pad else own.clone()


class ShardedStep:
    """One rank's side of the sharded step.  ops: see CudaOps.  All tensors are torch tensors on the ops' device."""

    def __init__(self, ops, offsets, M, rank, world, group=None):
        if M % world:
            raise ValueError("the workers (%d) must divide evenly over the ranks (%d)" % (M, world))
        self.ops, self.rank, self.world, self.group = ops, rank, world, group
        self.offsets = np.asarray(offsets, dtype=np.int64)
        self.M, self.M_loc = M, M // world
        self.ranges = [RangeLayout(self.offsets, l0, l1) for (l0, l1) in partition_layers(self.offsets, world)]
        self.own = self.ranges[rank]

    # The step in four phases, so that a test can drive several ranks' objects in one process (on one GPU)
    # by handing the messages over itself; step() below drives them with torch.distributed.
    def local_norms(self, grads_local):
        """Step 7, first half: max over this rank's workers of ||g_l^(i)||_2, per layer."""
        return self.ops.worker_norms(grads_local).max(dim=0).values.contiguous()

    def quantize(self, nu, grads_local, seed, step):
        """Step 7, second half: this rank's workers, range by range.  Returns [(levels, signs)] per owner."""
        return [self.ops.quantize_range(q, self.ranges[q], grads_local, self.ranges[q].scales(nu), seed, step)
                for q in range(self.world)]

    def receive_buffers(self, device):
        lb, sb = self.ops.plane_bytes(self.own)
        return (torch.empty(self.M * lb, dtype=torch.uint8, device=device),
                torch.empty(self.M * sb, dtype=torch.uint8, device=device))

    def slot(self, lv_all, sg_all, src):
        """Where the planes of rank `src`'s workers go in the owner's buffers (global worker order: rank-major)."""
        lb, sb = lv_all.numel() // self.M, sg_all.numel() // self.M
        return (lv_all[src * self.M_loc * lb:(src + 1) * self.M_loc * lb],
                sg_all[src * self.M_loc * sb:(src + 1) * self.M_loc * sb])

    def update(self, nu, lv_all, sg_all, theta, mom_own, hp):
        """Steps 9 and 12 on the owned range; theta[a:b] is rewritten."""
        own = self.own
        theta_own = theta[own.a8:own.b].clone()          # (private copy: the pad elements are another owner's)
        self.ops.aggregate_update(own, lv_all, sg_all, own.scales(nu), theta_own, mom_own, hp)
        theta[own.a:own.b].copy_(theta_own[own.pad:])

    def update_pull(self, nu, planes_by_src, theta, mom_own, hp):
        """Steps 9 and 12 on the owned range, the planes read where the ranks left them: planes_by_src[src] =
        (levels, signs) of rank src's M/G workers for THIS rank's range (tensors, or base addresses of mapped
        peer memory)."""
        own = self.own
        lb, sb = self.ops.plane_bytes(own)
        lv_ptrs, sg_ptrs = [], []
        for src in range(self.world):
            lv, sg = planes_by_src[src]
            lv0 = lv.data_ptr() if isinstance(lv, torch.Tensor) else int(lv)
            sg0 = sg.data_ptr() if isinstance(sg, torch.Tensor) else int(sg)
            lv_ptrs += [lv0 + j * lb for j in range(self.M_loc)]         # global worker order: rank-major
            sg_ptrs += [sg0 + j * sb for j in range(self.M_loc)]
        theta_own = theta[own.a8:own.b].clone()
        self.ops.aggregate_update_gather(own, lv_ptrs, sg_ptrs, own.scales(nu), theta_own, mom_own, hp)
        theta[own.a:own.b].copy_(theta_own[own.pad:])

    def _pull_layout(self):
        """Byte offsets, in every rank's outgoing buffer, of the level and sign planes meant for owner q."""
        offs, at = [], 0
        for q in range(self.world):
            lb, sb = self.ops.plane_bytes(self.ranges[q])
            offs.append((at, at + self.M_loc * lb))
            at += self.M_loc * (lb + sb)                                  # (plane sizes are multiples of 16 bytes)
        return offs, at

    def step_pull(self, theta, mom_own, grads_local, seed, step, hp):
        """The step with the "pull" exchange.  Needs CUDA ranks of one node with peer access.  Not run on more
        than one GPU so far (one-GPU environment): the kernel path is covered by driving several ranks' objects
        in one process, the mapping of the peers' buffers is not."""
        layout, total = self._pull_layout()
        multi = self.world > 1
        if getattr(self, "_out", None) is None:
            if multi:
                import os
                os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")    # plain peer mappings, no NVLink multicast object
                import torch.distributed._symmetric_memory as symm_mem
                self._out = symm_mem.empty(total, dtype=torch.uint8, device=theta.device)
                hdl = symm_mem.rendezvous(self._out, self.group if self.group is not None else dist.group.WORLD)
                self._bases = [int(p) for p in hdl.buffer_ptrs]
            else:
                self._out = torch.empty(total, dtype=torch.uint8, device=theta.device)
                self._bases = [self._out.data_ptr()]
        nu = self.local_norms(grads_local)
        if multi:
            dist.all_reduce(nu, op=dist.ReduceOp.MAX, group=self.group)
        for q in range(self.world):
            lb, sb = self.ops.plane_bytes(self.ranges[q])
            lo, so = layout[q]
            self.ops.quantize_range(q, self.ranges[q], grads_local, self.ranges[q].scales(nu), seed, step,
                                    out=(self._out[lo:lo + self.M_loc * lb], self._out[so:so + self.M_loc * sb]))
        if multi:
            torch.cuda.current_stream().synchronize()
            dist.barrier(group=self.group)                                # every rank's planes are complete
        lo, so = layout[self.rank]
        self.update_pull(nu, [(b + lo, b + so) for b in self._bases], theta, mom_own, hp)
        if multi:
            torch.cuda.current_stream().synchronize()
            dist.barrier(group=self.group)                                # nobody rewrites planes that are still being read
            for r, rg in enumerate(self.ranges):
                dist.broadcast(theta[rg.a:rg.b], src=r, group=self.group)
        return nu

    def step(self, theta, mom_own, grads_local, seed, step, hp):
        """theta: the full parameter vector (updated in place on every rank); mom_own: the momentum of this
        rank's range, own.n elements with the pad in front (updated in place); grads_local: this rank's
        M/G gradient vectors."""
        nu = self.local_norms(grads_local)
        if self.world > 1:
            dist.all_reduce(nu, op=dist.ReduceOp.MAX, group=self.group)
        mine = self.quantize(nu, grads_local, seed, step)
        lv_all, sg_all = self.receive_buffers(nu.device)
        reqs = []
        for src in range(self.world):
            lv_dst, sg_dst = self.slot(lv_all, sg_all, src)
            if src == self.rank:
                lv_dst.copy_(mine[src][0])
                sg_dst.copy_(mine[src][1])
            else:       # plain point-to-point receives into this rank's own buffers
                reqs += [dist.P2POp(dist.irecv, lv_dst, src, self.group), dist.P2POp(dist.irecv, sg_dst, src, self.group)]
        for q in range(self.world):
            if q != self.rank:
                reqs += [dist.P2POp(dist.isend, mine[q][0], q, self.group), dist.P2POp(dist.isend, mine[q][1], q, self.group)]
        if reqs:
            for w in dist.batch_isend_irecv(reqs):
                w.wait()
        self.update(nu, lv_all, sg_all, theta, mom_own, hp)
        if self.world > 1:      # every owner's range of theta to everybody
            for r, rg in enumerate(self.ranges):
                dist.broadcast(theta[rg.a:rg.b], src=r, group=self.group)
        return nu


class CudaOps:
    """The three operations of the sharded step on the CUDA library (through the C-ABI binding)."""

    def __init__(self, api, offsets, M, M_loc, rank, world, bits, rng_bits=16):
        self.api, self.M, self.M_loc, self.rank = api, M, M_loc, rank
        self.offsets = np.asarray(offsets, dtype=np.int64)
        self.h = self.offsets.size - 1
        self.bits, self.rng_bits = bits, rng_bits
        self.plan_norms = api.dat_plan_create(self.offsets, M_loc, bits, rng_bits=rng_bits)
        self.plans_q, self.plans_agg = {}, {}

    def close(self):
        for p in [self.plan_norms] + list(self.plans_q.values()) + list(self.plans_agg.values()):
            self.api.dat_plan_destroy(p)
        self.plans_q, self.plans_agg, self.plan_norms = {}, {}, None

    def _plan(self, table, rg, workers, worker_base):
        key = (rg.l0, rg.l1)
        if key not in table:
            p = self.api.dat_plan_create(rg.offsets, workers, self.bits, rng_bits=self.rng_bits)
            self.api.dat_plan_set_origin(p, rg.a8, worker_base)
            table[key] = p
        return table[key]

    def plane_bytes(self, rg):
        lb, sb, _, _ = self.api.dat_plan_sizes(self._plan(self.plans_agg, rg, self.M, 0))
        return lb, sb

    def worker_norms(self, grads_local):
        out = torch.empty(self.M_loc * self.h, dtype=torch.float32, device=grads_local[0].device)
        self.api.dat_worker_norms(self.plan_norms, grads_local, out)
        return out.view(self.M_loc, self.h)

    def quantize_range(self, q, rg, grads_local, scales, seed, step, out=None):
        plan = self._plan(self.plans_q, rg, self.M_loc, self.rank * self.M_loc)
        lb, sb, ns, _ = self.api.dat_plan_sizes(plan)
        dev = grads_local[0].device
        lv, sg = out if out is not None else (torch.empty(self.M_loc * lb, dtype=torch.uint8, device=dev),
                                              torch.empty(self.M_loc * sb, dtype=torch.uint8, device=dev))
        sc = torch.empty(ns, dtype=torch.float32, device=dev)
        self.api.dat_quantize(plan, [g[rg.a8:rg.b] for g in grads_local], seed, step, lv, sg, sc, scales_in=scales.contiguous())
        return lv, sg

    def aggregate_update_gather(self, rg, lv_ptrs, sg_ptrs, scales, theta_own, mom_own, hp):
        plan = self._plan(self.plans_agg, rg, self.M, 0)
        g_hat = torch.empty(rg.n, dtype=torch.float32, device=theta_own.device)
        self.api.dat_aggregate_gather(plan, lv_ptrs, sg_ptrs, scales.contiguous(), None, g_hat)
        self.api.dat_lalr_step(plan, theta_own, mom_own, g_hat, hp)

    def aggregate_update(self, rg, lv_all, sg_all, scales, theta_own, mom_own, hp):
        plan = self._plan(self.plans_agg, rg, self.M, 0)
        g_hat = torch.empty(rg.n, dtype=torch.float32, device=theta_own.device)
        self.api.dat_aggregate(plan, lv_all, sg_all, scales.contiguous(), None, g_hat)
        self.api.dat_lalr_step(plan, theta_own, mom_own, g_hat, hp)
