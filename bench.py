#!/usr/bin/env python
"""Benchmark of the fused DAT outer-minimisation step (quantize + aggregate + LALR).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config resnet50] [--impl reference]

One "step" is one pass of the whole hot path (dat_step) over one batch of synthetic input:
the M worker gradient buffers, parameters and momentum of the chosen workload, resident in HBM.
Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an independent replica
of the workload on its own GPU (the path has no exchange step on one node: replicas only);
the time is the maximum over ranks and the value the sum of all ranks' elements.

--impl reference times the CPU oracle (the only reference implementation that exists for this
path) on the host cores, on a bounded sample of the same workload.
"""
import argparse
import json
import os
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "worker-grad elems/s through quantize+aggregate+LALR"
UNIT = "elems/s"
NOMINAL_HBM_GBS = 8000.0
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "traffic.json")


def kernel_source_hash():
    """sha256 over the CUDA sources of the library (what the ncu traffic figures are keyed by)."""
    import hashlib
    csrc = os.path.join(ROOT, "paper_2206_06257_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")):
            h.update(name.encode())
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic(path, cfg):
    """DRAM bytes per step from the ncu capture summarised under profiles/ -- or None when no capture
    exists for this path and workload, or when the kernels have changed since it was taken."""
    try:
        table = json.load(open(TRAFFIC_JSON))
    except Exception:
        return None, None
    key = "%s:%s_m%d_b%d_rng%d" % (path, cfg.name, cfg.M, cfg.bits, cfg.rng_bits)
    rec = table.get(key)
    if not rec or rec.get("source_hash") != kernel_source_hash():
        return None, None
    return int(rec["dram_bytes_per_step"]), rec.get("summary")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


# ------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, device_index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:          # no NVML: report that, do not fail the benchmark
            self.err = repr(e)
            self.h = None

    def sample(self):
        if self.h is None:
            return
        try:
            self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
            try:
                r = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                r = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            for bit, name in self.REASONS.items():
                if r & bit and name != "gpu_idle":
                    self.reasons.add(name)
        except Exception:
            pass

    def start(self):
        if self.h is None:
            return
        def loop():
            while not self._stop.is_set():
                self.sample()
                time.sleep(0.01)
        self._thread = threading.Thread(target=loop, daemon=True)
        self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()
        return {"sm_mhz": int(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------
def oracle_layer_sample(cfg, max_worker_elems):
    """A prefix-free sample of layers: every k-th layer, largest stride that keeps the sample
    below max_worker_elems (whole workload if it fits)."""
    sizes = np.diff(cfg.offsets)
    total = int(sizes.sum()) * cfg.M
    if total <= max_worker_elems:
        return list(range(cfg.h)), "whole workload (%d layers, %.3g worker-elems)" % (cfg.h, total)
    stride = 1
    while True:
        stride += 1
        idx = list(range(0, cfg.h, stride))
        n = int(sizes[idx].sum()) * cfg.M
        if n <= max_worker_elems or stride >= cfg.h:
            return idx, "every %d-th layer of the workload (%d of %d layers, %.3g of %.3g worker-elems)" % (
                stride, len(idx), cfg.h, n, total)


def time_oracle(cfg, theta, mom, grads, layers, threads, step=0):
    """One oracle step restricted to `layers` (numpy inputs).  Returns (seconds, worker_elems)."""
    import oracle
    offs = cfg.offsets
    hp = (cfg.lr, cfg.momentum, cfg.weight_decay, cfg.c_l, cfg.c_u)

    def run(l):
        a, b = int(offs[l]), int(offs[l + 1])
        oracle.step(offs, theta[a:b], mom[a:b], [g[a:b] for g in grads], cfg.bits, cfg.seed, step, *hp,
                    l0=l, l1=l + 1, window=True, want_code_sum=False, rng_bits=cfg.rng_bits)
        return (b - a) * cfg.M
    order = sorted(layers, key=lambda l: -(offs[l + 1] - offs[l]))     # big layers first
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        n = sum(ex.map(run, order))
    return time.perf_counter() - t0, n


def host_threads():
    try:
        n = len(os.sched_getaffinity(0))
    except Exception:
        n = os.cpu_count() or 1
    return max(1, min(n, 32))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    from paper_2206_06257_b200 import synth
    oracle.lib()
    cfg = synth.config(args.config)
    theta, mom = synth.make_params(cfg)
    grads = [g.numpy() for g in synth.make_grads(cfg, 0)]
    theta, mom = theta.numpy(), mom.numpy()
    threads = host_threads()
    # calibrate on a small sample, then size each step for a run of a few minutes at most
    cal_layers, _ = oracle_layer_sample(cfg, 4_000_000)
    t_cal, n_cal = time_oracle(cfg, theta, mom, grads, cal_layers, threads)
    rate = n_cal / t_cal
    budget_s = 150.0 / max(1, args.steps + args.warmup)
    layers, what = oracle_layer_sample(cfg, max(2_000_000, int(rate * min(budget_s, 20.0))))
    for w in range(args.warmup):
        time_oracle(cfg, theta, mom, grads, layers, threads, step=w)
    t_tot, n_tot = 0.0, 0
    for k in range(args.steps):
        t, n = time_oracle(cfg, theta, mom, grads, layers, threads, step=k)
        t_tot += t
        n_tot += n
    value = n_tot / t_tot
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(cfg, "n/a (host)"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def max_over_ranks(value, world, device):
    """Maximum of a per-rank scalar over all ranks (the slowest rank sets the job's time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world, elems_per_step, steps, seconds):
    """Whole-job throughput of `world` independent replicas that all took `seconds` (the maximum)."""
    return world * elems_per_step * steps / seconds


def workload_config(cfg, l2_note):
    return {"workload": cfg.name, "d": cfg.d, "layers": cfg.h, "workers_M": cfg.M, "bits": cfg.bits, "rng_bits": cfg.rng_bits,
            "lr": cfg.lr, "momentum": cfg.momentum, "weight_decay": cfg.weight_decay,
            "grad_dist": cfg.grad_dist, "parallelism": "replicas", "l2": l2_note}


# ------------------------------------------------------------------------------------------
def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2206_06257_b200 import api, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for this path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg = synth.config(args.config)
    if args.bits:
        cfg.bits = args.bits
    if args.rng_bits:
        cfg.rng_bits = args.rng_bits
    theta, mom = synth.make_params(cfg, device=dev)
    grads = synth.make_grads(cfg, 0, device=dev)
    hp = (cfg.lr, cfg.momentum, cfg.weight_decay, cfg.c_l, cfg.c_u)
    variant = args.path.split("_", 1)[1] if args.path.startswith(("unfused_", "step_")) else ""
    plan = api.dat_plan_create(cfg.offsets, cfg.M, cfg.bits, rng_bits=cfg.rng_bits,
                               scale_mode=api.DAT_SCALE_PER_WORKER if variant == "per_worker" else api.DAT_SCALE_SHARED_MAX)
    stream = torch.cuda.current_stream()
    working_set = (cfg.M + 2) * cfg.d * 4
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    l2_note = ("inputs larger than L2 (%.0f MB touched per step vs %.0f MB L2), no flush" %
               (working_set / 1e6, l2_bytes / 1e6))
    flush = None
    if working_set < 2 * l2_bytes:       # cache-resident workload: flush L2 between timed steps
        flush = torch.empty(int(2.5 * l2_bytes) // 4, dtype=torch.float32, device=dev)
        l2_note = "L2 flushed between timed steps (%.0f MB buffer written)" % (flush.numel() * 4 / 1e6)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    unfused = args.path.startswith("unfused")
    if unfused:
        if cfg.bits == 32:
            raise SystemExit("--path unfused needs a quantized configuration (bits < 32)")
        lb, sb, ns, _ = api.dat_plan_sizes(plan)
        u_levels = torch.empty(cfg.M * lb, dtype=torch.uint8, device=dev)
        u_signs = torch.empty(cfg.M * sb, dtype=torch.uint8, device=dev)
        u_scales = torch.empty(ns, dtype=torch.float32, device=dev)
        u_ghat = torch.empty(cfg.d, dtype=torch.float32, device=dev)
        if variant == "two_sided":      # the server's own message (Algorithm A1 Step 10)
            s_levels = torch.empty(lb, dtype=torch.uint8, device=dev)
            s_signs = torch.empty(sb, dtype=torch.uint8, device=dev)
            s_scales = torch.empty(cfg.h, dtype=torch.float32, device=dev)
    if args.path == "step_two_sided":   # workspace for the aggregate / the receiver's value (Algorithm A1 Step 10)
        ts_ghat = torch.empty(cfg.d, dtype=torch.float32, device=dev)
    if variant == "lamb":               # Algorithm A2: second moment, the paper's ImageNet hyper-parameters
        var = torch.zeros(cfg.d, dtype=torch.float32, device=dev)
        lamb_hp = (cfg.lr, 0.9, 0.999, 1e-6, 1e-4, cfg.c_l, cfg.c_u)

    def one_step(step_index):
        if unfused:
            api.dat_quantize(plan, grads, cfg.seed, step_index, u_levels, u_signs, u_scales)
            api.dat_aggregate(plan, u_levels, u_signs, u_scales, None, u_ghat)
            if variant == "two_sided":
                api.dat_requantize(plan, u_ghat, cfg.seed, step_index, s_levels, s_signs, s_scales)
            if variant == "lamb":
                api.dat_lamb_step(plan, theta, mom, var, u_ghat, lamb_hp, step_index + 1)
            else:
                api.dat_lalr_step(plan, theta, mom, u_ghat, hp)
        elif args.path == "passes":
            api.dat_step_passes(plan, theta, mom, grads, cfg.seed, step_index, hp)
        elif args.path == "step_lamb":
            api.dat_step_lamb(plan, theta, mom, var, grads, cfg.seed, step_index, lamb_hp, step_index + 1)
        elif args.path == "step_two_sided":
            api.dat_step_two_sided(plan, theta, mom, grads, cfg.seed, step_index, hp, ts_ghat)
        elif args.path == "pipelined":
            api.dat_step_pipelined(plan, theta, mom, grads, cfg.seed, step_index, hp)
        else:
            api.dat_step(plan, theta, mom, grads, cfg.seed, step_index, hp)

    # ---- warm-up
    step_no = 0
    for _ in range(max(args.warmup, 3)):
        one_step(step_no)
        step_no += 1
    torch.cuda.synchronize()
    status = api.dat_get_status(plan)
    if status:
        raise SystemExit("device status word not clean after warm-up: %d" % status)

    # ---- timed region: exactly K steps, per-step CUDA events on the launching stream
    K = args.steps
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * K)]
    sampler = ClockSampler(local)
    launches0 = api.dat_plan_launch_count(plan)
    barrier()
    sampler.start()
    t_wall0 = time.perf_counter()
    for k in range(K):
        if flush is not None:
            flush.fill_(1.0)
        ev[2 * k].record(stream)
        one_step(step_no)
        ev[2 * k + 1].record(stream)
        step_no += 1
    sampler.sample()
    barrier()
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    launches = api.dat_plan_launch_count(plan) - launches0
    step_ms = np.array([ev[2 * k].elapsed_time(ev[2 * k + 1]) for k in range(K)])
    region_ms = ev[0].elapsed_time(ev[2 * K - 1]) if flush is None else float(step_ms.sum())
    status = api.dat_get_status(plan)
    finite = bool(torch.isfinite(theta).all().item() and torch.isfinite(mom).all().item())

    region_ms_max = max_over_ranks(region_ms, world, dev)
    elems_per_step = cfg.M * cfg.d
    value = job_value(world, elems_per_step, K, region_ms_max * 1e-3)

    # ---- end to end through the host-buffer entry point (H2D + step + D2H inside the timed region)
    e2e = None
    if not args.no_e2e and not unfused and not variant:
        th_h = theta.detach().cpu().pin_memory()
        mo_h = mom.detach().cpu().pin_memory()
        g_h = [g.detach().cpu().pin_memory() for g in grads]
        n_e2e = max(2, min(K, args.e2e_steps))
        api.dat_step_host(plan, th_h, mo_h, g_h, cfg.seed, step_no, hp)      # allocates the staging buffers
        barrier()
        t0 = time.perf_counter()
        for k in range(n_e2e):
            api.dat_step_host(plan, th_h, mo_h, g_h, cfg.seed, step_no + 1 + k, hp)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt_max = max_over_ranks(dt, world, dev)
        e2e = {"value": job_value(world, elems_per_step, n_e2e, dt_max), "unit": UNIT,
               "h2d_bytes_per_step": (cfg.M + 2) * cfg.d * 4, "d2h_bytes_per_step": 2 * cfg.d * 4,
               "steps": n_e2e, "ms_per_step": 1e3 * dt_max / n_e2e}

    # ---- CPU oracle beside it (rank 0, N = 1 only), on a bounded sample of the same workload
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        oracle.lib()
        th_c, mo_c = synth.make_params(cfg)
        g_c = [g.numpy() for g in synth.make_grads(cfg, 0)]
        threads = host_threads()
        cal_layers, _ = oracle_layer_sample(cfg, 4_000_000)
        t_cal, n_cal = time_oracle(cfg, th_c.numpy(), mo_c.numpy(), g_c, cal_layers, threads)
        layers, what = oracle_layer_sample(cfg, int(n_cal / t_cal * 15.0))
        t_or, n_or = time_oracle(cfg, th_c.numpy(), mo_c.numpy(), g_c, layers, threads)
        reps = 1
        while t_or * threads < 20.0 and reps < 50:                      # about 20 core-seconds of oracle work
            t_k, n_k = time_oracle(cfg, th_c.numpy(), mo_c.numpy(), g_c, layers, threads, step=reps)
            t_or, n_or, reps = t_or + t_k, n_or + n_k, reps + 1
        cpu = {"value": n_or / t_or, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": what + ", %d step(s), %.1f s wall on %d threads" % (reps, t_or, threads)}

    api.dat_plan_destroy(plan)
    if rank == 0:
        peak, peak_src = measured_peaks()
        kernel_ms = float(step_ms.mean())
        if unfused:     # norm pass + quantize pass over the gradients, planes written and read, g_hat, two LALR passes
            beta = (cfg.bits + 1) / 8.0
            algo_bytes = int((8 * cfg.M + 2 * beta * cfg.M + 32) * cfg.d)
            if variant == "two_sided":  # norm pass and quantize pass over g_hat, the server's planes written and read, g_hat rewritten
                algo_bytes += int((12 + 2 * beta) * cfg.d)
            if variant == "lamb":       # pass 1 reads theta, m, v, g_hat and writes m, v; pass 2 reads theta, m, v and writes theta
                algo_bytes += 12 * cfg.d
        else:
            algo_bytes = (4 * cfg.M + 16) * cfg.d
            if variant == "lamb":       # v read and written in the Q part, read again in the U part
                algo_bytes += 8 * cfg.d
            if variant == "two_sided":  # g_hat written once (the receiver's value is the call's output)
                algo_bytes += 4 * cfg.d
        achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
        # the quantizer norm forces a second read of a layer whose M gradients (4 M n_l bytes) exceed the L2 cache
        sizes = np.diff(np.asarray(cfg.offsets, dtype=np.int64))
        second_read = int(4 * cfg.M * sizes[4 * cfg.M * sizes > l2_bytes].sum()) if not unfused and cfg.bits != 32 else 0
        per_step = launches // K
        traffic, traffic_src = ncu_traffic(args.path, cfg)
        kernel_name = {"step": "dat_step (k_step_pipelined)", "pipelined": "dat_step_pipelined (k_step_pipelined)",
                       "passes": "dat_step_passes"}.get(args.path, args.path)
        kernel_name += ": %d launch%s per step, the whole step timed" % (per_step, "" if per_step == 1 else "es")
        sm_mhz = clocks.get("sm_mhz") or 0
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
            "ms_per_step": region_ms_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(cfg, l2_note), path=args.path),
            "step_latency_us": {"median": 1e3 * float(np.median(step_ms)), "min": 1e3 * float(step_ms.min()),
                                "mean": 1e3 * kernel_ms},
            "pct_of_8TBps": 100.0 * achieved / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "traffic_source": traffic_src, "algorithmic_bytes_per_launch": algo_bytes // max(per_step, 1),
                         "algorithmic_bytes_per_step": algo_bytes, "kernel": kernel_name, "peak_source": peak_src,
                         "sm_cycles_per_step": (1e3 * kernel_ms) * sm_mhz if sm_mhz else None,
                         "bytes_2pass": algo_bytes + second_read,
                         "frac_2pass": (algo_bytes + second_read) / (kernel_ms * 1e-3) / 1e9 / peak},
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "status_word": int(status), "outputs_finite": finite, "wall_s_timed_region": t_wall,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_sharded(args):
    """The sharded step (paper_2206_06257_b200/sharded.py): total work fixed, divided over the ranks."""
    import torch
    import torch.distributed as dist
    from paper_2206_06257_b200 import api, synth
    from paper_2206_06257_b200.sharded import CudaOps, ShardedStep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for this path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    cfg = synth.config(args.config)
    if args.bits:
        cfg.bits = args.bits
    if args.rng_bits:
        cfg.rng_bits = args.rng_bits
    if cfg.M % world:
        raise SystemExit("--sharded needs the workload's %d workers to divide over %d ranks" % (cfg.M, world))
    M_loc = cfg.M // world
    theta, mom = synth.make_params(cfg, device=dev)
    grads = synth.make_grads(cfg, 0, device=dev)[rank * M_loc:(rank + 1) * M_loc]      # this rank's workers
    hp = (cfg.lr, cfg.momentum, cfg.weight_decay, cfg.c_l, cfg.c_u)
    ops = CudaOps(api, cfg.offsets, cfg.M, M_loc, rank, world, cfg.bits, cfg.rng_bits)
    st = ShardedStep(ops, cfg.offsets, cfg.M, rank, world)
    do_step = st.step_pull if args.exchange == "pull" else st.step
    mom_own = mom[st.own.a8:st.own.b].clone()
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_no = 0
    for _ in range(max(args.warmup, 3)):
        do_step(theta, mom_own, grads, cfg.seed, step_no, hp)
        step_no += 1
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0.record(stream)
    for _ in range(K):
        do_step(theta, mom_own, grads, cfg.seed, step_no, hp)
        step_no += 1
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    finite = bool(torch.isfinite(theta).all().item())
    own_bytes = sum(ops.plane_bytes(rg)[0] + ops.plane_bytes(rg)[1] for q, rg in enumerate(st.ranges) if q != rank) * M_loc
    ops.close()
    if rank == 0:
        peak, peak_src = measured_peaks()
        value = cfg.M * cfg.d * K / (ms * 1e-3)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": dict(workload_config(cfg, "inputs larger than L2, no flush"), parallelism="sharded: %d worker(s) and one layer range per rank, exchange %s" % (M_loc, args.exchange),
                           path="sharded (dat_worker_norms, dat_quantize, plane exchange, dat_aggregate, dat_lalr_step, theta broadcast)"),
            "roofline": None, "cpu_baseline": None, "e2e": None,
            "sent_plane_bytes_per_rank_and_step": int(own_bytes), "clocks": clocks, "outputs_finite": finite,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100,
                    help="timed steps (after about 60 ms of back-to-back steps the GPU comes under its power cap and the clocks drop: "
                         "the measured peak this is compared with is a burst figure too)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="resnet50",
                    choices=["tiny_mlp", "resnet18", "resnet50", "resnet50_m32", "flat1b", "flat_small"])
    ap.add_argument("--bits", type=int, default=0, help="override the config's bits")
    ap.add_argument("--rng-bits", type=int, default=0, choices=[0, 16, 23],
                    help="override the resolution of the quantizer's uniform number (0: the config's)")
    ap.add_argument("--impl", default="dat", choices=["dat", "reference"])
    ap.add_argument("--path", default="step",
                    choices=["step", "step_per_worker", "step_lamb", "step_two_sided", "pipelined", "passes", "unfused", "unfused_per_worker", "unfused_two_sided", "unfused_lamb"],
                    help="step: dat_step (the headline: one pipelined launch); pipelined: the same by its own name; "
                         "step_per_worker: dat_step on a plan with one quantizer norm per worker; step_lamb: dat_step_lamb; step_two_sided: dat_step_two_sided (Step 10 in the same launch); "
                         "passes: dat_step_passes, three streaming passes; unfused: dat_quantize + dat_aggregate + dat_lalr_step; "
                         "unfused_per_worker: the same with one quantizer norm per worker; unfused_two_sided: with "
                         "dat_requantize after the aggregation; unfused_lamb: with dat_lamb_step as the update")
    ap.add_argument("--sharded", action="store_true",
                    help="the step sharded over the --gpus ranks (layer ranges owned by ranks, planes exchanged, "
                         "theta broadcast) instead of independent replicas; the M workers are divided over the ranks")
    ap.add_argument("--exchange", default="sendrecv", choices=["sendrecv", "pull"],
                    help="with --sharded: planes sent to their owners (NCCL point-to-point), or left in symmetric memory "
                         "and read from there by the owner's aggregation kernel (dat_aggregate_gather)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.sharded:
        return run_sharded(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
