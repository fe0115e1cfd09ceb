#!/usr/bin/env python
"""Throughput of the fused S3GD-MV step on B200, with its roofline and a CPU baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--K K] [--impl ours|reference]

A step is one s3gd_step call (top-K sign, majority vote, update) on one synthetic
gradient batch.  Rank r of an N-GPU launch runs its own replica of the step on its
own GPU (the method's workers are rows of the batch, not ranks: there is nothing to
exchange), so the job's value is N times a rank's work divided by the slowest rank's
device time.  One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "grad elements/s (M*d) through top-K+sign+majority vote+update"
UNIT = "elements/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes per launch of the filter kernel from the ncu capture summarised under
# profiles/, keyed by workload, with the digest of the kernel sources they were taken
# at.  Reported only while the sources are unchanged.
NCU_TRAFFIC = {
    # 358.41 MB read + 3.97 MB written for 8 rows (profiles/filter_band_kernel_resnet18_M8.md), traffic proportional to rows
    "resnet18:11174": {"bytes": int((358.406144e6 + 3.968512e6) * 100 / 8), "digest": "c35375498f1ef2e9"},
}
KERNEL_SOURCES = ("s3gd_filter.cu", "s3gd_tile.cuh", "s3gd_common.cuh")
# The dominant kernel of every FILTER_EVENTS_EVERY-th timed step is bracketed by two CUDA events (an event
# record between two kernels costs a microsecond or two of the step, about 5 us per step for the pair).
FILTER_EVENTS_EVERY = 4


def kernel_digest() -> str:
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2302_07475_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def byte_models(M, d, K):
    """Algorithmic bytes of one step under the four models that are reported side by side.

    json   4Md + message written and read + int32 vote counters (8d) + x read and written (8d): the
           count the throughput target was stated on (K = d: 4Md + 16d, there is no message)
    dense  the same with the vote counters this library uses in the fused step (one byte per
           coordinate up to 127 workers: 2d; int32 above: 8d)
    moved  dense without the message: the fused step without optional outputs never writes one
    min    4Md + 8 bytes for every coordinate that can receive a vote (x touched only where voted)
    """
    words = (K + 31) // 32
    b_grad = 4 * M * d
    if K == d:          # signSGD with majority vote: no selection, no message, no counters in memory
        return {"grad": b_grad, "json": b_grad + 16 * d, "dense": b_grad + 8 * d, "moved": b_grad + 8 * d,
                "min": b_grad + 8 * d}
    b_sel = 2 * M * (4 * K + 4 * words)
    b_count = 2 * d if M <= 127 else 8 * d
    return {"grad": b_grad, "json": b_grad + b_sel + 16 * d, "dense": b_grad + b_sel + b_count + 8 * d,
            "moved": b_grad + b_count + 8 * d, "min": b_grad + 8 * min(d, M * K)}


def fractions(models, ms_step, peak):
    """GB/s and the fraction of the nominal and of the measured peak for every byte model."""
    out = {}
    for name in ("json", "dense", "moved", "min"):
        gbs = models[name] / (ms_step * 1e-3) / 1e9
        out[name] = {"bytes": models[name], "GBps": gbs, "of_8TBps": gbs / NOMINAL_HBM_GBS, "of_measured": gbs / peak}
    return out


class ClockSampler:
    """Polls SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.ok = False

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            return self
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def _run(self):
        nv = self._nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# --------------------------------------------------------------------------- CPU side
CPU_SAMPLE_ROWS = 2          # workers of the workload that one oracle step covers, at full d


def workload_config(spec, K, world=1):
    """The `config` object of the JSON line; the same for both arms."""
    return {"workload": spec.name, "d": spec.d, "M": spec.M, "K": K, "lr": spec.lr,
            "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
            "l2_policy": f"inputs ({4 * spec.M * spec.d / 1e6:.0f} MB of gradients per step) larger than L2"}


def oracle_sample(spec, rows):
    """The first `rows` workers of the workload at full d, on the host, plus x."""
    from paper_2302_07475_b200 import workloads as W
    s = W.spec(spec.name, M=rows)
    return s, W.make_grads(s, "cpu").numpy(), W.make_x(s, "cpu").numpy()


def oracle_definition_time(spec, K, rows, budget_s=12.0, max_steps=4, randk=False):
    """Times the oracle's definitional step (sort-based) on `rows` workers at full d, one host thread."""
    import torch
    from oracle import s3gd_oracle as O
    torch.set_num_threads(1)
    s, g, x = oracle_sample(spec, rows)
    times = []
    while len(times) < max_steps and sum(times) < budget_s:
        t0 = time.perf_counter()
        x, _, _, _ = O.randk_step(x, g, K, s.lr, 1, 0) if randk else O.step(x, g, K, s.lr)
        times.append(time.perf_counter() - t0)
    return times, rows * s.d


def _fast_rows_worker(args):
    """Pool worker: draws its rows on the host, then times the oracle's threshold route on them."""
    name, d, M, K, rows = args
    import numpy as np
    import torch
    torch.set_num_threads(1)
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200 import workloads as W
    s = W.spec(name, d=d, M=M)
    g = W.make_rows(s, rows, "cpu").numpy()
    t0 = time.perf_counter()
    idx, sgn = O.topk_sign_threshold(g, K)
    return rows, idx, sgn, time.perf_counter() - t0


def oracle_fast_all_cores(spec, K, cores, rows_total):
    """The oracle's threshold route with the workers spread over `cores` processes, then its vote and
    update in the parent.  Returns (seconds, elements, processes).  Drawing the inputs is not timed."""
    import multiprocessing as mp
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200 import workloads as W
    rows_total = min(rows_total, spec.M)
    procs = max(1, min(cores, rows_total))
    shares = [list(range(p, rows_total, procs)) for p in range(procs)]
    ctx = mp.get_context("spawn")               # never fork a process that has touched the GPU
    with ctx.Pool(procs) as pool:
        parts = pool.map(_fast_rows_worker, [(spec.name, spec.d, spec.M, K, sh) for sh in shares])
    import numpy as np
    idx = np.zeros((rows_total, K), np.uint32)
    sgn = np.zeros((rows_total, (K + 31) // 32), np.uint32)
    for rows, i, sg, _ in parts:
        idx[rows], sgn[rows] = i, sg
    x = W.make_x(spec, "cpu").numpy()
    t0 = time.perf_counter()
    vote, _ = O.majority_vote(idx, sgn, rows_total, K, spec.d)
    O.apply_vote(x, vote, spec.lr)
    t_vote = time.perf_counter() - t0
    return max(p[3] for p in parts) + t_vote, rows_total * spec.d, procs


def run_reference(args):
    """The oracle as the timed program: each step is the oracle's definitional step on the same
    bounded sample of the workload that the other arm's cpu_baseline times."""
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200 import workloads as W
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    torch.set_num_threads(1)
    spec = W.SPECS[args.workload]
    K = args.K or spec.Ks[0]
    rows = min(args.cpu_rows, spec.M)
    s, g, x = oracle_sample(spec, rows)
    for _ in range(args.warmup):
        x, _, _, _ = O.step(x, g, K, s.lr)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        x, _, _, _ = O.step(x, g, K, s.lr)
    dt = time.perf_counter() - t0
    value = rows * s.d * args.steps / dt
    sample = f"{rows} of {spec.M} workers at full d={s.d}, K={K}, per step (definitional oracle, numpy, one thread)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32",
        "data": "synthetic", "config": workload_config(spec, K, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------- multi-rank plumbing
def max_over_ranks(values, dist, device):
    """Element-wise maximum of a short list of floats over all ranks (identity without a process group)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(world, M, d, steps, ms_total):
    """Elements/s of the whole job: every rank steps its own M x d replica; time is the slowest rank's."""
    return world * M * d * steps / (ms_total * 1e-3)


def pick_repeats(requested, steps, est_ms_step, target_ms=1000.0, lo=5, hi=50):
    """How many back-to-back timed regions of `steps` steps: enough for about a second under load."""
    if requested > 0:
        return requested
    need = int(target_ms / max(steps * est_ms_step, 1e-3)) + 1
    return max(lo, min(hi, need))


# --------------------------------------------------------------------------- GPU side
def timed_regions(one_step, steps, repeats, stream, barrier):
    """`repeats` back-to-back regions of `steps` steps each, every region bracketed by CUDA events on the
    launching stream, the whole bracketed by barrier + synchronize.  Returns the region times in ms."""
    import torch
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    barrier()
    ev[0].record(stream)
    for r in range(repeats):
        for _ in range(steps):
            one_step()
        ev[r + 1].record(stream)
    barrier()
    return [ev[r].elapsed_time(ev[r + 1]) for r in range(repeats)]


def acceptance_case(S, W, spec, K, dev, stream, barrier, peak, steps=20, repeats=5, grads=None, x=None):
    """One (workload, K) of the acceptance range: fused step without optional outputs, timed like the headline."""
    import torch
    M, d = spec.M, spec.d
    if grads is None:
        grads = W.make_grads(spec, dev)
    if x is None:
        x = W.make_x(spec, dev)
    ws = S.alloc_workspace(M, d, K, dev)

    def one_step():
        S.s3gd_step(x, grads, K, spec.lr, ws)

    for _ in range(3):
        one_step()
    code, info = S.s3gd_device_status(ws)
    n_marked = (steps * repeats + FILTER_EVENTS_EVERY - 1) // FILTER_EVENTS_EVERY
    S.s3gd_profile_begin_filter_every(n_marked, FILTER_EVENTS_EVERY)
    regions = timed_regions(one_step, steps, repeats, stream, barrier)
    phases, _ = S.s3gd_profile_end(n_marked)
    S.s3gd_device_status(ws)
    ms_step = statistics.median(regions) / steps
    filt = [p[1] for p in phases]
    filter_ms = (sum(filt) / len(filt)) if (filt and K != d) else ms_step
    models = byte_models(M, d, K)
    out = {"workload": spec.name, "d": d, "M": M, "K": K, "K_over_d": K / d,
           "in_target_range": bool(d >= 11_000_000 and M >= 32 and K * 100 <= d + 99),
           "ms_per_step": ms_step, "ms_per_step_min": min(regions) / steps, "ms_per_step_max": max(regions) / steps,
           "steps": steps, "repeats": repeats, "elements_per_s": M * d / (ms_step * 1e-3),
           "streaming_kernel_ms": filter_ms,
           "streaming_kernel_GBps": models["grad"] / (filter_ms * 1e-3) / 1e9,
           "step_bytes": fractions(models, ms_step, peak),
           "rows_off_single_read_route": info[1], "max_candidates_per_row": info[4]}
    del ws
    return out


def run_acceptance(S, W, dev, stream, barrier, peak, headline_grads, headline_x, headline_spec):
    """Every (workload, K) inside the target range d >= 11M, M >= 32, K <= 1 %, the K = d path, the K = 10 %
    point of the tie-stress sweep and, if the device has room, the 2.1e9-coordinate workload."""
    import torch
    cases = []
    cases.append(acceptance_case(S, W, headline_spec, headline_spec.d, dev, stream, barrier, peak,
                                 grads=headline_grads, x=headline_x.clone()))
    del headline_grads
    torch.cuda.empty_cache()
    r50 = W.SPECS["resnet50_ties"]
    g = W.make_grads(r50, dev)
    x = W.make_x(r50, dev)
    for K in r50.Ks:
        cases.append(acceptance_case(S, W, r50, K, dev, stream, barrier, peak, grads=g, x=x.clone()))
    del g, x
    torch.cuda.empty_cache()
    big = W.SPECS["large"]
    free, _ = torch.cuda.mem_get_info(dev)
    need = 4 * big.M * big.d + 8 * big.d + S.s3gd_workspace_bytes(big.M, big.d, big.Ks[0]) + (4 << 30)
    if free >= need:
        cases.append(acceptance_case(S, W, big, big.Ks[0], dev, stream, barrier, peak, steps=5, repeats=3))
        torch.cuda.empty_cache()
    else:
        cases.append({"workload": "large", "skipped": f"needs {need / 1e9:.0f} GB on the device, {free / 1e9:.0f} GB free"})
    return cases


def run_ours(args):
    import torch
    import paper_2302_07475_b200 as S
    from paper_2302_07475_b200 import build as B, workloads as W

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        B.build()
    if dist is not None:
        dist.barrier()
    S.load()

    spec = W.spec(args.workload, d=args.d or None, M=args.M or None)
    K = args.K or spec.Ks[0]
    M, d = spec.M, spec.d
    grads = W.make_grads(spec, dev)
    x = W.make_x(spec, dev)
    ws = S.alloc_workspace(M, d, K, dev)
    stream = torch.cuda.current_stream(dev)
    extended = args.error_feedback or args.momentum is not None
    err = torch.zeros((M, d), dtype=torch.float32, device=dev) if args.error_feedback else None
    vmom = torch.zeros(d, dtype=torch.float32, device=dev) if args.momentum is not None else None
    # With error memory the same gradients every step would make every unkept coordinate grow in lockstep
    # towards the threshold, which no training run does: alternate between two seeded batches instead.
    grads_b = W.make_grads(spec, dev, step=1) if args.error_feedback else None

    step_no = [0]
    if args.unfused:                            # the three calls with the message written to device memory
        words = S.binding.words(K)
        m_idx = torch.empty((M, K), dtype=torch.int32, device=dev)
        m_sgn = torch.empty((M, words), dtype=torch.int32, device=dev)
        m_vote = torch.empty(d, dtype=torch.int8, device=dev)

    sharded = None
    if args.shard_rows:                         # every rank's M rows are M of the job's world*M workers
        from paper_2302_07475_b200.sharded import ShardedStep
        sharded = ShardedStep(M, d, K, dev, downlink=args.downlink)

    def one_step():
        if sharded is not None:
            sharded.step(x, grads, spec.lr)
        elif args.unfused:
            S.s3gd_topk_sign(grads, K, m_idx, m_sgn, ws)
            S.s3gd_majority_vote(m_idx, m_sgn, M, K, d, m_vote, ws)
            S.s3gd_apply(x, m_vote, spec.lr)
        elif args.randk:
            step_no[0] += 1
            S.s3gd_step_randk(x, grads, K, spec.lr, 20230207, step_no[0], ws)
        elif extended:
            step_no[0] += 1
            g_now = grads_b if (grads_b is not None and step_no[0] % 2 == 0) else grads
            S.s3gd_step_ex(x, g_now, K, spec.lr, ws, err=err, eta=1.0, v=vmom, mu=args.momentum or 0.0)
        else:
            S.s3gd_step(x, grads, K, spec.lr, ws)

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize(dev)

    warmup = max(args.warmup, 3)
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(warmup):
        if i == warmup - 1:
            w0.record(stream)
        one_step()
    w1.record(stream)
    code, info = S.s3gd_device_status(ws)
    est_ms = max(w0.elapsed_time(w1), 1e-3)
    repeats = pick_repeats(args.repeats, args.steps, est_ms)
    if args.graph:                              # capture the step once, replay it in the timed loops
        eager_step = one_step
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            eager_step()
        one_step = graph.replay
        stream = torch.cuda.current_stream(dev)

    # ---- timed region: device-resident inputs; `repeats` back-to-back regions of `steps` steps, the
    # median region is the reported one.  The library brackets the dominant (filter) kernel of every
    # fourth timed step with two events; the other phase boundaries are not marked here, because each
    # event record between two kernels costs a microsecond or two of the step.
    sampler = ClockSampler(physical_gpu_index(local_rank)).start()
    n_marked = (args.steps * repeats + FILTER_EVENTS_EVERY - 1) // FILTER_EVENTS_EVERY
    S.s3gd_profile_begin_filter_every(n_marked, FILTER_EVENTS_EVERY)
    regions = timed_regions(one_step, args.steps, repeats, stream, barrier)
    phases, launches = S.s3gd_profile_end(n_marked)
    clocks = sampler.stop()
    S.s3gd_device_status(ws)
    ms_total = statistics.median(regions)
    kernel_ms = [p[1] for p in phases]
    if K == d:                                   # one kernel is the whole step
        kernel_ms = [ms_total / args.steps]
    launches_per_region = launches / repeats if repeats else launches

    # ---- the phase breakdown, from a separate short pass with every boundary marked (not the timed one)
    n_break = min(args.steps, 50)
    if not args.graph:
        S.s3gd_profile_begin(n_break)
        for _ in range(n_break):
            one_step()
        phases, _ = S.s3gd_profile_end(n_break)
        S.s3gd_device_status(ws)

    # ---- end to end: gradients start in pinned host memory, the updated x is read back
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    e2e_err = "skipped"
    try:
        if args.e2e_steps <= 0:
            raise RuntimeError("skipped")
        host_g = torch.empty((M, d), dtype=torch.float32, pin_memory=True)
        host_g.copy_(grads)
        host_x = torch.empty(d, dtype=torch.float32, pin_memory=True)
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for _ in range(e2e_steps):
            grads.copy_(host_g, non_blocking=True)
            one_step()
            host_x.copy_(x, non_blocking=True)
        f1.record(stream)
        barrier()
        e2e_ms = f0.elapsed_time(f1)
        del host_g
    except RuntimeError as exc:          # pinned allocation refused
        e2e_ms = None
        e2e_err = str(exc).splitlines()[0]

    ms_total, ms_min, ms_max, e2e_max = max_over_ranks(
        [ms_total, min(regions), max(regions), e2e_ms if e2e_ms is not None else 0.0], dist, dev)

    plain = not (args.unfused or args.randk or extended or args.graph or sharded is not None or args.M or args.d)
    acceptance = None
    peak, peak_kind = measured_peak()
    if rank == 0 and world == 1 and plain and args.workload == "resnet18" and not args.K and not args.no_acceptance:
        del ws
        acceptance = run_acceptance(S, W, dev, stream, barrier, peak, grads, x, spec)
        grads = None

    if rank == 0:
        elems_per_step = world * M * d
        ms_step = ms_total / args.steps
        value = whole_job_value(world, M, d, args.steps, ms_total)
        models = byte_models(M, d, K)
        if args.error_feedback:                  # + read and write of the error memory (fused ideal: 12 B per element)
            for k in ("json", "dense", "moved", "min"):
                models[k] += 8 * M * d
        if args.momentum is not None:            # + read and write of v
            for k in ("json", "dense", "moved", "min"):
                models[k] += 8 * d
        mean_phase = [sum(p[k] for p in phases) / max(len(phases), 1) for k in range(5)]
        dominant = max(range(5), key=lambda k: mean_phase[k])
        kernel_name = "signplane_step_kernel" if K == d else "filter_band_kernel"
        if args.unfused or args.error_feedback or sharded is not None:
            kernel_name = "filter_kernel / filter_scan_kernel"      # the ranked form of the pass
        dom_ms = sum(kernel_ms) / max(len(kernel_ms), 1)      # from the timed steps
        b_grad = models["grad"]
        if args.randk:
            # random-K never streams the gradients: M*K gathers of one 32-byte sector each, M*K integer
            # atomics on the counters, then the counter pass (4 B read per coordinate, x touched where voted)
            kernel_name, dom_ms = "randk_kernel", mean_phase[3]
            b_grad = M * K * (32 + 8)
            for k in ("json", "dense", "moved", "min"):
                models[k] = b_grad + 4 * d + 4 * d
        achieved = b_grad / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else None
        tr = NCU_TRAFFIC.get(f"{spec.name}:{K}")
        traffic = tr["bytes"] if tr and tr.get("digest") == kernel_digest() else None
        fr = fractions(models, ms_step, peak)
        config = workload_config(spec, K, world)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "repeats": repeats, "ms_per_step": ms_step,
            "ms_per_step_min": ms_min / args.steps, "ms_per_step_max": ms_max / args.steps,
            "timing": f"median of {repeats} back-to-back regions of {args.steps} steps, CUDA events on the launching stream",
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u32+f32", "data": "synthetic",
            "config": config,
            "steps_per_s": 1e3 / ms_step,
            "step_bytes": {"dense_model": models["dense"], "min_model": models["min"], "json_model": models["json"],
                           "moved_model": models["moved"],
                           "dense_GBps": fr["dense"]["GBps"], "frac_of_measured": fr["dense"]["of_measured"],
                           "frac_of_nominal_8TBps": fr["dense"]["of_8TBps"], "models": fr},
            "phase_ms": dict(zip(S.binding.PHASES, [round(v, 5) for v in mean_phase])),
            "phase_ms_source": f"separate pass of {n_break} steps with every phase boundary marked (after the timed region)",
            "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                         "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s",
                         "frac": achieved / peak if achieved else None, "traffic": traffic,
                         "algorithmic_bytes_per_launch": b_grad, "kernel_ms": dom_ms,
                         "kernel_ms_source": f"CUDA events around every {FILTER_EVENTS_EVERY}th launch inside the timed "
                                             f"region, {len(kernel_ms)} launches averaged",
                         "dominant_phase": S.binding.PHASES[dominant]},
            "clocks": clocks,
            "gpu_launches": int(round(launches_per_region)),
            "gpu_launches_note": f"kernels of this library enqueued per region of {args.steps} steps",
            "device_info": {"rows_off_single_read_route": info[1], "max_candidates_per_row": info[4]},
        }
        if acceptance is not None:
            line["acceptance"] = acceptance
        if args.randk:
            line["config"]["variant"] = {"selection": "RandKSign (Section 3.4)"}
        if sharded is not None:
            line["config"]["parallelism"] = f"workers sharded over {world} rank(s), {world * M} workers in the vote"
            line["config"]["variant"] = {"calls": sharded.describe(),
                                         "message_bytes_per_rank": sharded.message_bytes_per_rank()}
            line["roofline"] = None
            line["phase_ms"] = None
        if args.graph:
            line["config"].setdefault("variant", {})["launch"] = "CUDA graph replay"
            line["roofline"] = None             # the library's phase events are not part of a captured step
            line["phase_ms"] = None
        if args.unfused:
            line["config"]["variant"] = {"calls": "s3gd_topk_sign + s3gd_majority_vote + s3gd_apply"}
            line["roofline"] = None             # the phase events belong to s3gd_step; only the step time is reported
            line["phase_ms"] = None
        if extended:
            line["config"]["variant"] = {"error_feedback_eta": 1.0 if args.error_feedback else None, "momentum_mu": args.momentum}
        if args.M or args.d:
            line["config"]["note"] = "reduced case of the named workload (not the headline configuration)"
        if e2e_ms is not None:
            line["e2e"] = {"value": elems_per_step * e2e_steps / (e2e_max * 1e-3), "unit": UNIT,
                           "h2d_bytes_per_step": 4 * M * d, "d2h_bytes_per_step": 4 * d, "steps": e2e_steps,
                           "ms_per_step": e2e_max / e2e_steps}
        else:
            line["e2e"] = {"value": None, "unit": UNIT, "error": e2e_err}
        if world == 1 and not args.no_cpu_baseline:
            rows = min(args.cpu_rows, M)
            t, elems = oracle_definition_time(spec, K, rows, randk=args.randk)
            best = min(t)
            line["cpu_baseline"] = {"value": elems / best, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": f"{rows} of {M} workers at full d={d}, K={K}, per step; {len(t)} steps of "
                                              f"{best:.1f} s (definitional oracle, numpy, one thread)",
                                    "host_cores_available": os.cpu_count()}
            if not args.randk:
                cores = os.cpu_count() or 1
                sec, el, procs = oracle_fast_all_cores(spec, K, cores, 2 * cores)
                line["cpu_baseline"]["all_cores"] = {
                    "value": el / sec, "unit": UNIT, "cores": procs, "threads_per_process": 1, "kind": "oracle",
                    "sample": f"{el // d} of {M} workers at full d={d}, K={K}, one step in {sec:.1f} s (threshold route "
                              f"of the oracle, one process per core, then its vote and update in one process)"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=0,
                    help="back-to-back timed regions of --steps steps (default: enough for about one second, 5 to 50)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18",
                    choices=["tiny", "small_cnn", "resnet18", "resnet50_ties", "large"])
    ap.add_argument("--K", type=int, default=0, help="sparsity (default: the workload's first K)")
    ap.add_argument("--M", type=int, default=0, help="override the number of workers (smaller case of the same recipe)")
    ap.add_argument("--d", type=int, default=0, help="override the model size (smaller case of the same recipe)")
    ap.add_argument("--error-feedback", action="store_true",
                    help="time s3gd_step_ex with error memory (eta = 1, the paper's default) instead of s3gd_step")
    ap.add_argument("--momentum", type=float, default=None, help="also use the momentum update with this mu")
    ap.add_argument("--shard-rows", action="store_true",
                    help="the deployment shape: each rank's rows are its own workers; the message is all-gathered "
                         "and every rank votes over all of them (default: independent replicas)")
    ap.add_argument("--downlink", default="replicated", choices=["replicated", "two_bit", "sparse"],
                    help="with --shard-rows: how the vote reaches the ranks")
    ap.add_argument("--graph", action="store_true",
                    help="capture the step in a CUDA graph and time replays (for the launch-bound small workloads)")
    ap.add_argument("--unfused", action="store_true",
                    help="time the three separate calls (message written out) instead of the fused step")
    ap.add_argument("--randk", action="store_true",
                    help="time s3gd_step_randk (RandKSign, Section 3.4) instead of s3gd_step")
    ap.add_argument("--no-acceptance", action="store_true",
                    help="skip the extra (workload, K) cases that the default run times after the headline")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-rows", type=int, default=CPU_SAMPLE_ROWS)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
