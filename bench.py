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
    # 362.11 MB read+written for 8 rows (the ncu summary of the filter kernel under profiles/), traffic proportional to rows
    "resnet18:11174": {"bytes": int(362.11e6 * 100 / 8), "digest": "35b76863fdbace2f"},
}
KERNEL_SOURCES = ("s3gd_filter.cu", "s3gd_tile.cuh", "s3gd_common.cuh")


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
    """Algorithmic bytes of one step: the dense model and the model that only touches voted x."""
    words = (K + 31) // 32
    b_grad = 4 * M * d
    b_sel = 2 * M * (4 * K + 4 * words)
    b_count = 2 * d if M <= 127 else 8 * d        # vote counters cleared + read: bytes up to 127 workers, else int32
    b_dense = b_grad + b_sel + b_count + 8 * d
    b_min = b_grad + 8 * min(d, M * K)
    return b_grad, b_dense, b_min


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
def oracle_sample_time(spec, K, rows, reps=1, randk=False):
    """Times the oracle's whole step on `rows` workers of the workload at full d (host cores)."""
    import torch
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200 import workloads as W
    s = W.spec(spec.name, M=rows)
    g = W.make_grads(s, "cpu").numpy()
    x = W.make_x(s, "cpu").numpy()
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        x, _, _, _ = O.randk_step(x, g, K, s.lr, 1, 0) if randk else O.step(x, g, K, s.lr)
        times.append(time.perf_counter() - t0)
    return times, rows * s.d, torch.get_num_threads()


def run_reference(args):
    """The oracle as the timed program: each step is the oracle's step on a bounded sample."""
    import torch
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200 import workloads as W
    if int(os.environ.get("RANK", "0")) != 0:
        return
    spec = W.SPECS[args.workload]
    K = args.K or spec.Ks[0]
    rows = 1
    s = W.spec(spec.name, M=rows)
    g = W.make_grads(s, "cpu").numpy()
    x = W.make_x(s, "cpu").numpy()
    for _ in range(args.warmup):
        x, _, _, _ = O.step(x, g, K, s.lr)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        x, _, _, _ = O.step(x, g, K, s.lr)
    dt = time.perf_counter() - t0
    value = rows * s.d * args.steps / dt
    sample = f"{rows} of {spec.M} workers at full d={s.d}, K={K}, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32",
        "data": "synthetic", "config": {"workload": spec.name, "d": s.d, "M": spec.M, "K": K, "sample": sample},
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


# --------------------------------------------------------------------------- GPU side
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

    step_no = [0]
    if args.unfused:                            # the three calls with the message written to device memory
        words = S.binding.words(K)
        m_idx = torch.empty((M, K), dtype=torch.int32, device=dev)
        m_sgn = torch.empty((M, words), dtype=torch.int32, device=dev)
        m_vote = torch.empty(d, dtype=torch.int8, device=dev)

    sharded = None
    if args.shard_rows:                         # every rank's M rows are M of the job's world*M workers
        from paper_2302_07475_b200.sharded import ShardedStep
        sharded = ShardedStep(M, d, K, dev)

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
            S.s3gd_step_ex(x, grads, K, spec.lr, ws, err=err, eta=1.0, v=vmom, mu=args.momentum or 0.0)
        else:
            S.s3gd_step(x, grads, K, spec.lr, ws)

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize(dev)

    for _ in range(max(args.warmup, 3)):
        one_step()
    code, info = S.s3gd_device_status(ws)
    if args.graph:                              # capture the step once, replay it in the timed loops
        eager_step = one_step
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            eager_step()
        one_step = graph.replay
        stream = torch.cuda.current_stream(dev)

    # ---- timed region: device-resident inputs; the library brackets the dominant (filter) kernel of
    # every timed step with two events.  The other phase boundaries are not marked here, because each
    # event record between two kernels costs a few microseconds of the step.
    sampler = ClockSampler(physical_gpu_index(local_rank)).start()
    S.s3gd_profile_begin_filter(args.steps)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        one_step()
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    phases, launches = S.s3gd_profile_end(args.steps)
    clocks = sampler.stop()
    S.s3gd_device_status(ws)
    kernel_ms = [p[1] for p in phases]
    if K == d:                                   # one kernel is the whole step
        kernel_ms = [ms_total / args.steps]

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

    ms_total, e2e_max = max_over_ranks([ms_total, e2e_ms if e2e_ms is not None else 0.0], dist, dev)

    if rank == 0:
        elems_per_step = world * M * d
        ms_step = ms_total / args.steps
        value = whole_job_value(world, M, d, args.steps, ms_total)
        b_grad, b_dense, b_min = byte_models(M, d, K)
        if args.error_feedback:                  # + read and write of the error memory (fused ideal: 12 B per element)
            b_dense += 8 * M * d
            b_min += 8 * M * d
        if args.momentum is not None:            # + read and write of v
            b_dense += 8 * d
            b_min += 8 * d
        peak, peak_kind = measured_peak()
        mean_phase = [sum(p[k] for p in phases) / max(len(phases), 1) for k in range(5)]
        dominant = max(range(5), key=lambda k: mean_phase[k])
        kernel_name = "signplane_step_kernel" if K == d else "filter_kernel"
        dom_ms = sum(kernel_ms) / max(len(kernel_ms), 1)      # from the timed steps
        if args.randk:
            # random-K never streams the gradients: M*K gathers of one 32-byte sector each, M*K integer
            # atomics on the counters, then the counter pass (4 B read per coordinate, x touched where voted)
            kernel_name, dom_ms = "randk_kernel", mean_phase[3]
            b_grad = M * K * (32 + 8)
            b_dense = b_min = b_grad + 4 * d + 4 * d
        achieved = b_grad / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else None
        tr = NCU_TRAFFIC.get(f"{spec.name}:{K}")
        traffic = tr["bytes"] if tr and tr.get("digest") == kernel_digest() else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u32+f32", "data": "synthetic",
            "config": {"workload": spec.name, "d": d, "M": M, "K": K, "lr": spec.lr,
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                       "l2_policy": f"inputs ({b_grad / 1e6:.0f} MB of gradients per step) larger than L2"},
            "steps_per_s": 1e3 / ms_step,
            "step_bytes": {"dense_model": b_dense, "min_model": b_min,
                           "dense_GBps": b_dense / (ms_step * 1e-3) / 1e9,
                           "frac_of_measured": b_dense / (ms_step * 1e-3) / 1e9 / peak,
                           "frac_of_nominal_8TBps": b_dense / (ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
            "phase_ms": dict(zip(S.binding.PHASES, [round(v, 5) for v in mean_phase])),
            "phase_ms_source": f"separate pass of {n_break} steps with every phase boundary marked (after the timed region)",
            "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                         "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s",
                         "frac": achieved / peak if achieved else None, "traffic": traffic,
                         "algorithmic_bytes_per_launch": b_grad, "kernel_ms": dom_ms,
                         "dominant_phase": S.binding.PHASES[dominant]},
            "clocks": clocks,
            "gpu_launches": launches,
            "device_info": {"rows_off_single_read_route": info[1], "max_candidates_per_row": info[4]},
        }
        if args.randk:
            line["config"]["variant"] = {"selection": "RandKSign (Section 3.4)"}
        if sharded is not None:
            line["config"]["parallelism"] = f"workers sharded over {world} rank(s), {world * M} workers in the vote"
            line["config"]["variant"] = {"calls": "s3gd_topk_sign + all-gather of the message + s3gd_majority_vote + s3gd_apply",
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
            rows = args.cpu_rows
            t, elems, threads = oracle_sample_time(spec, K, rows, randk=args.randk)
            line["cpu_baseline"] = {"value": elems / t[0], "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": f"{rows} of {M} workers at full d={d}, K={K}, one step, {t[0]:.1f} s",
                                    "host_cores_available": os.cpu_count()}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
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
    ap.add_argument("--graph", action="store_true",
                    help="capture the step in a CUDA graph and time replays (for the launch-bound small workloads)")
    ap.add_argument("--unfused", action="store_true",
                    help="time the three separate calls (message written out) instead of the fused step")
    ap.add_argument("--randk", action="store_true",
                    help="time s3gd_step_randk (RandKSign, Section 3.4) instead of s3gd_step")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-rows", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
