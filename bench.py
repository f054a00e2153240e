#!/usr/bin/env python
"""Benchmark of the DiLoCo outer step with eager updates (and the kernels around it) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1] [--impl ours|reference]

One "step" is one fused eager outer step (Algorithm 3, lines 7-12: local outer gradients,
M-way mean, eager combination, Nesterov update, replica reset) over all M replicas of the
workload; between steps an untimed stand-in for the inner phase moves the replicas
(theta_m <- start_m + N(0, 1e-3)) and a 256 MB buffer is written to flush L2.  For the
phase workloads (cfg2, cfg3) a step is H fused AdamW steps followed by the eager outer step.

Prints ONE JSON line.  `value` is flat parameters advanced per second (P / t), whole job
(sum over ranks); `roofline` compares the algorithmic bytes of the dominant kernel with the
measured HBM copy peak; `e2e` is the same step through diloco_outer_step_host with the state
in pinned host memory (copies inside the timed region); `cpu_baseline` is the CPU oracle
timed on this machine's host cores.

With --impl reference the CPU oracle itself is timed on the same workload (there is no
reference implementation of this path; the paper ships no code).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "outer_step_params_per_s"
UNIT = "params/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# ncu dram__bytes_read.sum + dram__bytes_write.sum per parameter index for one launch of the
# dominant kernel, from the captures summarised under profiles/ (None: not captured yet).
NCU_TRAFFIC_BYTES_PER_PARAM = {
    ("diloco_outer_eager", 4, 0): 134.38,    # profiles/outer_eager_f32_M4_P35M_cfg1.md
    ("diloco_inner_adamw", 4, 1): 86.35,     # profiles/inner_adamw_bf16_M4_P35M_cfg2slice.md (35 M slice, scaled by P)
    ("diloco_outer_eager", 16, 0): 516.2,    # profiles/outer_eager_f32_M16_P15M.md (15 M slice, scaled by P)
}


def outer_bytes_per_param(variant: int, M: int, theta_kind: int) -> int:
    """Algorithmic HBM bytes per parameter index: every state word read once, written once."""
    th_r = {0: 4, 1: 2, 2: 4}[theta_kind]            # master mode reads the fp32 master only
    th_w = {0: 4, 1: 2, 2: 6}[theta_kind]            # ... and writes master + bf16 copy
    per_replica_rw = 2 * (4 + 4)                      # start, outer_mom: read + write
    if variant == 2:                                  # eager: + delta_prev_local r/w, delta_prev_avg r/w
        return M * (th_r + th_w + per_replica_rw + 8) + 8
    if variant == 1:
        return M * (th_r + th_w + per_replica_rw) + 8
    return M * (th_r + th_w + per_replica_rw)


def adamw_bytes_per_param(M: int, theta_kind: int, grad_kind: int) -> int:
    th = {0: 8, 1: 4, 2: 10}[theta_kind]             # theta read+write (master: 4 r, 4+2 w)
    g = 4 if grad_kind == 0 else 2
    return M * (th + g + 16)                          # + moments read+write


def load_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 100 ms from the warm-up on; the timed region's own samples are used when there are at least three."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float, t_fallback: float = None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.25]
        window = "timed region"
        if len(rows) < 3 and t_fallback is not None:       # under load since the warm-up began
            rows = [r for (t, r) in self.rows if t_fallback <= t <= t1 + 0.25]
            window = "warm-up + timed region"
        if not rows:
            rows, window = [r for (_, r) in self.rows], "whole run"
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                mhz.append(float(r[0]))
                mx = float(r[1])
            except Exception:
                continue
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        mhz.sort()
        return {"sm_mhz": (mhz[len(mhz) // 2] if mhz else None), "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz), "window": window}


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def shard_bounds(P_total: int, world: int, rank: int, quantum: int = 64):
    """Contiguous, quantum-aligned ranges of the parameter axis, one per rank (all M replicas'
    slices live on the same rank, so no step of the path crosses ranks)."""
    q = (P_total + quantum - 1) // quantum
    lo = (q * rank // world) * quantum
    hi = min(P_total, (q * (rank + 1) // world) * quantum)
    return lo, hi


# ------------------------------------------------------------------------------------ CPU arm
def time_oracle_eager(h, M, P, stride, theta_kind, eta, mu, nthreads, budget_s, max_steps=None):
    import oracle
    steps, t0 = 0, time.perf_counter()
    times = []
    while True:
        a = time.perf_counter()
        oracle.outer_step(oracle.EAGER, M=M, P=P, stride=stride, eta=eta, mu=mu, theta=h["theta"], start=h["start"],
                          outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                          delta_prev_avg=h["delta_prev_avg"], master=h.get("master"), theta_kind=theta_kind,
                          nthreads=nthreads)
        times.append(time.perf_counter() - a)
        steps += 1
        if time.perf_counter() - t0 >= budget_s or (max_steps and steps >= max_steps):
            break
    return times


def host_state(w, P, seed):
    """The workload's state drawn on the CPU as numpy arrays for the oracle."""
    import numpy as np
    import torch
    from paper_2502_12996_b200 import inputs
    st = inputs.make_outer_state(w.M, P, seed, device="cpu", theta_kind=w.theta_kind)
    h = {}
    for k in ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom"):
        t = st.get(k)
        if t is None:
            h[k] = None
        elif t.dtype == torch.bfloat16:
            h[k] = t.view(torch.int16).numpy().view(np.uint16)
        else:
            h[k] = t.numpy()
    return st, h


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    from paper_2502_12996_b200 import inputs
    oracle.build()
    w = inputs.WORKLOADS[args.workload]
    P = args.P or min(w.P, 35_000_000)                     # bounded sample of larger workloads
    cores = os.cpu_count() or 1
    st, h = host_state(w, P, w.seed)
    stride = st["stride"]
    for _ in range(max(1, args.warmup)):
        time_oracle_eager(h, w.M, P, stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 0, 1)
    times = time_oracle_eager(h, w.M, P, stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 1e9, args.steps)
    ms = 1e3 * sum(times) / len(times)
    value = P / (ms * 1e-3)
    sample = f"eager outer step, M={w.M}, P={P} of {w.P} (all replicas), {len(times)} steps, {cores} OpenMP threads"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "variant": "eager", "M": w.M, "P": P, "theta": ["f32", "bf16", "f32 master + bf16 copy"][w.theta_kind]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "cpu_model": cpu_model()},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
            "note": "the paper ships no code: the reference arm is the CPU oracle (plain C, -O2, no FMA) on the host cores"}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2502_12996_b200 import binding, build, inputs

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    if not binding.LIB_PATH.exists():
        build.build_library()
    # one rank per GPU; ranks beyond the device count (a gloo dry run on one GPU) share devices
    backend = os.environ.get("DILOCO_BENCH_BACKEND", "nccl")
    gpu = local_rank % torch.cuda.device_count()
    torch.cuda.set_device(gpu)
    dev = torch.device("cuda", gpu)
    red_dev = dev if backend == "nccl" else torch.device("cpu")      # where the tiny reductions live
    if world > 1:
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=dev)
        else:
            dist.init_process_group(backend)
    w = inputs.WORKLOADS[args.workload]
    P = args.P or w.P                                       # per GPU: weak scaling, every rank the full shape
    if args.strong:                                         # total work fixed: this rank's 64-aligned range
        lo, hi = shard_bounds(P, world, rank)
        P = hi - lo
    variant = {"standard": 0, "delayed": 1, "eager": 2}[args.variant]
    M = w.M
    phase = w.H > 0 and not args.outer_only
    th = {0: 4, 1: 2, 2: 6}[w.theta_kind]
    need = M * P * (th + 12 + (8 + (2 if w.grad_kind else 4) if phase else 0)) + 4 * P + M * P * 4 + (512 << 20)
    free = torch.cuda.mem_get_info(dev)[0]
    if need > free:                                         # report, never run the device out of memory
        if rank == 0:
            print(json.dumps({"metric": METRIC, "unit": UNIT, "value": None, "n_gpus": world,
                              "config": {"workload": args.workload},
                              "skipped": f"needs {need / 2**30:.1f} GiB of device memory, {free / 2**30:.1f} GiB free"}))
        return 0
    st = inputs.make_outer_state(M, P, w.seed + 1000 * rank, device=dev, theta_kind=w.theta_kind, with_adam=phase)
    stride = st["stride"]
    state = binding.State.from_dict(st, H=w.H, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum, beta1=w.beta1,
                                    beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay, grad_kind=w.grad_kind,
                                    impl=args.kernel)
    grads = None
    if phase:
        if w.segments:
            grads = torch.zeros((M, stride), dtype=torch.bfloat16 if w.grad_kind else torch.float32, device=dev)
            inputs.make_segment_grads(M, inputs.segment_sizes(P, w.segments),
                                      inputs.segment_scales(w.segments, st["gen"], dev).tolist(), st["gen"], grads)
        else:
            grads = inputs.make_grads(M, P, stride, st["gen"], dev, w.grad_kind)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    comm = {"f32": (0, 0, 0), "bf16": (1, 0, 0), "e4m3": (2, 4, 3), "e5m2": (2, 5, 2), "e2m1": (2, 2, 1),
            "e3m0": (2, 3, 0)}[args.comm]
    if comm[0]:
        scratch = torch.zeros(64, dtype=torch.int32, device=dev)
        state.close()
        state = binding.State.from_dict(st, H=w.H, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum, beta1=w.beta1,
                                        beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay, grad_kind=w.grad_kind,
                                        impl=args.kernel, comm_scratch=scratch)
    run_outer = (lambda: state.outer_quantized(variant, *comm)) if comm[0] else (lambda: state.outer(variant))
    outer_bpp = outer_bytes_per_param(variant, M, w.theta_kind)
    if comm[0] == 2:                                    # the max-|Delta_m| pass re-reads theta and start
        outer_bpp += M * ({0: 4, 1: 2, 2: 4}[w.theta_kind] + 4)
    adam_bpp = adamw_bytes_per_param(M, w.theta_kind, w.grad_kind)

    def one_step(timed):
        """Returns (ms of the whole step, ms of the outer kernel alone)."""
        if not phase:
            inputs.inner_phase_standin(st)
        flush.fill_(1)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        if phase:
            for _ in range(w.H):
                state.inner_adamw(grads, w.inner_lr)
        e1.record()
        run_outer()
        e2.record()
        if not timed:
            return None
        e2.synchronize()
        return e0.elapsed_time(e2), e1.elapsed_time(e2), e0.elapsed_time(e1)

    sampler = ClockSampler(gpu)                            # started before the warm-up: a short timed region
    t_warm = time.perf_counter()                           # may see too few 100 ms samples of its own
    for _ in range(args.warmup):
        one_step(False)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    n0 = binding.launch_count()
    t0 = time.perf_counter()
    rows = [one_step(True) for _ in range(args.steps)]
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    launches = binding.launch_count() - n0
    clocks = sampler.stop(t0, t1, t_warm)
    if world > 1:
        dist.barrier()
    step_ms = sum(r[0] for r in rows) / len(rows)
    outer_ms = sum(r[1] for r in rows) / len(rows)
    outer_sorted = sorted(r[1] for r in rows)
    outer_median, outer_min = outer_sorted[len(outer_sorted) // 2], outer_sorted[0]
    adam_ms = sum(r[2] for r in rows) / len(rows) / max(1, w.H) if phase else None
    if world > 1:
        t = torch.tensor([step_ms, outer_ms], device=red_dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        step_ms, outer_ms = float(t[0]), float(t[1])
        l = torch.tensor([launches], device=red_dev)
        dist.all_reduce(l)
        launches = int(l[0])
    P_job = P * world
    if args.strong:
        t = torch.tensor([P], device=red_dev, dtype=torch.int64)
        if world > 1:
            dist.all_reduce(t)
        P_job = int(t[0])
    value = P_job / (step_ms * 1e-3)

    # --- roofline of the dominant kernel
    peak, peak_kind = load_peak()
    if phase and adam_ms * w.H > outer_ms:
        dom, dom_ms, dom_bpp = "diloco_inner_adamw", adam_ms, adam_bpp
    else:
        dom, dom_ms, dom_bpp = f"diloco_outer_{args.variant}", outer_ms, outer_bpp
    achieved = dom_bpp * P / (dom_ms * 1e-3) / 1e9
    tr = None if comm[0] else NCU_TRAFFIC_BYTES_PER_PARAM.get((dom, M, w.theta_kind))
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_param": dom_bpp, "traffic": (tr * P if tr else None),
                "kernel_ms": dom_ms, "outer_ms_median": outer_median, "outer_ms_min": outer_min}

    # --- extra: the sibling kernels at the same shape (outer-only workloads, rank 0's GPU)
    kernels = {}
    if args.siblings and not phase:
        def time_kernel(fn, n=5):
            ms = []
            for _ in range(2 + n):
                inputs.inner_phase_standin(st)
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record(); b.synchronize()
                ms.append(a.elapsed_time(b))
            ms = ms[2:]
            return sum(ms) / len(ms)
        for name, v in (("standard", 0), ("delayed", 1), ("eager", 2)):
            ms = time_kernel(lambda v=v: state.outer(v))
            bpp = outer_bytes_per_param(v, M, w.theta_kind)
            kernels[f"outer_{name}"] = {"ms": ms, "GBps": bpp * P / ms / 1e6, "frac": bpp * P / ms / 1e6 / peak,
                                        "params_per_s": P / ms * 1e3}
        # the worker form: one replica, Delta_m sent / summed Delta received (40 B per index in fp32)
        if w.theta_kind == 0:
            sw = binding.State(M=1, P=P, stride=stride, theta=st["theta"][0], start=st["start"][0],
                               outer_mom=st["outer_mom"][0], delta_prev_local=st["delta_prev_local"].view(-1, stride)[0])
            send, recv = torch.zeros(stride, device=dev), torch.zeros(stride, device=dev)
            ms = time_kernel(lambda: sw.worker_outer_apply(binding.EAGER, M, recv, send))
            kernels["worker_outer_eager"] = {"ms": ms, "GBps": 40 * P / ms / 1e6, "frac": 40 * P / ms / 1e6 / peak,
                                             "params_per_s": P / ms * 1e3}
            sw.close(); del send, recv
        if 28 * M * stride < torch.cuda.mem_get_info(dev)[0] * 0.8:
            am = torch.zeros((M, stride), device=dev); av = torch.zeros((M, stride), device=dev)
            g = inputs.make_grads(M, P, stride, st["gen"], dev, 0)
            sa = binding.State(M=M, P=P, stride=stride, theta=st["theta"], master=st["master"], start=st["start"],
                               outer_mom=st["outer_mom"], adam_m=am, adam_v=av, theta_kind=w.theta_kind)
            ms = time_kernel(lambda: sa.inner_adamw(g, 4e-4))
            bpp = adamw_bytes_per_param(M, w.theta_kind, 0)
            kernels["inner_adamw"] = {"ms": ms, "GBps": bpp * P / ms / 1e6, "frac": bpp * P / ms / 1e6 / peak,
                                      "params_per_s": P / ms * 1e3}
            sa.close(); del am, av, g

    # --- end to end: state in pinned host memory, copies inside the timed region
    e2e = None
    if args.e2e and not phase and not comm[0]:
        keys = ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom")
        need = sum(st[k].numel() * st[k].element_size() for k in keys if st.get(k) is not None)
        try:
            pinned = {k: (torch.empty_like(st[k], device="cpu").pin_memory() if st.get(k) is not None else None) for k in keys}
            for k in keys:
                if pinned[k] is not None:
                    pinned[k].copy_(st[k])
            host = binding.make_buffers(**pinned)
            streams = [torch.cuda.Stream(device=dev) for _ in range(3)]
            torch.cuda.synchronize()
            per = []
            n_e2e = max(3, min(args.steps, 10))
            def host_step(buffers):
                """One end-to-end step, timed on the device: from the first copy-in (stream 0) to
                the last copy-out (stream 2)."""
                torch.cuda.synchronize()
                e_a, e_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e_a.record(streams[0])
                state.outer_step_host(variant, buffers, streams, args.chunk)
                e_b.record(streams[2])
                e_b.synchronize()
                return e_a.elapsed_time(e_b)

            for i in range(2 + n_e2e):
                per.append(host_step(host))
            per = per[2:]
            e_ms = sum(per) / len(per)
            if world > 1:
                t = torch.tensor([e_ms], device=red_dev, dtype=torch.float64)
                dist.all_reduce(t, op=dist.ReduceOp.MAX)
                e_ms = float(t[0])
            def leg_bytes(k):
                rows = 1 if k == "delta_prev_avg" else M
                return rows * P * pinned[k].element_size()
            used = [k for k in keys if pinned[k] is not None and not (k == "delta_prev_local" and variant != 2)
                    and not (k == "delta_prev_avg" and variant == 0)]
            h2d = sum(leg_bytes(k) for k in used if not (k == "theta" and w.theta_kind == 2))
            d2h = sum(leg_bytes(k) for k in used)
            e2e = {"value": P_job / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                   "ms_per_step": e_ms, "chunk": args.chunk, "timing": "CUDA events: first copy-in stream to last copy-out stream",
                   "pcie_GBps_each_way": h2d / e_ms / 1e6}
            # second flavour: only theta crosses PCIe, the outer-optimiser state stays on the device
            host_t = binding.make_buffers(theta=pinned["theta"], master=pinned["master"])
            per = []
            for i in range(2 + n_e2e):
                per.append(host_step(host_t))
            t_ms = sum(per[2:]) / len(per[2:])
            th_bytes = sum(leg_bytes(k) for k in ("theta", "master") if pinned[k] is not None)
            e2e["theta_only"] = {"value": P_job / (t_ms * 1e-3), "ms_per_step": t_ms, "h2d_bytes_per_step":
                                 th_bytes if w.theta_kind != 2 else leg_bytes("master"), "d2h_bytes_per_step": th_bytes,
                                 "note": "theta travels, start / momentum / previous gradients resident on the device"}
            del pinned
        except RuntimeError as ex:
            e2e = {"value": None, "unit": UNIT, "error": str(ex)[:200]}

    # --- CPU baseline: the oracle as it stands, bounded sample, rank 0 at N = 1 only
    cpu = None
    if args.cpu_baseline and world == 1:
        import oracle
        oracle.build()
        Ps = min(P, 35_000_000)
        _, h = host_state(w, Ps, w.seed)
        cores = os.cpu_count() or 1
        s_stride = inputs.padded_stride(Ps)
        time_oracle_eager(h, M, Ps, s_stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 0, 1)
        tm = time_oracle_eager(h, M, Ps, s_stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 8.0)
        t1c = time_oracle_eager(h, M, Ps, s_stride, w.theta_kind, w.outer_lr, w.outer_momentum, 1, 4.0)
        cpu = {"value": Ps / (sum(tm) / len(tm)), "unit": UNIT, "cores": cores, "kind": "oracle", "cpu_model": cpu_model(),
               "sample": f"eager outer step on M={M}, P={Ps} of {P} (all replicas, drawn on the host with the same recipe), "
                         f"{len(tm)} steps with {cores} OpenMP threads",
               "single_thread_value": Ps / (sum(t1c) / len(t1c))}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": step_ms, "higher_is_better": True, "scaling": "strong" if args.strong else "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": {"workload": args.workload, "variant": args.variant, "M": M, "P_per_gpu": P,
                           "theta": ["f32", "bf16", "f32 master + bf16 copy"][w.theta_kind],
                           "step": (f"{w.H} x inner AdamW + 1 outer {args.variant}" if phase else f"1 outer {args.variant} step"),
                           "outer_lr": w.outer_lr, "outer_momentum": w.outer_momentum,
                           "l2": "state >> 126 MB L2 and a 256 MB flush write between steps",
                           "sharding": "parameter axis split across ranks, all M replicas of an index on one rank, no collective",
                           "kernel_impl": ["auto", "direct", "bulk"][args.kernel], "outer_gradient_wire_format": args.comm},
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
                "replica_params_per_s": value * M, "kernels": kernels or None}
        print(json.dumps(line))
    state.close()
    if world > 1:
        dist.destroy_process_group()
    return 0


def report(args):
    """One bench process per workload (so that each starts from an empty device), all kernels
    of all five configurations as a table on stderr; the JSON lines go to stdout."""
    from paper_2502_12996_b200 import inputs
    rows = []
    for name, w in inputs.WORKLOADS.items():
        runs = [["--workload", name, "--steps", str(max(3, args.steps if w.P < 2e8 else 5))]]
        if w.H:
            runs = [runs[0] + ["--steps", "3"], runs[0] + ["--outer-only"]]
        for extra in runs:
            cmd = [sys.executable, str(ROOT / "bench.py"), "--no-e2e", "--no-cpu-baseline"] + extra
            out = subprocess.run(cmd, capture_output=True, text=True)
            line = [l for l in out.stdout.splitlines() if l.startswith("{")]
            if out.returncode != 0 or not line:
                rows.append((name, "failed", out.stderr[-200:]))
                continue
            print(line[-1])
            d = json.loads(line[-1])
            if d.get("skipped"):
                rows.append((name, "skipped", d["skipped"]))
                continue
            r = d["roofline"]
            rows.append((name, d["config"]["step"], f"M={d['config']['M']} P={d['config']['P_per_gpu']:,} {d['config']['theta']}",
                         r["kernel"], f"{r['kernel_ms']:.3f} ms", f"{r['achieved']:.0f} GB/s", f"{r['frac']:.3f} {r['peak_kind']}",
                         f"{r['frac_of_nominal_8000']:.3f} of nominal", f"{d['value']:.3e} params/s",
                         f"sm {d['clocks']['sm_mhz']} MHz {','.join(d['clocks']['reasons'])}"))
            for k, v in (d.get("kernels") or {}).items():
                rows.append((name, "", "", k, f"{v['ms']:.3f} ms", f"{v['GBps']:.0f} GB/s", f"{v['frac']:.3f}", "", f"{v['params_per_s']:.3e} params/s", ""))
    for r in rows:
        print(" | ".join(str(x) for x in r), file=sys.stderr)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--variant", default="eager", choices=["standard", "delayed", "eager"])
    ap.add_argument("--P", type=int, default=0, help="override the workload's parameter count (per GPU)")
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 direct, 2 bulk")
    ap.add_argument("--comm", default="f32", choices=["f32", "bf16", "e4m3", "e5m2", "e2m1", "e3m0"],
                    help="wire format of the outer gradients (quantised communication)")
    ap.add_argument("--chunk", type=int, default=64 * 16384, help="elements per chunk of the host-buffer path")
    ap.add_argument("--strong", action="store_true", help="split the workload's P across ranks instead of one full shape per rank")
    ap.add_argument("--outer-only", action="store_true", help="phase workloads: time the outer step alone")
    ap.add_argument("--no-e2e", dest="e2e", action="store_false")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--no-siblings", dest="siblings", action="store_false")
    ap.add_argument("--report", action="store_true",
                    help="run every workload (one process each) and print a table of all kernels to stderr")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.report:
        return report(args)
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
