#!/usr/bin/env python
"""Benchmark of the DiLoCo outer step with eager updates (and the kernels around it) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4a] [--impl ours|reference]

One "step" is one fused eager outer step (Algorithm 3, lines 7-12: local outer gradients,
M-way mean, eager combination, Nesterov update, replica reset) over all M replicas of the
workload; between steps an untimed stand-in for the inner phase moves the replicas
(theta_m <- start_m + N(0, 1e-3)) and a 256 MB buffer is written to flush L2.  For the
phase workloads (cfg2, cfg3) a step is H fused AdamW steps followed by the eager outer step.

The default workload is the largest outer-step shape of the five configurations that fits one
GPU (cfg4a: M = 2, P = 2.4e9 fp32, 86 GB of state).  Prints ONE JSON line.  `value` is flat
parameters advanced per second (P / t), whole job (sum over ranks); `roofline` compares the
algorithmic bytes of the dominant kernel with the measured HBM copy peak; `e2e` is the same
step through diloco_outer_step_host with the state in pinned host memory (copies inside the
timed region); `cpu_baseline` is the CPU oracle timed on this machine's host cores; `shapes`
(default single-GPU run only) holds the same kernel measurements for every other headline
shape - cfg1, cfg4b, cfg4c, the cfg2 and cfg3 phases, cfg0 cold and warm - each with the
clock samples of its own timed region, and `replica_sweep` the eager step at the replica counts
in between (M = 1 ... 64), one figure per kernel form.

With --impl reference the CPU oracle itself is timed on the same workload (there is no
reference implementation of this path; the paper ships no code).
"""
from __future__ import annotations

import argparse
import gc
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
L2_BYTES = 126 << 20
DEFAULT_WORKLOAD = "cfg4a"
THETA_NAMES = ["f32", "bf16", "f32 master + bf16 copy"]
KERNEL_IMPLS = ["auto", "direct", "bulk (1-D TMA rows)", "split R2", "split R4", "tensor (2-D TMA) T256", "tensor T128",
                "tensor T64"]
VARIANTS = {"standard": 0, "delayed": 1, "eager": 2}
# measured DRAM traffic per parameter index, one row per profiled kernel form
TRAFFIC_TABLE = ROOT / "profiles" / "ncu_dram_bytes_per_index.txt"


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


def state_bytes_per_param(M: int, theta_kind: int, variant: int = 2) -> int:
    th = {0: 4, 1: 2, 2: 6}[theta_kind]
    return M * (th + 8 + (4 if variant == 2 else 0)) + (4 if variant else 0)


def load_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def load_traffic():
    """(kernel, variant, M, theta_kind) -> (DRAM bytes per index from an ncu capture, source).
    The table is plain text: kernel variant M theta_kind bytes_per_index source."""
    table = {}
    try:
        for line in TRAFFIC_TABLE.read_text().splitlines():
            f = line.split()
            if len(f) < 6 or line.lstrip().startswith("#"):
                continue
            table[(f[0], f[1], int(f[2]), int(f[3]))] = (float(f[4]), f[5])
    except OSError:
        pass
    return table


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 100 ms for the whole run; every timed
    region asks for the samples of its own window."""
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

    def window(self, t0: float, t1: float, t_fallback: float = None):
        """Median SM clock and the throttle reasons seen between t0 and t1 (a region shorter than
        three samples falls back to the window that began with its warm-up, at t_fallback)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.25]
        window = "timed region"
        if len(rows) < 3 and t_fallback is not None:       # under load since the warm-up began
            rows = [r for (t, r) in self.rows if t_fallback <= t <= t1 + 0.25]
            window = "warm-up + timed region"
        if not rows:
            rows, window = [r for (_, r) in self.rows], "whole run"
        mhz, mx, watts, reasons = [], None, [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                mhz.append(float(r[0]))
                mx = float(r[1])
                watts.append(float(r[2]))
            except Exception:
                continue
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        mhz.sort()
        return {"sm_mhz": (mhz[len(mhz) // 2] if mhz else None), "sm_max_mhz": mx, "reasons": sorted(reasons),
                "power_w_max": (max(watts) if watts else None), "samples": len(mhz), "window": window}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def mem_available_bytes() -> int:
    """Host memory this process may still take: MemAvailable, capped by what the control group
    (a container's memory limit) has left, whichever is smaller."""
    avail = 0
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                avail = int(line.split()[1]) * 1024
    except OSError:
        pass
    for limit_file, usage_file in (("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory.current"),
                                   ("/sys/fs/cgroup/memory/memory.limit_in_bytes",
                                    "/sys/fs/cgroup/memory/memory.usage_in_bytes")):
        try:
            limit = open(limit_file).read().strip()
            if limit == "max":
                continue
            left = int(limit) - int(open(usage_file).read().strip())
            if 0 < int(limit) < (1 << 60):
                avail = min(avail, max(0, left)) if avail else max(0, left)
        except (OSError, ValueError):
            continue
    return avail


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def shard_bounds(P_total: int, world: int, rank: int, quantum: int = 64):
    """Contiguous, quantum-aligned ranges of the parameter axis, one per rank (all M replicas'
    slices live on the same rank, so no step of the path crosses ranks)."""
    q = (P_total + quantum - 1) // quantum
    lo = (q * rank // world) * quantum
    hi = min(P_total, (q * (rank + 1) // world) * quantum)
    return lo, hi


def workload_of(args, inputs):
    """The named workload, with its replica count replaced if --M was given (other kernel forms)."""
    import dataclasses
    w = inputs.WORKLOADS[args.workload]
    return dataclasses.replace(w, M=args.M) if getattr(args, "M", 0) else w


def config_dict(args, w, P_per_gpu: int) -> dict:
    """What the workload is; the same dict in both arms (GPU path and CPU reference)."""
    phase = w.H > 0 and not args.outer_only
    state = state_bytes_per_param(w.M, w.theta_kind) * P_per_gpu
    l2 = ("state >> 126 MB L2" if state > 4 * L2_BYTES else "state fits the 126 MB L2: cold-L2 figure") \
        + ", 256 MB flush write before every timed step"
    return {"workload": args.workload, "variant": args.variant, "M": w.M, "P_per_gpu": P_per_gpu,
            "theta": THETA_NAMES[w.theta_kind],
            "step": (f"{w.H} x inner AdamW + 1 outer {args.variant}" if phase else f"1 outer {args.variant} step"),
            "outer_lr": w.outer_lr, "outer_momentum": w.outer_momentum, "l2": l2,
            "sharding": "one full shape per rank (weak scaling), all M replicas of an index on one rank, no collective"
            if not args.strong else "parameter axis split across ranks, all M replicas of an index on one rank, no collective",
            "kernel_impl": KERNEL_IMPLS[args.kernel], "outer_gradient_wire_format": args.comm}


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


def oracle_sample_size(w, P: int) -> int:
    """Bounded sample of a workload for the CPU oracle: the per-parameter cost of the elementwise
    path does not depend on P, so large shapes are timed on the first 1.4e8 / M parameters of
    every replica (a few seconds per step on 16 cores)."""
    return min(P, 140_000_000 // w.M)


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    from paper_2502_12996_b200 import inputs
    oracle.build()
    w = workload_of(args, inputs)
    P_cfg = args.P or w.P
    P = oracle_sample_size(w, P_cfg)
    cores = os.cpu_count() or 1
    st, h = host_state(w, P, w.seed)
    stride = st["stride"]
    for _ in range(max(1, min(args.warmup, 3))):
        time_oracle_eager(h, w.M, P, stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 0, 1)
    times = time_oracle_eager(h, w.M, P, stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 1e9, args.steps)
    ms = 1e3 * sum(times) / len(times)
    value = P / (ms * 1e-3)
    sample = (f"eager outer step on the first {P} of {P_cfg} parameters of all {w.M} replicas "
              f"({len(times)} steps, {cores} OpenMP threads); per-parameter cost does not depend on P")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": config_dict(args, w, P_cfg),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "cpu_model": cpu_model()},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
            "note": "the paper ships no code: the reference arm is the CPU oracle (plain C, -O2, no FMA) on the host cores; "
                    "ms_per_step is the time of one step over the sample"}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------ GPU arm
COMM = {"f32": (0, 0, 0), "bf16": (1, 0, 0), "e4m3": (2, 4, 3), "e5m2": (2, 5, 2), "e2m1": (2, 2, 1), "e3m0": (2, 3, 0)}


def stats(xs):
    s = sorted(xs)
    return {"mean": sum(s) / len(s), "median": s[len(s) // 2], "min": s[0], "max": s[-1], "n": len(s)}


class Shape:
    """One workload resident on the device: state, library handle, gradients, and the timed loop."""

    def __init__(self, name, args, dev, rank, world, P=None, phase=None, variant=None, comm="f32", workload=None):
        import torch
        from paper_2502_12996_b200 import binding, inputs
        self.torch, self.binding, self.inputs = torch, binding, inputs
        self.name, self.dev = name, dev
        w = self.w = workload or inputs.WORKLOADS[name]
        self.P = P or w.P
        if args.strong and P is None:
            lo, hi = shard_bounds(self.P, world, rank)
            self.P = hi - lo
        self.variant = VARIANTS[args.variant] if variant is None else variant
        self.phase = (w.H > 0 and not args.outer_only) if phase is None else phase
        self.comm = COMM[comm]
        self.kernel = args.kernel
        self.seed = w.seed + 1000 * rank
        self.st = self.state = self.grads = self.scratch = self.status = None

    def need_bytes(self):
        w, M, P = self.w, self.w.M, self.P
        th = {0: 4, 1: 2, 2: 6}[w.theta_kind]
        per = th + 12 + ((8 + (2 if w.grad_kind else 4)) if self.phase else 0)
        # state + one [M, P] fp32 temporary of the generator + stand-in chunks + the L2 flush buffer
        return M * P * per + 4 * P + M * P * 4 + (768 << 20)

    def fits(self):
        free = self.torch.cuda.mem_get_info(self.dev)[0]
        need = self.need_bytes()
        return (need <= free), f"needs {need / 2**30:.1f} GiB of device memory, {free / 2**30:.1f} GiB free"

    def allocate(self):
        torch, binding, inputs, w = self.torch, self.binding, self.inputs, self.w
        st = self.st = inputs.make_outer_state(w.M, self.P, self.seed, device=self.dev, theta_kind=w.theta_kind,
                                               with_adam=self.phase)
        kw = dict(H=w.H, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                  weight_decay=w.weight_decay, grad_kind=w.grad_kind, impl=self.kernel)
        if self.comm[0]:
            self.scratch = torch.zeros(64, dtype=torch.int32, device=self.dev)
            kw["comm_scratch"] = self.scratch
        if self.kernel in (2, 5, 6, 7):                     # the staged forms report a timed-out wait here
            self.status = torch.zeros(1, dtype=torch.int32, device=self.dev)
            kw["device_status"] = self.status
        self.state = binding.State.from_dict(st, **kw)
        if self.phase:
            if w.segments:
                self.grads = torch.zeros((w.M, st["stride"]), dtype=torch.bfloat16 if w.grad_kind else torch.float32,
                                         device=self.dev)
                inputs.make_segment_grads(w.M, inputs.segment_sizes(self.P, w.segments),
                                          inputs.segment_scales(w.segments, st["gen"], self.dev).tolist(), st["gen"],
                                          self.grads)
            else:
                self.grads = inputs.make_grads(w.M, self.P, st["stride"], st["gen"], self.dev, w.grad_kind)
        return self

    def free(self):
        if self.state is not None:
            self.state.close()
        self.st = self.state = self.grads = self.scratch = None
        gc.collect()
        self.torch.cuda.empty_cache()

    def run_outer(self):
        if self.comm[0]:
            self.state.outer_quantized(self.variant, *self.comm)
        else:
            self.state.outer(self.variant)

    def one_step(self, flush, timed=True, move=True, do_flush=True):
        """(ms of the whole step, ms of the outer kernel, ms of the H AdamW steps), CUDA events on
        the launching stream; the stand-in for the inner phase and the L2 flush are outside them."""
        torch = self.torch
        if not self.phase and move:
            self.inputs.inner_phase_standin(self.st)
        if do_flush:
            flush.fill_(1)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        if self.phase:
            for _ in range(self.w.H):
                self.state.inner_adamw(self.grads, self.w.inner_lr)
        e1.record()
        self.run_outer()
        e2.record()
        if not timed:
            return None
        e2.synchronize()
        return e0.elapsed_time(e2), e1.elapsed_time(e2), e0.elapsed_time(e1)

    def bytes_per_param(self):
        w = self.w
        outer = outer_bytes_per_param(self.variant, w.M, w.theta_kind)
        if self.comm[0] == 2:                                    # the max-|Delta_m| pass re-reads theta and start
            outer += w.M * ({0: 4, 1: 2, 2: 4}[w.theta_kind] + 4)
        return outer, adamw_bytes_per_param(w.M, w.theta_kind, w.grad_kind)

    def measure(self, flush, sampler, steps, warmup, barrier=None, move=True, do_flush=True):
        """warmup untimed steps, then `steps` timed ones; returns the per-step rows, the launch
        count of the timed region and the clock samples of that region."""
        torch, binding = self.torch, self.binding
        t_warm = time.perf_counter()
        for _ in range(warmup):
            self.one_step(flush, timed=False, move=move, do_flush=do_flush)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        n0 = binding.launch_count()
        t0 = time.perf_counter()
        rows = [self.one_step(flush, move=move, do_flush=do_flush) for _ in range(steps)]
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        launches = binding.launch_count() - n0
        if barrier:
            barrier()
        self.state.check_device_status()                    # raises if a staged form gave up a wait
        return rows, launches, sampler.window(t0, t1, t_warm)

    def record(self, rows, clocks, peak, traffic):
        """The figures of one shape as they go into the JSON line (rounded: the line carries many)."""
        w, P = self.w, self.P
        outer_bpp, adam_bpp = self.bytes_per_param()
        outer = stats([r[1] for r in rows])
        vname = [k for k, v in VARIANTS.items() if v == self.variant][0]
        in_l2 = state_bytes_per_param(w.M, w.theta_kind) * P <= 4 * L2_BYTES   # ncu's per-index DRAM traffic was

        def kernel(name, ms, bpp, key):                                         # captured on HBM-resident sizes
            gbs = bpp * P / (ms["mean"] * 1e-3) / 1e9
            tr = None if in_l2 else traffic.get(key)
            return {"kernel": name, "ms": {k: round(ms[k], 5) for k in ("mean", "median", "min")}, "n": ms["n"],
                    "algorithmic_bytes_per_param": bpp, "GBps": round(gbs, 1), "frac": round(gbs / peak, 4),
                    "frac_of_nominal_8000": round(gbs / NOMINAL_HBM_GBS, 4),
                    "ncu_dram_bytes_per_param": (tr[0] if tr else None)}
        step = stats([r[0] for r in rows])
        rec = {"M": w.M, "P": P, "theta": THETA_NAMES[w.theta_kind],
               "state_GB": round(state_bytes_per_param(w.M, w.theta_kind) * P / 1e9, 2),
               "step_ms": round(step["mean"], 5), "params_per_s": round(P / (step["mean"] * 1e-3), 1),
               "outer": kernel(f"diloco_outer_{vname}", outer, outer_bpp,
                               ("outer", vname, w.M, w.theta_kind) if not self.comm[0] else None),
               "clocks": {k: clocks.get(k) for k in ("sm_mhz", "reasons", "power_w_max", "samples")}}
        if self.phase:
            adam = stats([r[2] / w.H for r in rows])
            rec["adamw"] = kernel("diloco_inner_adamw", adam, adam_bpp, ("adamw", "-", w.M, w.theta_kind))
            rec["step"] = f"{w.H} x inner AdamW + 1 outer {vname}"
        else:
            rec["step"] = f"1 outer {vname} step"
        return rec


class HostBuffer:
    """A page-locked host tensor of exactly the size asked for.  The caching pinned allocator
    rounds every request up to a power of two, which would double an 86 GB state, so the memory
    is an anonymous mapping that is advised to use huge pages (on this pool plain 4 KB pages cost
    the copies 15-20 % of their PCIe rate: 35 against 43 GB/s each way) and then page-locked in
    place with cudaHostRegister."""

    def __init__(self, torch, like):
        import mmap
        self.torch = torch
        nbytes = like.numel() * like.element_size()
        huge = 2 << 20
        self.map = mmap.mmap(-1, max(huge, (nbytes + huge - 1) // huge * huge))
        try:
            self.map.madvise(mmap.MADV_HUGEPAGE)
        except (AttributeError, OSError, ValueError):
            pass                                            # no transparent huge pages here: 4 KB pages then
        self.tensor = torch.frombuffer(self.map, dtype=like.dtype, count=like.numel()).view(like.shape)
        rc = torch.cuda.cudart().cudaHostRegister(self.tensor.data_ptr(), nbytes, 0)
        if int(rc) != 0:
            raise RuntimeError(f"cudaHostRegister failed with {rc}")
        self.tensor.copy_(like)

    def release(self):
        try:
            self.torch.cuda.cudart().cudaHostUnregister(self.tensor.data_ptr())
        except Exception:
            pass
        self.tensor = None                                  # the mapping goes with the last reference to it


def run_e2e(shape, args, world, dist, red_dev, n_steps):
    """The same outer step through diloco_outer_step_host: the state lives in pinned HOST memory,
    every step copies what the step reads to the device, runs the kernel chunk by chunk and
    copies what it wrote back, all inside the timed region."""
    torch, binding = shape.torch, shape.binding
    st, w, P, M, variant = shape.st, shape.w, shape.P, shape.w.M, shape.variant
    keys = ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom")
    pinned, owners, t_pin = {}, [], time.perf_counter()
    try:
        for k in keys:
            if st.get(k) is None:
                pinned[k] = None
                continue
            owners.append(HostBuffer(torch, st[k]))
            pinned[k] = owners[-1].tensor
        t_pin = time.perf_counter() - t_pin
        host = binding.make_buffers(**pinned)
        streams = [torch.cuda.Stream(device=shape.dev) for _ in range(3)]
        torch.cuda.synchronize()

        def host_step(buffers):
            """One end-to-end step, timed on the device: from the first copy-in (stream 0) to the
            last copy-out (stream 2)."""
            torch.cuda.synchronize()
            e_a, e_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e_a.record(streams[0])
            shape.state.outer_step_host(variant, buffers, streams, args.chunk)
            e_b.record(streams[2])
            e_b.synchronize()
            return e_a.elapsed_time(e_b)

        def leg_bytes(k):
            rows = 1 if k == "delta_prev_avg" else M
            return rows * P * pinned[k].element_size()

        per = [host_step(host) for _ in range(2 + n_steps)][2:]
        e_ms = sum(per) / len(per)
        if world > 1:
            t = torch.tensor([e_ms], device=red_dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e_ms = float(t[0])
        used = [k for k in keys if pinned[k] is not None and not (k == "delta_prev_local" and variant != 2)
                and not (k == "delta_prev_avg" and variant == 0)]
        h2d = sum(leg_bytes(k) for k in used if not (k == "theta" and w.theta_kind == 2))
        d2h = sum(leg_bytes(k) for k in used)
        e2e = {"value": P * world / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "workload": shape.name, "M": M, "P_per_gpu": P, "ms_per_step": e_ms, "steps": len(per), "chunk": args.chunk,
               "call": "diloco_outer_step_host: whole state in pinned host memory, copied in and out every step",
               "timing": "CUDA events: first copy-in stream to last copy-out stream",
               "pcie_GBps_each_way": h2d / e_ms / 1e6, "host_register_s": t_pin,
               "host_memory": "anonymous mappings advised to huge pages, page-locked with cudaHostRegister"}
        # second flavour: only theta crosses PCIe, the outer-optimiser state stays on the device
        host_t = binding.make_buffers(theta=pinned["theta"], master=pinned["master"])
        per = [host_step(host_t) for _ in range(2 + n_steps)][2:]
        t_ms = sum(per) / len(per)
        th_bytes = sum(leg_bytes(k) for k in ("theta", "master") if pinned[k] is not None)
        e2e["theta_only"] = {"value": P * world / (t_ms * 1e-3), "ms_per_step": t_ms, "h2d_bytes_per_step":
                             th_bytes if w.theta_kind != 2 else leg_bytes("master"), "d2h_bytes_per_step": th_bytes,
                             "note": "theta travels, start / momentum / previous gradients resident on the device"}
        torch.cuda.synchronize()
        return e2e
    except Exception as ex:                                 # the end-to-end leg must never take the bench line with it
        return {"value": None, "unit": UNIT, "workload": shape.name, "error": f"{type(ex).__name__}: {ex}"[:200]}
    finally:
        host = host_t = None
        pinned.clear()
        for o in owners:
            o.release()
        owners.clear()
        gc.collect()


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
    barrier = dist.barrier if world > 1 else None
    peak, peak_kind = load_peak()
    traffic = load_traffic()
    w = workload_of(args, inputs)

    main = Shape(args.workload, args, dev, rank, world, P=args.P or None, comm=args.comm, workload=w)
    ok, why = main.fits()
    if world > 1:                                           # every rank must take the same branch
        t = torch.tensor([0 if ok else 1], device=red_dev)
        dist.all_reduce(t)
        ok = int(t[0]) == 0
    if not ok:                                              # report, never run the device out of memory
        if rank == 0:
            print(json.dumps({"metric": METRIC, "unit": UNIT, "value": None, "n_gpus": world,
                              "config": config_dict(args, w, main.P), "skipped": why}))
        return 0
    sampler = ClockSampler(gpu)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    main.allocate()
    rows, launches, clocks = main.measure(flush, sampler, args.steps, args.warmup, barrier)
    main_rec = main.record(rows, clocks, peak, traffic)
    step_ms = sum(r[0] for r in rows) / len(rows)
    outer_ms = sum(r[1] for r in rows) / len(rows)
    P, M, phase = main.P, w.M, main.phase
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
    dom = main_rec["adamw"] if (phase and main_rec["adamw"]["ms"]["mean"] * w.H > outer_ms) else main_rec["outer"]
    dom_ms = dom["ms"]["mean"] if dom is not main_rec["outer"] else outer_ms
    achieved = dom["algorithmic_bytes_per_param"] * P / (dom_ms * 1e-3) / 1e9
    tr = dom["ncu_dram_bytes_per_param"]
    tr_src = traffic.get(("adamw", "-", M, w.theta_kind) if dom is not main_rec["outer"] else ("outer", args.variant, M, w.theta_kind))
    roofline = {"bound": "hbm", "kernel": dom["kernel"], "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_param": dom["algorithmic_bytes_per_param"], "traffic": (tr * P if tr else None),
                "traffic_source": (f"ncu dram bytes per index of {tr_src[1]} x P" if tr and tr_src else None),
                "kernel_ms": dom_ms, "outer_ms_median": main_rec["outer"]["ms"]["median"],
                "outer_ms_min": main_rec["outer"]["ms"]["min"]}
    if roofline["frac"] > 1.0:
        roofline["frac_note"] = ("above 1: the denominator is a plain device copy (torch copy_), a reference point and "
                                 "not a ceiling; see frac_of_nominal_8000 and copy_gbs_this_run")

    # --- extra: the sibling kernels at the same shape (outer-only workloads, explicit request)
    kernels = {}
    if args.siblings and not phase:
        st = main.st
        state, stride = main.state, st["stride"]

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
        for name, v in VARIANTS.items():
            ms = time_kernel(lambda v=v: state.outer(v))
            bpp = outer_bytes_per_param(v, M, w.theta_kind)
            kernels[f"outer_{name}"] = {"ms": ms, "GBps": bpp * P / ms / 1e6, "frac": bpp * P / ms / 1e6 / peak,
                                        "params_per_s": P / ms * 1e3}
        # the standard step with one shared copy of start and momentum (8 M + 16 B per index in fp32)
        if w.theta_kind == 0:
            ss = binding.State(M=M, P=P, stride=stride, theta=st["theta"], start=st["start"][0], outer_mom=st["outer_mom"][0],
                               shared_outer_state=True)
            ms = time_kernel(lambda: ss.outer_standard())
            bpp = 8 * M + 16
            kernels["outer_standard_shared_state"] = {"ms": ms, "GBps": bpp * P / ms / 1e6, "frac": bpp * P / ms / 1e6 / peak,
                                                      "params_per_s": P / ms * 1e3}
            ss.close()
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

    # --- end to end: state in pinned host memory, copies inside the timed region.  On the main
    # workload if its state may be page-locked (a fraction of the host's available memory, shared
    # by the ranks of this node), else on the largest other eager shape that may, and says which.
    e2e, e2e_shape = None, None
    if args.e2e and not phase and not main.comm[0]:
        budget = mem_available_bytes() * args.e2e_host_fraction / max(1, int(os.environ.get("LOCAL_WORLD_SIZE", world)))
        order = [args.workload] + [n for n in ("cfg4a", "cfg4b", "cfg4c", "cfg1", "cfg0") if n != args.workload]
        if args.P:
            order = [args.workload]
        idx = len(order)
        for i, n in enumerate(order):
            Pn = main.P if n == args.workload else inputs.WORKLOADS[n].P
            wn = inputs.WORKLOADS[n]
            if wn.H == 0 and state_bytes_per_param(wn.M, wn.theta_kind) * Pn <= budget:
                idx = i
                break
        if world > 1:                                       # every rank must run the same shape: the smallest choice wins
            t = torch.tensor([idx], device=red_dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            idx = int(t[0])
        pick = order[idx] if idx < len(order) else None
        if pick == args.workload:
            e2e = run_e2e(main, args, world, dist, red_dev, max(3, min(args.steps, 10 if main.P < 2e8 else 3)))
            if e2e.get("value") is None and world == 1 and not args.P and args.workload != "cfg1":
                e2e, e2e_shape = None, "cfg1"                 # page-locking failed: a small shape instead
        elif pick is not None:
            e2e_shape = pick                                   # measured below, once the main state is freed
        else:
            e2e = {"value": None, "unit": UNIT, "error": f"no shape fits {budget / 2**30:.0f} GiB of pinned host memory"}
    main.free()
    if e2e_shape is not None:
        sh = Shape(e2e_shape, args, dev, rank, world)
        ok, why = sh.fits()
        if ok:
            sh.allocate()
            e2e = run_e2e(sh, args, world, dist, red_dev, 3)
            e2e["note"] = (f"{args.workload}'s state could not be page-locked on this host; measured on "
                           f"{e2e_shape}, the largest eager shape that could")
        else:
            e2e = {"value": None, "unit": UNIT, "workload": e2e_shape, "error": why}
        sh.free()

    # --- the other headline shapes, each measured like the main one, with its own clock record
    shapes = {}
    if args.shapes and world == 1 and not args.P and not args.M:
        shapes[args.workload] = main_rec
        plan = [("cfg1", None, 10), ("cfg4a", None, 10), ("cfg4b", None, 10), ("cfg4c", None, 10),
                ("cfg2", True, 3), ("cfg3", True, 3)]
        for name, ph, n in plan:
            if name == args.workload and ph is None:
                continue
            sh = Shape(name, args, dev, rank, world, phase=ph, variant=2)
            ok, why = sh.fits()
            if not ok:
                shapes[name] = {"skipped": why}
                continue
            try:
                sh.allocate()
                r, _, c = sh.measure(flush, sampler, min(args.steps, n), 3)
                shapes[name] = sh.record(r, c, peak, traffic)
            except Exception as ex:                             # e.g. an allocation that fails after the pre-check
                shapes[name] = {"skipped": f"{type(ex).__name__}: {ex}"[:200]}
            sh.free()
        # cfg0: 37.7 MB of state, smaller than L2.  Cold = as everywhere (replicas moved, L2 flushed
        # before each step); warm = the same launches back to back on an L2-resident state.
        sh = Shape("cfg0", args, dev, rank, world, variant=2)
        try:
            sh.allocate()
            r, _, c = sh.measure(flush, sampler, 20, 3)
            cold = sh.record(r, c, peak, traffic)
            r, _, c = sh.measure(flush, sampler, 50, 5, move=False, do_flush=False)
            warm = sh.record(r, c, peak, traffic)
            shapes["cfg0"] = dict(cold, l2="cold: L2 flushed before every step",
                                  warm_l2={"outer": warm["outer"], "clocks": warm["clocks"],
                                           "l2": "warm: back-to-back launches, state resident in L2; GB/s is not HBM bandwidth"})
        except Exception as ex:
            shapes["cfg0"] = {"skipped": f"{type(ex).__name__}: {ex}"[:200]}
        sh.free()

    # --- the eager step at the replica counts between and beyond the configurations' (fp32, 6e8 / M
    # parameters: about 20 GB of traffic per step), so that every kernel form has a figure in this line
    sweep = {}
    if args.shapes and world == 1 and not args.P and not args.M:
        for M_ in (1, 3, 5, 6, 7, 9, 11, 12, 13, 20, 24, 32, 64):
            wl = inputs.Workload(f"sweep_M{M_}", 9, M=M_, P=int(6e8 / M_) // 1024 * 1024 + 3, shape_index=M_)
            sh = Shape(wl.name, args, dev, rank, world, variant=2, workload=wl)
            if not sh.fits()[0]:
                continue
            try:
                sh.allocate()
                r, _, c = sh.measure(flush, sampler, 5, 3)
                o = sh.record(r, c, peak, traffic)["outer"]
                sweep[str(M_)] = {"P": sh.P, "ms": round(o["ms"]["mean"], 4), "GBps": o["GBps"],
                                  "frac_of_nominal_8000": o["frac_of_nominal_8000"], "sm_mhz": c["sm_mhz"]}
            except Exception as ex:
                sweep[str(M_)] = {"skipped": f"{type(ex).__name__}: {ex}"[:120]}
            sh.free()

    # --- a plain device copy measured in this run, the same way the recorded peak was
    copy_gbs = None
    if world == 1:
        n = 1 << 30
        if torch.cuda.mem_get_info(dev)[0] > 6 * n:
            a = torch.empty(n, dtype=torch.bfloat16, device=dev); b = torch.empty_like(a)
            a.fill_(1)
            best = 1e9
            for _ in range(10):
                x, y = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                x.record(); b.copy_(a); y.record(); y.synchronize()
                best = min(best, x.elapsed_time(y))
            copy_gbs = 2 * 2 * n / best / 1e6
            del a, b

    # --- CPU baseline: the oracle as it stands, bounded sample, rank 0 at N = 1 only
    cpu = None
    if args.cpu_baseline and world == 1:
        import oracle
        oracle.build()
        Ps = oracle_sample_size(w, P)
        _, h = host_state(w, Ps, w.seed)
        cores = os.cpu_count() or 1
        s_stride = inputs.padded_stride(Ps)
        time_oracle_eager(h, M, Ps, s_stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 0, 1)
        tm = time_oracle_eager(h, M, Ps, s_stride, w.theta_kind, w.outer_lr, w.outer_momentum, cores, 8.0)
        t1c = time_oracle_eager(h, M, Ps, s_stride, w.theta_kind, w.outer_lr, w.outer_momentum, 1, 4.0)
        cpu = {"value": Ps / (sum(tm) / len(tm)), "unit": UNIT, "cores": cores, "kind": "oracle", "cpu_model": cpu_model(),
               "sample": f"eager outer step on the first {Ps} of {P} parameters of all {M} replicas (drawn on the host "
                         f"with the same recipe), {len(tm)} steps with {cores} OpenMP threads",
               "single_thread_value": Ps / (sum(t1c) / len(t1c))}
    sampler.stop()

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": step_ms, "higher_is_better": True, "scaling": "strong" if args.strong else "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic", "config": config_dict(args, w, P),
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
                "replica_params_per_s": value * M, "copy_gbs_this_run": copy_gbs, "kernels": kernels or None,
                "shapes": shapes or None, "replica_sweep": sweep or None}
        print(json.dumps(line))
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
            cmd = [sys.executable, str(ROOT / "bench.py"), "--no-e2e", "--no-cpu-baseline", "--no-shapes", "--siblings"] + extra
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
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--variant", default="eager", choices=list(VARIANTS))
    ap.add_argument("--P", type=int, default=0, help="override the workload's parameter count (per GPU)")
    ap.add_argument("--M", type=int, default=0, help="override the workload's replica count (1 .. 64)")
    ap.add_argument("--kernel", type=int, default=0, choices=range(len(KERNEL_IMPLS)),
                    help="kernel form, DILOCO_IMPL_*: " + ", ".join(f"{i} {n}" for i, n in enumerate(KERNEL_IMPLS)))
    ap.add_argument("--comm", default="f32", choices=list(COMM),
                    help="wire format of the outer gradients (quantised communication)")
    ap.add_argument("--chunk", type=int, default=64 * 65536,
                    help="elements per chunk of the host-buffer path (4 Mi: 16 MB copies measured 7 %% faster than 4 MB ones)")
    ap.add_argument("--e2e-host-fraction", type=float, default=0.5,
                    help="share of the host's available memory that the end-to-end leg may page-lock")
    ap.add_argument("--strong", action="store_true", help="split the workload's P across ranks instead of one full shape per rank")
    ap.add_argument("--outer-only", action="store_true", help="phase workloads: time the outer step alone")
    ap.add_argument("--no-e2e", dest="e2e", action="store_false")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--no-shapes", dest="shapes", action="store_false",
                    help="skip the record of the other headline shapes (single-GPU default run)")
    ap.add_argument("--siblings", action="store_true", help="also time the sibling kernels at the main shape")
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
