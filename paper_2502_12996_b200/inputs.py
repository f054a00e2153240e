"""Seeded synthetic inputs for the DiLoCo outer step and inner AdamW.

This module only DRAWS numbers and lays them out; it holds none of the method's arithmetic
and is the one module that both the CUDA path's callers and the CPU oracle's callers use, so
that both sides always see the same tensors (the oracle receives copies, never a second
draw).  The synthetic vectors stand in for the flattened parameters and gradients of the
paper's transformer models (Table 5: 35M ... 1B parameters) trained on its text corpora,
which are not needed to exercise an elementwise optimiser path.

Recipe (standard deviations, not variances):
    start_m      = s0 ~ N(0, 0.02)                     identical for every replica m
    theta_m      = s0 + N(0, 1e-3)                     a stand-in for one inner phase
    dpl_m        ~ N(0, 1e-3)                          previous local outer gradients
    dpa          = (dpl_0 + ... + dpl_{M-1}) / M       what the previous all-reduce returned
    outer_mom    = 0, adam_m = adam_v = 0
    grads        ~ N(0, 1e-2), optionally times a per-segment scale 10^U(-3,-1) / 1e-2
Draw order is fixed: s0, theta noise m = 0..M-1, dpl m = 0..M-1, then per-step draws in
(step, m) order, all from one torch.Generator seeded with 12996 + config index.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

THETA_F32, THETA_BF16, THETA_MASTER_BF16 = 0, 1, 2
GRAD_F32, GRAD_BF16 = 0, 1

BASE_SEED = 12996


def padded_stride(P: int) -> int:
    """Row stride for a vector of P elements: the library needs rows that are multiples of 128
    bytes (64 elements covers bf16 rows too); rows that start on 4 KB boundaries measured 1-2 %
    faster on B200 (M = 4, 8), so the stride is rounded up to 1024 elements.  (Coarser
    alignments, up to 8 MB, were tried at the full benchmark sizes: within run-to-run noise.)"""
    return (int(P) + 1023) // 1024 * 1024


@dataclass
class Workload:
    """One (M, P) shape of one of the five benchmark configurations."""
    name: str
    config_index: int
    M: int
    P: int
    theta_kind: int = THETA_F32
    grad_kind: int = GRAD_F32
    H: int = 0                   # inner steps per phase (0: outer-only configuration)
    outer_steps: int = 3         # outer steps (= phases) the configuration runs
    outer_lr: float = 0.7
    outer_momentum: float = 0.9
    inner_lr: float = 4e-4
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    weight_decay: float = 0.1
    segments: int = 0            # > 0: per-segment gradient scales (configuration 3)
    shape_index: int = 0

    @property
    def seed(self) -> int:
        return BASE_SEED + self.config_index + 100 * self.shape_index

    @property
    def stride(self) -> int:
        return padded_stride(self.P)


WORKLOADS: Dict[str, Workload] = {w.name: w for w in [
    Workload("cfg0", 0, M=2, P=1_048_576, outer_steps=3),
    Workload("cfg1", 1, M=4, P=35_000_000, outer_steps=10),
    Workload("cfg2", 2, M=4, P=550_000_000, theta_kind=THETA_BF16, grad_kind=GRAD_BF16, H=30, outer_steps=5),
    Workload("cfg3", 3, M=4, P=1_300_000_000, theta_kind=THETA_MASTER_BF16, grad_kind=GRAD_BF16, H=100,
             outer_steps=3, segments=256),
    Workload("cfg4a", 4, M=2, P=2_400_000_000, outer_steps=3, shape_index=0),
    Workload("cfg4b", 4, M=8, P=550_000_000, outer_steps=3, shape_index=1),
    Workload("cfg4c", 4, M=16, P=150_000_000, outer_steps=3, shape_index=2),
]}


def generator(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _fill_normal_rows(dst: torch.Tensor, P: int, std: float, gen: torch.Generator, chunk: int = 1 << 26):
    """dst[m, :P] ~ N(0, std) for every row, drawn row by row, in place, in bounded chunks."""
    for m in range(dst.shape[0]):
        for a in range(0, P, chunk):
            b = min(P, a + chunk)
            dst[m, a:b].normal_(0.0, std, generator=gen)


def make_outer_state(M: int, P: int, seed: int, device="cpu", theta_kind: int = THETA_F32,
                     with_adam: bool = False, stride: Optional[int] = None,
                     gen: Optional[torch.Generator] = None, overlap_steps: int = 1) -> Dict[str, torch.Tensor]:
    """Allocate and fill every state buffer of one DiLoCo state on `device`.

    Returns a dict with keys theta, master (or None), start, delta_prev_local, delta_prev_avg,
    outer_mom, adam_m, adam_v (or None) and the generator under "gen" for further draws.
    Padding elements (index >= P) are zero.  With overlap_steps = D > 1 the previous-gradient
    buffers hold D generations, shaped [D, M, stride] and [D, stride], each drawn like the one.
    """
    stride = padded_stride(P) if stride is None else int(stride)
    dev = torch.device(device)
    gen = generator(seed, dev) if gen is None else gen
    f32 = dict(dtype=torch.float32, device=dev)
    start = torch.zeros((M, stride), **f32)
    start[0, :P].normal_(0.0, 0.02, generator=gen)
    for m in range(1, M):
        start[m, :P].copy_(start[0, :P])
    noisy = torch.zeros((M, stride), **f32)
    _fill_normal_rows(noisy, P, 1e-3, gen)
    noisy[:, :P] += start[:, :P]
    if theta_kind == THETA_F32:
        theta, master = noisy, None
    elif theta_kind == THETA_BF16:
        theta, master = noisy.to(torch.bfloat16), None
        del noisy
    else:
        theta, master = noisy.to(torch.bfloat16), noisy
    D = int(overlap_steps)
    dpl = torch.zeros((D * M, stride), **f32)
    _fill_normal_rows(dpl, P, 1e-3, gen)
    dpl = dpl.view(D, M, stride)
    dpa = torch.zeros((D, stride), **f32)
    for g in range(D):
        dpa[g].copy_(dpl[g, 0])
        for m in range(1, M):
            dpa[g] += dpl[g, m]
    dpa /= float(M)
    if D == 1:
        dpl, dpa = dpl[0], dpa[0]
    out = dict(theta=theta, master=master, start=start, delta_prev_local=dpl, delta_prev_avg=dpa,
               outer_mom=torch.zeros((M, stride), **f32), adam_m=None, adam_v=None, gen=gen,
               M=M, P=P, stride=stride, theta_kind=theta_kind)
    if with_adam:
        out["adam_m"] = torch.zeros((M, stride), **f32)
        out["adam_v"] = torch.zeros((M, stride), **f32)
    return out


def inner_phase_standin(state: Dict[str, torch.Tensor], chunk: int = 1 << 26) -> None:
    """Outer-only configurations: before each further outer step move the replicas as one
    inner phase would, theta_m <- start_m + N(0, 1e-3), with fresh draws from the state's
    generator (the rule that built the first step's replicas)."""
    M, P, gen = state["M"], state["P"], state["gen"]
    tk = state["theta_kind"]
    for m in range(M):
        for a in range(0, P, chunk):
            b = min(P, a + chunk)
            noise = torch.empty(b - a, dtype=torch.float32, device=state["start"].device)
            noise.normal_(0.0, 1e-3, generator=gen)
            noise += state["start"][m, a:b]
            if tk == THETA_F32:
                state["theta"][m, a:b].copy_(noise)
            elif tk == THETA_BF16:
                state["theta"][m, a:b].copy_(noise)          # rounds to bf16 (nearest even)
            else:
                state["master"][m, a:b].copy_(noise)
                state["theta"][m, a:b].copy_(noise)


def segment_sizes(P: int, segments: int, d_model: int = 2048) -> List[int]:
    """Tensor-like segment sizes: a transformer block's matrices and vectors cycled
    (d^2 x4, 4d^2 x2, d x4), the last segment taking the remainder so that they sum to P."""
    d = d_model
    cycle = [d * d] * 4 + [4 * d * d] * 2 + [d] * 4
    sizes, total = [], 0
    for s in range(segments - 1):
        sz = cycle[s % len(cycle)]
        if total + sz >= P:          # small P: shrink the cycle so that every segment is non-empty
            sz = max(1, (P - total) // (segments - s))
        sizes.append(sz)
        total += sz
    sizes.append(P - total)
    assert sizes[-1] > 0 and sum(sizes) == P
    return sizes


def segment_scales(segments: int, gen: torch.Generator, device) -> torch.Tensor:
    """sigma_s = 10^U(-3,-1): log-uniform on [1e-3, 1e-1], geometric mean 1e-2."""
    u = torch.empty(segments, dtype=torch.float64, device=device).uniform_(-3.0, -1.0, generator=gen)
    return torch.pow(torch.tensor(10.0, dtype=torch.float64, device=device), u).to(torch.float32)


def make_grads(M: int, P: int, gstride: int, gen: torch.Generator, device, grad_kind: int = GRAD_F32,
               out: Optional[torch.Tensor] = None, seg_sizes: Optional[List[int]] = None,
               seg_scales: Optional[torch.Tensor] = None, chunk: int = 1 << 26) -> torch.Tensor:
    """One inner step's gradients for all replicas: g ~ N(0, 1e-2), or sigma_seg(i) * N(0, 1)."""
    dt = torch.float32 if grad_kind == GRAD_F32 else torch.bfloat16
    if out is None:
        out = torch.zeros((M, gstride), dtype=dt, device=device)
    bounds = None
    if seg_sizes is not None:
        bounds = torch.tensor([0] + list(torch.tensor(seg_sizes).cumsum(0).tolist()), device=device)
    for m in range(M):
        for a in range(0, P, chunk):
            b = min(P, a + chunk)
            z = torch.empty(b - a, dtype=torch.float32, device=device)
            if bounds is None:
                z.normal_(0.0, 1e-2, generator=gen)
            else:
                z.normal_(0.0, 1.0, generator=gen)
                idx = torch.arange(a, b, device=device)
                seg = torch.bucketize(idx, bounds[1:], right=True)
                z *= seg_scales[seg]
            out[m, a:b].copy_(z)
    return out


def make_segment_grads(M: int, seg_sizes: List[int], seg_scales: List[float], gen: torch.Generator,
                       out: torch.Tensor) -> torch.Tensor:
    """g_i = sigma_seg(i) * N(0, 1), drawn segment by segment straight into `out` [M, >= P]
    (no full-size temporaries: for vectors that nearly fill the device)."""
    for m in range(M):
        lo = 0
        for size, sigma in zip(seg_sizes, seg_scales):
            out[m, lo:lo + size].normal_(0.0, float(sigma), generator=gen)
            lo += size
    return out
