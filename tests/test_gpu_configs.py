"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Configurations 0 and 1 are compared in full.  Configurations 2-4 (50-150 GB of state) are
compared on index slices gathered from the device before and after: every parameter index is
independent of every other (the only reduction runs over the replica axis at a fixed index),
so the oracle run on the gathered columns must reproduce exactly those columns of the full
GPU run.  Slices: the first and last 2^20 indices (ragged tail included), +-4096 around every
place where a per-row index or a flattened [M, stride] element offset crosses 2^30, 2^31,
2^32 or 2^33 (64-bit indexing), +-64 around every gradient-segment boundary, and 64 seeded
random blocks of 2^16 indices.
"""
import numpy as np
import pytest
import torch

from paper_2502_12996_b200 import binding, inputs
from gpu_util import assert_state_equal, host_copy, oracle_adamw, oracle_outer, to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
STATE_KEYS = ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom", "adam_m", "adam_v")


def need_gpu_bytes(n):
    import gc
    gc.collect()
    torch.cuda.empty_cache()            # earlier tests' freed blocks are still cached by torch
    free, _ = torch.cuda.mem_get_info(0)
    if free < n * 1.03 + (2 << 30):
        pytest.skip(f"needs {n / 2**30:.1f} GiB of device memory, {free / 2**30:.1f} GiB free")


def slice_index(M, P, stride, seed, extra_points=()):
    """Sorted unique parameter indices of the slices described in the module docstring."""
    rng = np.random.default_rng(seed)
    ranges = [(0, min(P, 1 << 20)), (max(0, P - (1 << 20) - 3), P)]
    for B in (1 << 30, 1 << 31, 1 << 32, 1 << 33):
        for m in range(M):
            i = B - m * stride                     # flattened offset m*stride + i crosses B here
            if 0 <= i < P:
                ranges.append((max(0, i - 4096), min(P, i + 4096)))
    for p in extra_points:
        ranges.append((max(0, p - 64), min(P, p + 64)))
    nblocks = P >> 16
    if nblocks > 64:
        for b in rng.choice(nblocks, size=64, replace=False):
            ranges.append((int(b) << 16, (int(b) + 1) << 16))
    idx = np.unique(np.concatenate([np.arange(a, b, dtype=np.int64) for a, b in ranges]))
    return idx


class SliceMirror:
    """Host mirror of the columns `idx` of a device state, laid out compactly for the oracle."""

    def __init__(self, st, idx):
        self.idx_np = idx
        self.idx = torch.from_numpy(idx).to(DEV)
        self.n = len(idx)
        self.stride = inputs.padded_stride(self.n)
        self.h = {k: self.gather(st.get(k)) for k in STATE_KEYS}

    def gather(self, t):
        if t is None:
            return None
        if t.dim() == 1:
            g = t[self.idx]
            out = np.zeros(self.stride, dtype=np.float32)
            out[:self.n] = g.cpu().numpy()
            return out
        g = t[:, self.idx]
        if t.dtype == torch.bfloat16:
            out = np.zeros((t.shape[0], self.stride), dtype=np.uint16)
            out[:, :self.n] = g.view(torch.int16).cpu().numpy().view(np.uint16)
        else:
            out = np.zeros((t.shape[0], self.stride), dtype=np.float32)
            out[:, :self.n] = g.cpu().numpy()
        return out

    def refresh(self, st, keys):
        for k in keys:
            if st.get(k) is not None:
                self.h[k] = self.gather(st[k])

    def check(self, st, what):
        got = {k: self.gather(st.get(k)) for k in STATE_KEYS}
        assert_state_equal(got, self.h, what=what)


def test_config0_full(oracle):
    """M = 2, P = 2^20, fp32, 3 consecutive eager steps from the seed; every element compared."""
    w = inputs.WORKLOADS["cfg0"]
    st = inputs.make_outer_state(w.M, w.P, w.seed, device=DEV)
    h = host_copy(st)
    state = binding.State.from_dict(st, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum)
    for k in range(w.outer_steps):
        if k:
            inputs.inner_phase_standin(st)
            h["theta"] = to_numpy(st["theta"])
        state.outer_eager()
        oracle_outer(oracle, 2, h, w.M, w.P, st["stride"], w.outer_lr, w.outer_momentum, 0)
        torch.cuda.synchronize()
        assert_state_equal(st, h, what=f"cfg0 step {k + 1}")


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_config1_full(oracle, variant):
    """M = 4, P = 35 M, fp32, 10 outer steps of each variant from the same seed; every element
    compared after the first and the last step (state carries, so a miss in between shows)."""
    w = inputs.WORKLOADS["cfg1"]
    st = inputs.make_outer_state(w.M, w.P, w.seed, device=DEV)
    h = host_copy(st)
    state = binding.State.from_dict(st, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum)
    for k in range(w.outer_steps):
        if k:
            inputs.inner_phase_standin(st)
            h["theta"] = to_numpy(st["theta"])
        state.outer(variant)
        oracle_outer(oracle, variant, h, w.M, w.P, st["stride"], w.outer_lr, w.outer_momentum, 0, nthreads=16)
        if k in (0, w.outer_steps - 1):
            torch.cuda.synchronize()
            assert_state_equal(st, h, what=f"cfg1 variant {variant} step {k + 1}")


def run_phases(oracle, w, phases, H, seg_sizes=None):
    M, P = w.M, w.P
    st = inputs.make_outer_state(M, P, w.seed, device=DEV, theta_kind=w.theta_kind, with_adam=True)
    stride = st["stride"]
    extra = np.cumsum(seg_sizes)[:-1] if seg_sizes is not None else ()
    mirror = SliceMirror(st, slice_index(M, P, stride, w.seed, extra))
    gelt = 2 if w.grad_kind else 4
    grads = torch.zeros((M, stride), dtype=torch.bfloat16 if w.grad_kind else torch.float32, device=DEV)
    seg_scales = inputs.segment_scales(len(seg_sizes), st["gen"], DEV).tolist() if seg_sizes is not None else None
    state = binding.State.from_dict(st, H=H, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum, beta1=w.beta1,
                                    beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay, grad_kind=w.grad_kind)
    hp = dict(lr=w.inner_lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.weight_decay)
    k = 0
    for ph in range(phases):
        for _ in range(H):
            k += 1
            if seg_sizes is None:
                inputs.make_grads(M, P, stride, st["gen"], DEV, w.grad_kind, out=grads)
            else:
                inputs.make_segment_grads(M, seg_sizes, seg_scales, st["gen"], grads)
            state.inner_adamw(grads, w.inner_lr)
            g = mirror.gather(grads)
            oracle_adamw(oracle, mirror.h, g, M, mirror.n, mirror.stride, mirror.stride, k, hp, w.theta_kind,
                         w.grad_kind, nthreads=16)
        state.outer_eager()
        oracle_outer(oracle, 2, mirror.h, M, mirror.n, mirror.stride, w.outer_lr, w.outer_momentum, w.theta_kind,
                     nthreads=16)
        torch.cuda.synchronize()
        mirror.check(st, f"{w.name} phase {ph + 1}")
    assert state.get_counters() == (H * phases, phases, 1)
    return mirror.n / P


def test_config2_phases_on_slices(oracle):
    """bf16 replicas + fp32 outer state, M = 4, P = 550 M, H = 30 fused AdamW steps with fresh
    N(0, 1e-2) bf16 gradients per step, then one eager outer step; 5 phases."""
    w = inputs.WORKLOADS["cfg2"]
    need_gpu_bytes(w.M * w.P * (2 + 4 * 5 + 2) + 4 * w.P)
    frac = run_phases(oracle, w, w.outer_steps, w.H)
    assert frac > 0.005


def test_config3_phases_on_slices(oracle):
    """fp32 master + bf16 working copy, M = 4, P = 1.3 B, H = 100, gradients scaled per
    tensor-sized segment (256 segments, scales log-uniform over two decades); 3 phases."""
    w = inputs.WORKLOADS["cfg3"]
    need_gpu_bytes(w.M * w.P * (2 + 4 * 6 + 2) + 4 * w.P)
    seg = inputs.segment_sizes(w.P, w.segments)
    run_phases(oracle, w, w.outer_steps, w.H, seg_sizes=seg)


@pytest.mark.parametrize("name", ["cfg4a", "cfg4b", "cfg4c"])
def test_config4_memory_sweep_on_slices(oracle, name):
    """fp32 eager steps at (M, P) = (2, 2.4 B), (8, 550 M), (16, 150 M); 3 steps each."""
    w = inputs.WORKLOADS[name]
    need_gpu_bytes(w.M * w.P * 16 + 4 * w.P + 4 * w.P)
    st = inputs.make_outer_state(w.M, w.P, w.seed, device=DEV)
    mirror = SliceMirror(st, slice_index(w.M, w.P, st["stride"], w.seed))
    state = binding.State.from_dict(st, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum)
    for k in range(w.outer_steps):
        if k:
            inputs.inner_phase_standin(st)
            mirror.refresh(st, ("theta",))
        state.outer_eager()
        oracle_outer(oracle, 2, mirror.h, w.M, mirror.n, mirror.stride, w.outer_lr, w.outer_momentum, 0, nthreads=16)
        torch.cuda.synchronize()
        mirror.check(st, f"{name} step {k + 1}")
