"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bar: bit-exact for every fp32 buffer (both sides perform the same IEEE operations in the
same order; FMA contraction is off on both), identical bit patterns for bf16 storage
(tolerance 1 bf16 ulp allowed by the contract, 0 expected and asserted).  +0 and -0 compare
equal.  All inputs are seeded and synthetic; the oracle receives copies of the device
tensors, never a second draw.
"""
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2502_12996_b200 import binding, inputs
from gpu_util import (assert_state_equal, host_copy, oracle_adamw, oracle_outer, to_numpy, with_guards)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
HP = dict(lr=4e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1)
NAMES = {0: "standard", 1: "delayed", 2: "eager"}


def make(M, P, seed, theta_kind=0, with_adam=False, guards=True):
    st = inputs.make_outer_state(M, P, seed, device=DEV, theta_kind=theta_kind, with_adam=with_adam)
    # non-zero momentum and sentinel padding so that a wrong index or a write past P shows
    st["outer_mom"][:, :P].normal_(0.0, 1e-3, generator=st["gen"])
    for k in ("theta", "master", "start", "delta_prev_local", "outer_mom", "adam_m", "adam_v"):
        if st.get(k) is not None:
            st[k][:, P:] = 3.0
    st["delta_prev_avg"][P:] = 3.0
    checks = with_guards(st, DEV) if guards else []
    return st, checks


def run_outer_steps(oracle, variant, M, P, theta_kind, steps, seed, have_prev=1, eta=0.7, mu=0.9, impl=0):
    st, checks = make(M, P, seed, theta_kind)
    h = host_copy(st)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    state = binding.State.from_dict(st, outer_lr=eta, outer_momentum=mu, have_prev=have_prev, impl=impl,
                                    device_status=status)
    hp = have_prev
    for k in range(steps):
        if k > 0:
            inputs.inner_phase_standin(st)
            h["theta"] = to_numpy(st["theta"])
            h["master"] = to_numpy(st["master"])
        state.outer(variant)
        oracle_outer(oracle, variant, h, M, P, st["stride"], eta, mu, theta_kind,
                     bootstrap=(variant != 0 and hp == 0))
        if variant != 0:
            hp = 1
        torch.cuda.synchronize()
        assert_state_equal(st, h, what=f"{NAMES[variant]} M={M} P={P} kind={theta_kind} step {k + 1}")
    for c in checks:
        c()
    assert state.get_counters()[1] == steps
    state.check_device_status()
    assert int(status.item()) == 0
    state.close()


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("M,P", [(1, 70_001), (2, (1 << 20) + 3), (3, 100_003), (4, 300_007), (5, 50_001),
                                 (8, 200_005), (12, 40_003), (16, 150_001), (24, 9_001), (32, 30_001), (64, 5_003)])
def test_outer_fp32(oracle, variant, M, P):
    run_outer_steps(oracle, variant, M, P, 0, steps=3, seed=100 + M)


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("theta_kind", [1, 2])
@pytest.mark.parametrize("M,P", [(2, 100_001), (4, 250_003), (7, 20_001), (8, 60_002), (16, 40_003), (64, 7_003)])
def test_outer_bf16_storage(oracle, variant, theta_kind, M, P):
    run_outer_steps(oracle, variant, M, P, theta_kind, steps=3, seed=200 + M)


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("theta_kind", [0, 1, 2])
@pytest.mark.parametrize("M", [2, 4, 6, 16, 64])
def test_first_outer_step_then_regular(oracle, variant, theta_kind, M):
    """have_prev = 0: the first call records and applies nothing (t = H), later calls apply."""
    run_outer_steps(oracle, variant, M, 33_335, theta_kind, steps=3, seed=300 + M, have_prev=0)


@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 63, 64, 65, 255, 1025])
def test_tiny_and_ragged_sizes(oracle, P):
    for variant in (0, 1, 2):
        for M in (2, 4, 5):
            run_outer_steps(oracle, variant, M, P, 0, steps=2, seed=400 + P)
    run_outer_steps(oracle, 2, 4, P, 1, steps=2, seed=500 + P)
    run_outer_steps(oracle, 2, 16, P, 2, steps=2, seed=600 + P)


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("theta_kind", [0, 1, 2])
@pytest.mark.parametrize("M,P", [(2, 700_003), (4, 400_005), (4, 511), (2, 1024)])
def test_bulk_staged_implementation(oracle, variant, theta_kind, M, P):
    """The TMA-staged form (tiles through shared memory, bounded mbarrier waits) must give the
    same bits as the oracle, including the ragged tail and sizes below one tile."""
    run_outer_steps(oracle, variant, M, P, theta_kind, steps=3, seed=650 + M, impl=binding.IMPL_BULK)


@pytest.mark.parametrize("impl", [binding.IMPL_TENSOR_T256, binding.IMPL_TENSOR_T128, binding.IMPL_TENSOR_T64])
@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("M,P", [(1, 70_001), (2, 300_003), (4, 200_005), (5, 9_999), (8, 60_001), (16, 50_003), (4, 255),
                                 (3, 1)])
def test_tensor_map_implementation(oracle, impl, variant, M, P):
    """The 2-D TMA form (one box copy per buffer and tile, all M replicas at once; columns
    beyond P zero-filled on load and clipped on store by the hardware) must give the oracle's
    bits, ragged sizes and sizes below one tile included."""
    run_outer_steps(oracle, variant, M, P, 0, steps=3, seed=670 + M, impl=impl)


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("theta_kind", [0, 1, 2])
@pytest.mark.parametrize("P", [150_001, 63, 4_100])
def test_sixteen_replicas_forms(oracle, variant, theta_kind, P):
    """M = 16 through its default form (two chained warps per 16 columns, the running sum handed
    from warp to warp through shared memory and a named barrier) and through both forced
    warp-split forms: the same ordered sum, the oracle's bits."""
    for impl in (binding.IMPL_AUTO, binding.IMPL_SPLIT_R2, binding.IMPL_SPLIT_R4):
        run_outer_steps(oracle, variant, 16, P, theta_kind, steps=2, seed=690 + theta_kind, impl=impl)


def test_tensor_map_implementation_large_m_and_fragments(oracle):
    """M = 32 and 64 (narrow tiles only: three stages of wider ones do not fit shared memory and
    the call falls back to the direct form), and a fragment whose base is not at column 0."""
    run_outer_steps(oracle, 2, 32, 20_001, 0, steps=2, seed=680, impl=binding.IMPL_TENSOR_T128)
    run_outer_steps(oracle, 2, 64, 9_001, 0, steps=2, seed=681, impl=binding.IMPL_TENSOR_T64)
    run_outer_steps(oracle, 2, 64, 9_001, 0, steps=2, seed=682, impl=binding.IMPL_TENSOR_T256)   # falls back
    M, P = 4, 100_003
    a, _ = make(M, P, 683, 0)
    b = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in a.items()}
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sa = binding.State.from_dict(a)
    sb = binding.State.from_dict(b, impl=binding.IMPL_TENSOR_T128, device_status=status)
    sa.outer_eager()
    for lo, hi in ((64 * 700, P), (0, 64 * 700)):
        sb.outer_fragment(binding.EAGER, False, lo, hi - lo)
    sb.check_device_status()
    torch.cuda.synchronize()
    for k in ("theta", "start", "delta_prev_local", "delta_prev_avg", "outer_mom"):
        assert torch.equal(a[k].view(torch.int32), b[k].view(torch.int32)), k


@pytest.mark.parametrize("M,P,impl", [(2, 8 * 1024 + 5, binding.IMPL_BULK), (4, 40 * 512, binding.IMPL_BULK),
                                      (4, 20_001, binding.IMPL_TENSOR_T128), (16, 3_001, binding.IMPL_TENSOR_T64)])
def test_bounded_device_wait_runs_out_and_is_reported(oracle, M, P, impl):
    """The staged form's only device-side waits are on mbarriers that the copy engine completes.
    Here every barrier is told to expect 16 bytes more than its copies deliver: all copies land,
    no wait can complete, every wait gives up after the 2 ms limit, the CTAs drain and return.
    Nothing faults or hangs: the host reads the status word, gets DEVICE_TIMEOUT, finds the
    state untouched, and the next ordinary call on a cleared status word equals the oracle."""
    import time
    st, checks = make(M, P, 660 + M, 0)
    h = host_copy(st)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    state = binding.State.from_dict(st, impl=impl, device_status=status)
    state.set_wait_limit(2_000_000, 16)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    state.outer_eager()
    with pytest.raises(binding.DilocoError) as e:
        state.check_device_status()
    elapsed = time.perf_counter() - t0
    assert e.value.status == binding.ERR_DEVICE_TIMEOUT
    assert int(status.item()) == 0x7101
    assert 0.002 <= elapsed < 5.0, elapsed                     # at least one limit, at most a handful
    assert_state_equal(st, h, what="after the timed-out launch")        # no tile was stepped
    for bad in (8, 2048):
        with pytest.raises(binding.DilocoError):
            state.set_wait_limit(0, bad)
    # recovery: same context, same state
    status.zero_()
    state.set_wait_limit(0, 0)
    state.set_counters(0, 0, 1)
    state.outer_eager()
    oracle_outer(oracle, 2, h, M, P, st["stride"], 0.7, 0.9, 0)
    state.check_device_status()
    assert int(status.item()) == 0
    assert_state_equal(st, h, what="ordinary call after the time-out")
    for c in checks:
        c()
    state.close()


@pytest.mark.parametrize("theta_kind", [0, 1, 2])
@pytest.mark.parametrize("M,P", [(1, 9_001), (2, 300_003), (4, 200_005), (5, 70_001), (8, 50_002), (16, 20_003), (64, 3_001),
                                 (3, 2)])
def test_standard_step_with_one_shared_copy_of_the_outer_state(oracle, theta_kind, M, P):
    """Algorithm 1 with start and outer_mom stored once ([stride]) instead of once per replica:
    theta and the shared copy must equal EVERY replica's row of the per-replica oracle, bit for
    bit, over several steps; every other outer call refuses such a state."""
    st, checks = make(M, P, 720 + M, theta_kind)
    h = host_copy(st)                                          # per-replica oracle: all M rows start equal
    h["outer_mom"][:] = h["outer_mom"][0]
    shared = dict(st)
    shared["start"] = st["start"][0].clone()
    shared["outer_mom"] = st["outer_mom"][0].clone()
    state = binding.State.from_dict(shared, shared_outer_state=True)
    for k in range(3):
        if k:
            inputs.inner_phase_standin(st)                     # theta_m <- start_m + noise; the rows of start are stale here,
            for key in ("theta", "master"):                    # so rebuild theta from the shared copy instead
                if st.get(key) is not None:
                    noise = st[key][:, :P].float() - st["start"][:, :P]
                    st[key][:, :P] = (shared["start"][:P] + noise).to(st[key].dtype)
            h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
        state.outer_standard()
        oracle_outer(oracle, 0, h, M, P, st["stride"], 0.7, 0.9, theta_kind)
        torch.cuda.synchronize()
        got = dict(theta=st["theta"], master=st["master"])
        assert_state_equal(got, h, keys=("theta", "master"), what=f"shared standard M={M} kind={theta_kind} step {k + 1}")
        for m in range(M):
            for key in ("start", "outer_mom"):
                one = {key: shared[key][:P]}
                assert_state_equal(one, {key: h[key][m, :P]}, keys=(key,), what=f"shared {key} vs replica {m}")
    assert float(shared["start"][P:].min()) == 3.0 and float(shared["outer_mom"][P:].max()) == 3.0   # padding untouched
    for c in checks:
        c()
    for call in (state.outer_eager, state.outer_delayed, lambda: state.outer_quantized(0, binding.COMM_BF16)):
        with pytest.raises(binding.DilocoError) as e:
            call()
        assert e.value.status == binding.ERR_BAD_STATE
    state.fragments_set([0], [min(P, 64)])
    state.outer_fragment_step(binding.STANDARD, 0)
    torch.cuda.synchronize()
    state.close()


@pytest.mark.parametrize("eta,mu", [(0.4, 0.9), (1.0, 0.0), (0.7, 0.0)])
def test_other_outer_hyperparameters(oracle, eta, mu):
    run_outer_steps(oracle, 2, 4, 65_537, 0, steps=3, seed=700, eta=eta, mu=mu)
    run_outer_steps(oracle, 0, 2, 65_537, 0, steps=2, seed=701, eta=eta, mu=mu)


def test_worked_example_on_gpu():
    """The hand-computed dyadic example (tests/golden): exact whatever the operation order."""
    from test_oracle_outer import GOLDEN, VARIANTS, read_golden
    g = read_golden(GOLDEN)
    M, P, stride = 2, 2, 64
    for name, variant in VARIANTS.items():
        def dev(key, rows=M):
            t = torch.zeros((rows, stride), dtype=torch.float32, device=DEV)
            t[:, :P] = torch.tensor(g[key], dtype=torch.float32).view(rows, P)
            return t
        st = dict(theta=dev("theta"), start=dev("start"), delta_prev_local=dev("delta_prev_local"),
                  delta_prev_avg=dev("delta_prev_avg", 1).view(-1), outer_mom=torch.zeros((M, stride), device=DEV))
        state = binding.State(M=M, P=P, stride=stride, outer_lr=g["eta"][0], outer_momentum=g["mu"][0], **st)
        for k in (1, 2):
            if k == 2:
                st["theta"][:, :P] += torch.tensor(g["inner_phase_2"], device=DEV).view(M, P)
            state.outer(variant)
            torch.cuda.synchronize()
            want = torch.tensor(g[f"{name}_theta_{k}"]).view(M, P)
            assert torch.equal(st["theta"][:, :P].cpu(), want), (name, k)
            assert torch.equal(st["start"][:, :P].cpu(), want)
            assert torch.equal(st["outer_mom"][:, :P].cpu(), torch.tensor(g[f"{name}_mom_{k}"]).view(M, P))
        state.close()


# ---------------------------------------------------------------- quantised communication
FORMATS = {"bf16": (binding.COMM_BF16, 0, 0), "e4m3": (binding.COMM_EXMY, 4, 3), "e5m2": (binding.COMM_EXMY, 5, 2),
           "e2m1": (binding.COMM_EXMY, 2, 1), "e3m0": (binding.COMM_EXMY, 3, 0)}


@pytest.mark.parametrize("fmt", list(FORMATS))
@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("M,P,theta_kind", [(2, 100_003, 0), (4, 300_001, 0), (4, 70_001, 1), (8, 50_002, 2),
                                            (16, 40_001, 0), (32, 10_001, 1), (64, 9_001, 2), (5, 20_003, 0), (1, 9_999, 0)])
def test_quantized_communication(oracle, fmt, variant, M, P, theta_kind):
    """The all-reduce operand rounded to bf16 / scaled EXMY: per-replica maxima reduced on the
    device, same scale, same rounding (ties included), same bits as the oracle; first call is
    the t = H bootstrap, then two regular steps."""
    comm, X, Y = FORMATS[fmt]
    st, checks = make(M, P, 1700 + M, theta_kind)
    h = host_copy(st)
    scratch = torch.full((64,), 0x7fffffff, dtype=torch.int32, device=DEV)     # stale contents must not matter
    state = binding.State.from_dict(st, have_prev=0, comm_scratch=scratch)
    for k in range(3):
        if k:
            inputs.inner_phase_standin(st)
            h["theta"] = to_numpy(st["theta"])
            h["master"] = to_numpy(st["master"])
        state.outer_quantized(variant, comm, X, Y)
        oracle.outer_step(variant, M=M, P=P, stride=st["stride"], eta=0.7, mu=0.9, theta=h["theta"], start=h["start"],
                          outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                          delta_prev_avg=h["delta_prev_avg"], master=h["master"], theta_kind=theta_kind,
                          bootstrap=(variant != 0 and k == 0), comm=comm, exp_bits=X, man_bits=Y, nthreads=8)
        torch.cuda.synchronize()
        assert_state_equal(st, h, what=f"quantised {fmt} {NAMES[variant]} M={M} step {k + 1}")
    for c in checks:
        c()
    assert state.get_counters()[1] == 3


def test_quantized_argument_checks():
    st, _ = make(2, 1000, 1800, 0, guards=False)
    state = binding.State.from_dict(st)                        # no comm_scratch
    with pytest.raises(binding.DilocoError) as e:
        state.outer_quantized(2, binding.COMM_EXMY, 4, 3)
    assert e.value.status == binding.ERR_BAD_STATE
    state.outer_quantized(2, binding.COMM_BF16)                 # bf16 needs no scratch
    for X, Y in ((0, 3), (6, 1), (4, 4), (3, -1)):
        with pytest.raises(binding.DilocoError) as e:
            state.outer_quantized(2, binding.COMM_EXMY, X, Y)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DilocoError):
        state.outer_quantized(2, 7)
    torch.cuda.synchronize()


# ---------------------------------------------------------------- D-outer-steps overlap
@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("D,M,P,theta_kind,have", [(2, 4, 150_003, 0, 0), (2, 2, 80_001, 1, 2), (3, 8, 40_002, 0, 1),
                                                   (4, 16, 20_001, 2, 0), (2, 5, 30_001, 0, 0)])
def test_overlap_by_D_outer_steps(oracle, variant, D, M, P, theta_kind, have):
    """All-reduce results consumed D outer steps late (D = 2 is the "two-outer-steps" overlap):
    D generations of recorded gradients in a ring; runs start with `have` generations seeded."""
    st = inputs.make_outer_state(M, P, 1900 + D + M, device=DEV, theta_kind=theta_kind, overlap_steps=D)
    h = host_copy(st)
    state = binding.State.from_dict(st, have_prev=have, overlap_steps=D)
    steps = 2 * D + 2
    for k in range(steps):
        if k:
            inputs.inner_phase_standin(st)
            h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
        state.outer(variant)
        have = oracle.outer_step_overlap(variant, k, have, M=M, P=P, stride=st["stride"], eta=0.7, mu=0.9,
                                         theta=h["theta"], master=h["master"], start=h["start"],
                                         outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                                         delta_prev_avg=h["delta_prev_avg"], theta_kind=theta_kind, nthreads=8)
        torch.cuda.synchronize()
        assert_state_equal(st, h, what=f"overlap D={D} {NAMES[variant]} step {k + 1}")
        assert state.get_counters() == (0, k + 1, have)


def test_overlap_with_quantised_wire_and_host_buffers(oracle):
    """The generation ring is honoured by the quantised call and by the host-buffer call."""
    D, M, P = 2, 4, 100_003
    st = inputs.make_outer_state(M, P, 1950, device=DEV, overlap_steps=D)
    h = host_copy(st)
    keys = ("theta", "start", "delta_prev_local", "delta_prev_avg", "outer_mom")
    pinned = {k: st[k].cpu().pin_memory() for k in keys}
    scratch = torch.zeros(64, dtype=torch.int32, device=DEV)
    state = binding.State.from_dict(st, overlap_steps=D, comm_scratch=scratch)
    streams = [torch.cuda.Stream(device=DEV) for _ in range(3)]
    have = D
    for k in range(5):
        if k % 2 == 0:
            state.outer_quantized(binding.EAGER, binding.COMM_EXMY, 4, 3)
            torch.cuda.synchronize()
            for key in keys:
                pinned[key].copy_(st[key])
            kw = dict(comm=oracle.COMM_EXMY, exp_bits=4, man_bits=3)
        else:
            state.outer_step_host(binding.EAGER, binding.make_buffers(**pinned), streams, 64 * 500)
            streams[2].synchronize()
            kw = {}
        have = oracle.outer_step_overlap(2, k, have, M=M, P=P, stride=st["stride"], eta=0.7, mu=0.9, theta=h["theta"],
                                         start=h["start"], outer_mom=h["outer_mom"],
                                         delta_prev_local=h["delta_prev_local"], delta_prev_avg=h["delta_prev_avg"], **kw)
        assert_state_equal(pinned, h, keys=keys, what=f"overlap mixed step {k + 1}")
        # next phase: both sides move the replicas the same way
        inputs.inner_phase_standin(st)
        h["theta"] = to_numpy(st["theta"])
        pinned["theta"].copy_(st["theta"])


# ---------------------------------------------------------------- inner AdamW
def run_adamw(oracle, M, P, theta_kind, grad_kind, steps, seed, segments=0):
    st, checks = make(M, P, seed, theta_kind, with_adam=True)
    stride = st["stride"]
    h = host_copy(st)
    state = binding.State.from_dict(st, grad_kind=grad_kind, beta1=HP["beta1"], beta2=HP["beta2"], eps=HP["eps"],
                                    weight_decay=HP["wd"])
    seg_sizes = seg_scales = None
    if segments:
        seg_sizes = inputs.segment_sizes(P, segments, d_model=16)
        seg_scales = inputs.segment_scales(segments, st["gen"], DEV)
    for k in range(1, steps + 1):
        g = inputs.make_grads(M, P, stride, st["gen"], DEV, grad_kind, seg_sizes=seg_sizes, seg_scales=seg_scales)
        state.inner_adamw(g, HP["lr"])
        oracle_adamw(oracle, h, to_numpy(g), M, P, stride, stride, k, HP, theta_kind, grad_kind)
        torch.cuda.synchronize()
        assert_state_equal(st, h, what=f"adamw M={M} P={P} kind={theta_kind}/{grad_kind} step {k}")
    for c in checks:
        c()
    assert state.get_counters()[0] == steps
    state.close()
    return st, h


@pytest.mark.parametrize("theta_kind,grad_kind", [(0, 0), (0, 1), (1, 0), (1, 1), (2, 0), (2, 1)])
@pytest.mark.parametrize("M,P", [(1, 10_001), (2, 1_000_003), (4, 300_005), (5, 777)])
def test_adamw(oracle, theta_kind, grad_kind, M, P):
    run_adamw(oracle, M, P, theta_kind, grad_kind, steps=4, seed=800 + M)


def test_adamw_segment_scaled_gradients(oracle):
    """Gradients with per-segment scales spread over two decades (the fourth configuration's law)."""
    run_adamw(oracle, 4, 200_003, 2, 1, steps=3, seed=900, segments=256)


@pytest.mark.parametrize("P", [1, 3, 4, 7, 64, 2049])
def test_adamw_tiny(oracle, P):
    run_adamw(oracle, 3, P, 0, 0, steps=2, seed=950 + P)
    run_adamw(oracle, 2, P, 1, 1, steps=2, seed=960 + P)


# ---------------------------------------------------------------- whole simulated phases
@pytest.mark.parametrize("theta_kind,grad_kind", [(0, 0), (1, 1), (2, 1)])
def test_full_phases(oracle, theta_kind, grad_kind):
    """H inner AdamW steps on every replica, then one eager outer step; 3 phases, the first
    outer step being the t = H bootstrap."""
    M, P, H, phases = 4, 120_007, 5, 3
    st, checks = make(M, P, 1000 + theta_kind, theta_kind, with_adam=True)
    st["outer_mom"].zero_()
    stride = st["stride"]
    h = host_copy(st)
    state = binding.State.from_dict(st, H=H, grad_kind=grad_kind, have_prev=0, beta1=HP["beta1"], beta2=HP["beta2"],
                                    eps=HP["eps"], weight_decay=HP["wd"])
    k = 0
    for ph in range(phases):
        for _ in range(H):
            k += 1
            g = inputs.make_grads(M, P, stride, st["gen"], DEV, grad_kind)
            state.inner_adamw(g, HP["lr"])
            oracle_adamw(oracle, h, to_numpy(g), M, P, stride, stride, k, HP, theta_kind, grad_kind)
        state.outer_eager()
        oracle_outer(oracle, 2, h, M, P, stride, 0.7, 0.9, theta_kind, bootstrap=(ph == 0))
        torch.cuda.synchronize()
        assert_state_equal(st, h, what=f"phase {ph + 1} kind={theta_kind}")
    assert state.get_counters() == (H * phases, phases, 1)
    for c in checks:
        c()


# ---------------------------------------------------------------- fragments, resume, host path
@pytest.mark.parametrize("theta_kind", [0, 1])
def test_fragments_equal_whole(oracle, theta_kind):
    """Every index is independent: the step applied fragment by fragment (as a streaming
    schedule would) gives the same bits as one call over the whole vector."""
    M, P = 4, 200_003
    a, _ = make(M, P, 1100, theta_kind)
    b = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in a.items()}
    sa = binding.State.from_dict(a)
    sb = binding.State.from_dict(b)
    sa.outer_eager()
    cuts = [0, 64 * 100, 64 * 1000, 64 * 1001, 64 * 3000, P]
    for lo, hi in reversed(list(zip(cuts[:-1], cuts[1:]))):
        sb.outer_fragment(binding.EAGER, False, lo, hi - lo)
    torch.cuda.synchronize()
    for k in ("theta", "start", "delta_prev_local", "delta_prev_avg", "outer_mom"):
        assert torch.equal(a[k].view(torch.int16 if a[k].dtype == torch.bfloat16 else torch.int32),
                           b[k].view(torch.int16 if b[k].dtype == torch.bfloat16 else torch.int32)), k
    with pytest.raises(binding.DilocoError) as e:
        sb.outer_fragment(binding.EAGER, False, 32 if theta_kind else 16, 100)
    assert e.value.status == binding.ERR_MISALIGNED
    with pytest.raises(binding.DilocoError) as e:
        sb.outer_fragment(binding.EAGER, False, 64, P)
    assert e.value.status == binding.ERR_INVALID_ARG


@pytest.mark.parametrize("D", [1, 2])
@pytest.mark.parametrize("variant,theta_kind,impl", [(2, 0, 0), (2, 1, 0), (1, 2, 0), (0, 0, 0), (2, 0, 2)])
def test_fragment_table_staggered_schedule(oracle, D, variant, theta_kind, impl):
    """Streaming schedule: three fragments, fragment f takes its outer step at global steps
    t = f mod 3, each with its own outer-step count (ring slot) and its own have_prev (its first
    D eager / delayed steps only record).  The library keeps that state per fragment; the oracle
    side runs the fragment helper with its own bookkeeping.  Bit-exact after every step."""
    M, P = 4, 40_005
    st = inputs.make_outer_state(M, P, 1150 + D, device=DEV, theta_kind=theta_kind, overlap_steps=D)
    st["outer_mom"][:, :P].normal_(0.0, 1e-3, generator=st["gen"])
    stride = st["stride"]
    h = host_copy(st)
    h["delta_prev_local"] = h["delta_prev_local"].reshape(D, M, stride)
    h["delta_prev_avg"] = h["delta_prev_avg"].reshape(D, stride)
    cuts = [(0, 64 * 200), (64 * 200, 64 * 300 + 1024), (64 * 500 + 1024, P - (64 * 500 + 1024))]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    state = binding.State.from_dict(st, have_prev=0, overlap_steps=D, impl=impl, device_status=status)
    state.fragments_set([c[0] for c in cuts], [c[1] for c in cuts])
    have, count = [0, 0, 0], [0, 0, 0]
    for t in range(3 * (D + 2)):
        if t:
            inputs.inner_phase_standin(st)
            h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
        f = t % 3
        state.outer_fragment_step(variant, f)
        have[f] = oracle.outer_step_fragment(variant, count[f], have[f], cuts[f][0], cuts[f][1], M=M, eta=0.7, mu=0.9,
                                             theta=h["theta"], master=h["master"], start=h["start"],
                                             outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                                             delta_prev_avg=h["delta_prev_avg"], theta_kind=theta_kind)
        count[f] += 1
        torch.cuda.synchronize()
        got = {key: st[key] for key in ("theta", "master", "start", "outer_mom")}
        got["delta_prev_local"] = st["delta_prev_local"].view(D, M, stride)
        got["delta_prev_avg"] = st["delta_prev_avg"].view(D, stride)
        assert_state_equal(got, h, keys=tuple(got), what=f"fragment schedule D={D} t={t} fragment {f}")
        assert state.fragment_get_counters(f) == (count[f], have[f])
    assert state.get_counters() == (0, 0, 0)                   # the whole-vector counters are not involved
    state.check_device_status()
    # resume: a fresh state with the fragments' counters restored continues identically
    saved = [state.fragment_get_counters(f) for f in range(3)]
    state.close()
    state = binding.State.from_dict(st, have_prev=0, overlap_steps=D)
    state.fragments_set([c[0] for c in cuts], [c[1] for c in cuts])
    for f, (n, hv) in enumerate(saved):
        state.fragment_set_counters(f, n, hv)
    inputs.inner_phase_standin(st)
    h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
    state.outer_fragment_step(variant, 1)
    oracle.outer_step_fragment(variant, count[1], have[1], cuts[1][0], cuts[1][1], M=M, eta=0.7, mu=0.9,
                               theta=h["theta"], master=h["master"], start=h["start"], outer_mom=h["outer_mom"],
                               delta_prev_local=h["delta_prev_local"], delta_prev_avg=h["delta_prev_avg"],
                               theta_kind=theta_kind)
    torch.cuda.synchronize()
    got = {key: st[key] for key in ("theta", "master", "start", "outer_mom")}
    got["delta_prev_local"] = st["delta_prev_local"].view(D, M, stride)
    got["delta_prev_avg"] = st["delta_prev_avg"].view(D, stride)
    assert_state_equal(got, h, keys=tuple(got), what="fragment schedule after resume")
    state.close()


@pytest.mark.parametrize("fmt", ["e2m1", "e4m3", "bf16"])
@pytest.mark.parametrize("D,theta_kind", [(1, 0), (2, 1)])
def test_fragment_schedule_with_quantised_wire(oracle, fmt, D, theta_kind):
    """Streaming fragments with a 4- or 8-bit wire, the combination behind the paper's bandwidth
    table: each fragment's exchange is rounded with a scale of its own (the maximum over the
    fragment's indices), on its own schedule."""
    comm, X, Y = FORMATS[fmt]
    M, P = 4, 30_005
    st = inputs.make_outer_state(M, P, 1170 + D, device=DEV, theta_kind=theta_kind, overlap_steps=D)
    stride = st["stride"]
    h = host_copy(st)
    h["delta_prev_local"] = h["delta_prev_local"].reshape(D, M, stride)
    h["delta_prev_avg"] = h["delta_prev_avg"].reshape(D, stride)
    cuts = [(0, 64 * 150), (64 * 150, 64 * 200), (64 * 350, P - 64 * 350)]
    scratch = torch.zeros(64, dtype=torch.int32, device=DEV)
    state = binding.State.from_dict(st, have_prev=0, overlap_steps=D, comm_scratch=scratch)
    state.fragments_set([c[0] for c in cuts], [c[1] for c in cuts])
    have, count = [0, 0, 0], [0, 0, 0]
    for t in range(3 * (D + 1) + 1):
        if t:
            inputs.inner_phase_standin(st)
            h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
        f = t % 3
        state.outer_fragment_step_quantized(binding.EAGER, f, comm, X, Y)
        have[f] = oracle.outer_step_fragment(2, count[f], have[f], cuts[f][0], cuts[f][1], M=M, eta=0.7, mu=0.9,
                                             theta=h["theta"], master=h["master"], start=h["start"],
                                             outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                                             delta_prev_avg=h["delta_prev_avg"], theta_kind=theta_kind, comm=comm,
                                             exp_bits=X, man_bits=Y)
        count[f] += 1
        torch.cuda.synchronize()
        got = {key: st[key] for key in ("theta", "master", "start", "outer_mom")}
        got["delta_prev_local"] = st["delta_prev_local"].view(D, M, stride)
        got["delta_prev_avg"] = st["delta_prev_avg"].view(D, stride)
        assert_state_equal(got, h, keys=tuple(got), what=f"quantised fragment schedule {fmt} D={D} t={t}")
        assert state.fragment_get_counters(f) == (count[f], have[f])
    no_scratch = binding.State.from_dict(st, overlap_steps=D)
    no_scratch.fragments_set([0], [64])
    with pytest.raises(binding.DilocoError) as e:
        no_scratch.outer_fragment_step_quantized(binding.EAGER, 0, binding.COMM_EXMY, 4, 3)
    assert e.value.status == binding.ERR_BAD_STATE
    state.close()


def test_fragment_table_argument_checks():
    st, _ = make(2, 10_000, 1160, 0, guards=False)
    state = binding.State.from_dict(st)
    for offs, lens, status in (([0, 64], [100, 10], binding.ERR_INVALID_ARG),       # overlap
                               ([16], [10], binding.ERR_MISALIGNED),
                               ([0], [0], binding.ERR_INVALID_ARG),
                               ([9984], [100], binding.ERR_INVALID_ARG)):             # past P
        with pytest.raises(binding.DilocoError) as e:
            state.fragments_set(offs, lens)
        assert e.value.status == status
    with pytest.raises(binding.DilocoError) as e:
        state.outer_fragment_step(binding.EAGER, 0)               # no table installed
    assert e.value.status == binding.ERR_INVALID_ARG
    state.fragments_set([0, 5024], [5000, 4976])
    with pytest.raises(binding.DilocoError):
        state.outer_fragment_step(binding.EAGER, 2)
    with pytest.raises(binding.DilocoError):
        state.fragment_set_counters(0, 0, 2)                       # have_prev > overlap_steps
    state.outer_fragment_step(binding.EAGER, 1)
    assert state.fragment_get_counters(1) == (1, 1) and state.fragment_get_counters(0) == (0, 1)
    state.fragments_set([], [])
    with pytest.raises(binding.DilocoError):
        state.outer_fragment_step(binding.EAGER, 0)
    torch.cuda.synchronize()
    state.close()


def test_resume_from_counters(oracle):
    """3 steps in one state == 1 step, state dropped, new state with restored counters, 2 steps."""
    M, P = 2, 50_001
    a, _ = make(M, P, 1200, 0, with_adam=True)
    b = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in a.items()}
    gs = [inputs.make_grads(M, P, a["stride"], a["gen"], DEV, 0) for _ in range(3)]
    sa = binding.State.from_dict(a, have_prev=0)
    for g in gs:
        sa.inner_adamw(g, 1e-3)
        sa.outer_eager()
    sb = binding.State.from_dict(b, have_prev=0)
    sb.inner_adamw(gs[0], 1e-3)
    sb.outer_eager()
    counters = sb.get_counters()
    sb.close()
    sc = binding.State.from_dict(b, have_prev=0)
    sc.set_counters(*counters)
    for g in gs[1:]:
        sc.inner_adamw(g, 1e-3)
        sc.outer_eager()
    torch.cuda.synchronize()
    for k in ("theta", "start", "delta_prev_local", "delta_prev_avg", "outer_mom", "adam_m", "adam_v"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("theta_kind", [0, 2])
def test_host_buffer_entry_point(oracle, variant, theta_kind):
    """State in pinned host memory, chunked copy-in / step / copy-out: same bits as the oracle."""
    M, P = 4, 300_001
    st, _ = make(M, P, 1300 + variant, theta_kind, guards=False)
    h = host_copy(st)
    pinned = {k: (st[k].cpu().pin_memory() if st.get(k) is not None else None)
              for k in ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom")}
    for k in ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom"):
        if st.get(k) is not None:
            st[k].fill_(-7.0)                                     # the device copy must come from the host
    state = binding.State.from_dict(st)
    streams = [torch.cuda.Stream(device=DEV) for _ in range(3)]
    host = binding.make_buffers(**pinned)
    for step in range(2):
        state.outer_step_host(variant, host, streams, 64 * 1000)
        streams[2].synchronize()
        oracle_outer(oracle, variant, h, M, P, st["stride"], 0.7, 0.9, theta_kind)
        assert_state_equal(pinned, h, keys=tuple(pinned), what=f"host path {NAMES[variant]} step {step + 1}")
    state.close()


def test_host_pointers_are_rejected_not_dereferenced():
    """A host tensor where a device buffer belongs: INVALID_ARG at init (or at the call, for
    per-call buffers), never a kernel fault."""
    st, _ = make(2, 1000, 1450, 0, with_adam=True, guards=False)
    bad = dict(st)
    bad["start"] = st["start"].cpu()
    with pytest.raises(binding.DilocoError) as e:
        binding.State.from_dict(bad)
    assert e.value.status == binding.ERR_INVALID_ARG
    bad["start"] = st["start"].cpu().pin_memory()
    with pytest.raises(binding.DilocoError) as e:
        binding.State.from_dict(bad)
    assert e.value.status == binding.ERR_INVALID_ARG
    state = binding.State.from_dict(st)
    with pytest.raises(binding.DilocoError) as e:
        state.inner_adamw(torch.zeros((2, st["stride"])), 1e-3)            # host gradients
    assert e.value.status == binding.ERR_INVALID_ARG
    assert state.get_counters()[0] == 0
    torch.cuda.synchronize()


def test_host_entry_with_resident_optimizer_state(oracle):
    """NULL host pointers keep those buffers on the device: only theta crosses the bus."""
    M, P = 4, 200_003
    st, _ = make(M, P, 1350, 0, guards=False)
    h = host_copy(st)
    theta_host = st["theta"].cpu().pin_memory()
    st["theta"][:, :P] = -7.0                                    # the device copy must come from the host
    state = binding.State.from_dict(st)
    streams = [torch.cuda.Stream(device=DEV) for _ in range(3)]
    state.outer_step_host(binding.EAGER, binding.make_buffers(theta=theta_host), streams, 64 * 700)
    streams[2].synchronize()
    oracle_outer(oracle, 2, h, M, P, st["stride"], 0.7, 0.9, 0)
    assert_state_equal(dict(st, theta=theta_host), h, what="host path, theta only")
    assert_state_equal(st, h, what="host path, device copy")
    with pytest.raises(binding.DilocoError):
        state.outer_step_host(binding.EAGER, binding.make_buffers(start=theta_host), streams, 64)
    with pytest.raises(binding.DilocoError) as e:                # device memory where host memory belongs
        state.outer_step_host(binding.EAGER, binding.make_buffers(theta=st["theta"].clone()), streams, 64 * 700)
    assert e.value.status == binding.ERR_INVALID_ARG
    assert state.get_counters()[1] == 1


def test_host_entry_rows_longer_than_the_2d_copy_pitch_limit(oracle):
    """Rows of 2^29 fp32 elements (2 GiB, the row length of the 550 M-parameter shapes and up)
    exceed the pitch the 2-D copy routines accept; the host entry copies row by row.  Only P
    elements per row are touched, so the buffers are allocated but never filled."""
    M, P, stride = 2, 70_001, 1 << 29
    if torch.cuda.mem_get_info()[0] < 24 << 30:
        pytest.skip("needs 18 GiB of device memory")
    small = inputs.make_outer_state(M, P, 1360, device=DEV)
    st = dict(M=M, P=P, stride=stride, theta_kind=0, master=None, adam_m=None, adam_v=None)
    for k in ("theta", "start", "delta_prev_local", "outer_mom"):
        st[k] = torch.empty((M, stride), dtype=torch.float32, device=DEV)
        st[k][:, :P] = small[k][:, :P]
    st["delta_prev_avg"] = torch.empty(stride, dtype=torch.float32, device=DEV)
    st["delta_prev_avg"][:P] = small["delta_prev_avg"][:P]
    h = {k: (None if st.get(k) is None else st[k][..., :P].cpu().numpy().copy()) for k in
         ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom")}
    theta_host = torch.empty((M, stride), dtype=torch.float32)   # pageable, only P elements per row ever touched
    theta_host[:, :P] = st["theta"][:, :P].cpu()
    st["theta"][:, :P] = -7.0
    state = binding.State.from_dict(st)
    streams = [torch.cuda.Stream(device=DEV) for _ in range(3)]
    state.outer_step_host(binding.EAGER, binding.make_buffers(theta=theta_host), streams, 64 * 300)
    for s_ in streams:
        s_.synchronize()
    oracle.outer_step(oracle.EAGER, M=M, P=P, stride=P, eta=0.7, mu=0.9, theta=h["theta"], start=h["start"],
                      outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"], delta_prev_avg=h["delta_prev_avg"])
    got = {k: st[k][..., :P].contiguous() for k in ("start", "delta_prev_local", "delta_prev_avg", "outer_mom")}
    got["theta"] = theta_host[:, :P].contiguous()
    assert_state_equal(got, h, keys=tuple(got), what="host path, 2 GiB rows")
    state.close()


def test_launch_counter():
    M, P = 2, 1000
    st, _ = make(M, P, 1400, 0, with_adam=True)
    state = binding.State.from_dict(st)
    n0 = binding.launch_count()
    state.outer_eager()
    state.outer_standard()
    state.inner_adamw(torch.zeros((M, st["stride"]), device=DEV), 1e-3)
    assert binding.launch_count() == n0 + 3
    torch.cuda.synchronize()


def test_outer_step_in_a_cuda_graph(oracle):
    """The steady-state outer step with overlap_steps = 1 launches one kernel whose arguments do
    not change from step to step, so it can be captured once and replayed (small fragments are
    launch-bound).  The host-side counters advance at capture time only; the replays must still
    equal the oracle step for step."""
    M, P = 4, 50_001
    st, _ = make(M, P, 1550, 0, guards=False)
    h = host_copy(st)
    state = binding.State.from_dict(st)
    stream = torch.cuda.Stream(device=DEV)
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        state.outer_eager(stream=stream)                       # warm-up launch outside the capture (also a real step)
        oracle_outer(oracle, 2, h, M, P, st["stride"], 0.7, 0.9, 0)
        stream.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            state.outer_eager(stream=stream)
    for k in range(3):
        inputs.inner_phase_standin(st)
        h["theta"] = to_numpy(st["theta"])
        graph.replay()
        torch.cuda.synchronize()
        oracle_outer(oracle, 2, h, M, P, st["stride"], 0.7, 0.9, 0)
        assert_state_equal(st, h, what=f"graph replay {k + 1}")
    assert state.get_counters()[1] == 2                        # the warm-up and the captured call; replays count nothing
    state.close()


def test_non_default_stream(oracle):
    M, P = 4, 100_001
    st, _ = make(M, P, 1500, 0)
    h = host_copy(st)
    state = binding.State.from_dict(st)
    s = torch.cuda.Stream(device=DEV)
    s.wait_stream(torch.cuda.current_stream())
    state.outer_eager(stream=s)
    s.synchronize()
    oracle_outer(oracle, 2, h, M, P, st["stride"], 0.7, 0.9, 0)
    assert_state_equal(st, h)


# ---------------------------------------------------------------- bench.py, two ranks
def test_bench_two_ranks_dry_run(tmp_path):
    """bench.py under torchrun with two ranks (gloo for the barrier and the reductions, both
    ranks on this one GPU: the ranks never wait on one another's kernels): one JSON line from
    rank 0, whole-job value = sum over ranks, launches counted on both."""
    import json, os, socket, subprocess, sys
    from pathlib import Path
    root = Path(__file__).resolve().parent.parent
    env = dict(os.environ, DILOCO_BENCH_BACKEND="gloo")
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(root / "bench.py"), "--gpus", "2", "--steps", "3", "--warmup", "3",
           "--workload", "cfg1", "--P", "2000000", "--no-cpu-baseline"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=str(root))
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["gpu_launches"] == 6 and d["scaling"] == "weak"
    assert abs(d["value"] - 2 * 2_000_000 / (d["ms_per_step"] * 1e-3)) < 1e-3 * d["value"]
    assert d["e2e"]["value"] > 0 and d["roofline"]["frac"] > 0


def test_bench_line_has_every_contract_key():
    """One rank, small P: the JSON line carries the keys the measurement contract names."""
    import json, subprocess, sys
    from pathlib import Path
    root = Path(__file__).resolve().parent.parent
    out = subprocess.run([sys.executable, str(root / "bench.py"), "--steps", "3", "--warmup", "3", "--P", "3000000"],
                         capture_output=True, text=True, timeout=900, cwd=str(root))
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert k in d, k
    assert d["config"]["workload"] == "cfg4a" and d["config"]["M"] == 2            # the default: largest outer-only shape
    assert d["vs_baseline"] is None and d["data"] == "synthetic" and d["shapes"] is None   # --P: one shape only
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["gpu_launches"] == 3 and d["higher_is_better"] is True
    for k in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert k in d["roofline"], k
    assert d["roofline"]["bound"] == "hbm" and abs(d["roofline"]["frac"] - d["roofline"]["achieved"] / d["roofline"]["peak"]) < 1e-9
    for k in ("value", "unit", "cores", "kind", "sample"):
        assert k in d["cpu_baseline"], k
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    for k in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert k in d["e2e"], k
    assert d["e2e"]["h2d_bytes_per_step"] == 3000000 * (4 * 8 + 4) and d["e2e"]["value"] < d["value"]
    assert d["e2e"]["workload"] == "cfg4a"
    for k in ("sm_mhz", "sm_max_mhz", "reasons"):
        assert k in d["clocks"], k


# ---------------------------------------------------------------- seeded random sweep
@pytest.mark.parametrize("case", range(48))
def test_random_configurations(oracle, case):
    """Seeded random (M, P, variant, storage, overlap, wire format, seeded generations): every
    replica count from 1 to 64 lands on one of the kernel forms (per-thread, lane split, warp
    chain, warp split with one or two column groups per block, first-steps form), and every
    combination must equal the oracle bit for bit over several outer steps."""
    rng = np.random.default_rng(31_000 + case)
    M = int(rng.choice([int(rng.integers(1, 65)), int(rng.choice([12, 20, 24, 28, 36, 40, 44, 48, 52, 56, 60, 64])),
                        int(rng.choice([5, 6, 7, 9, 11, 13, 17, 31, 33, 63]))]))
    P = int(rng.choice([int(rng.integers(1, 300)), int(rng.integers(300, 60_000))]))
    variant = int(rng.integers(0, 3))
    theta_kind = int(rng.integers(0, 3))
    D = int(rng.integers(1, 4))
    have = int(rng.integers(0, D + 1))
    wire = [(0, 0, 0), (1, 0, 0), (2, 4, 3), (2, 5, 2), (2, 2, 1), (2, 3, 0), (2, 3, 2)][int(rng.integers(0, 7))]
    eta, mu = float(rng.choice([0.4, 0.7, 1.0])), float(rng.choice([0.0, 0.5, 0.9]))
    what = f"case {case}: M={M} P={P} variant={variant} kind={theta_kind} D={D} have={have} wire={wire}"
    st = inputs.make_outer_state(M, P, 5000 + case, device=DEV, theta_kind=theta_kind, overlap_steps=D)
    st["outer_mom"][:, :P].normal_(0.0, 1e-3, generator=st["gen"])
    h = host_copy(st)
    h["delta_prev_local"] = h["delta_prev_local"].reshape(D, M, st["stride"])
    h["delta_prev_avg"] = h["delta_prev_avg"].reshape(D, st["stride"])
    scratch = torch.zeros(64, dtype=torch.int32, device=DEV)
    state = binding.State.from_dict(st, outer_lr=eta, outer_momentum=mu, have_prev=have, overlap_steps=D,
                                    comm_scratch=scratch)
    for k in range(D + 2):
        if k:
            inputs.inner_phase_standin(st)
            h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
        state.outer_quantized(variant, *wire)
        have = oracle.outer_step_overlap(variant, k, have, M=M, P=P, stride=st["stride"], eta=eta, mu=mu,
                                         theta=h["theta"], master=h["master"], start=h["start"],
                                         outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                                         delta_prev_avg=h["delta_prev_avg"], theta_kind=theta_kind, comm=wire[0],
                                         exp_bits=wire[1], man_bits=wire[2], nthreads=4)
        torch.cuda.synchronize()
        got = {key: st[key] for key in ("theta", "master", "start", "outer_mom")}
        got["delta_prev_local"] = st["delta_prev_local"].view(D, M, st["stride"])
        got["delta_prev_avg"] = st["delta_prev_avg"].view(D, st["stride"])
        assert_state_equal(got, h, keys=tuple(got), what=f"{what} step {k + 1}")
    state.close()
