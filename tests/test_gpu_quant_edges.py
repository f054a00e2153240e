"""Edge values of the quantised outer step on the GPU against the oracle, element by element:
a replica that did not move (max |Delta_m| = 0, scale 1), outer gradients that are fp32
subnormals or -0 (a scale that underflows), and a NaN or an infinity inside one replica's
outer gradient (the replica's scale is then NaN / infinite and everything it sends decodes to
NaN).  NaN compares equal to NaN, +0 to -0; everything else bit for bit.  Both the fused
M-replica call and the worker pair (codes + maxima gathered, mean formed by every worker)."""
import numpy as np
import pytest
import torch

from paper_2502_12996_b200 import binding, inputs
from gpu_util import assert_state_equal, bits, host_copy, to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
FORMATS = {"bf16": (binding.COMM_BF16, 0, 0), "e4m3": (binding.COMM_EXMY, 4, 3), "e2m1": (binding.COMM_EXMY, 2, 1),
           "e3m0": (binding.COMM_EXMY, 3, 0)}


def plant(st, case, P):
    """Overwrite a few replicas of a seeded fp32 state so that their outer gradients
    Delta_m = start_m - theta_m hit the edge `case`."""
    M = st["M"]
    th, s = st["theta"], st["start"]
    if case == "idle":                                   # replica 0 (and the last one) did not move at all
        th[0, :P] = s[0, :P]
        th[M - 1, :P] = s[M - 1, :P]
    elif case == "subnormal":                            # Delta_1 = integer multiples of 2^-149, some of them -0
        k = torch.randint(-5, 6, (P,), generator=st["gen"], device=DEV).float()
        s[M - 1, :P] = 0.0
        th[M - 1, :P] = -(k * 1.401298464e-45)
        th[M - 1, 0] = 0.0                               # s - theta = 0 - 0
        th[M - 1, 1 % P] = -0.0
        if M > 1:                                        # another replica with a subnormal but non-zero scale
            s[0, :P] = 0.0
            th[0, :P] = k * (2.0 ** -125)
    elif case == "nan":
        th[M - 1, (P // 2) % P] = float("nan")
    elif case == "inf":
        th[0, (P // 3) % P] = float("inf")
        th[M - 1, (P - 1) % P] = float("-inf")
    else:
        raise ValueError(case)


@pytest.mark.parametrize("case", ["idle", "subnormal", "nan", "inf"])
@pytest.mark.parametrize("fmt", list(FORMATS))
@pytest.mark.parametrize("M,P", [(1, 301), (2, 4_099), (4, 10_003), (5, 2_001), (9, 1_025), (16, 3_003)])
def test_fused_quantised_step_edge_values(oracle, case, fmt, M, P):
    comm, X, Y = FORMATS[fmt]
    st = inputs.make_outer_state(M, P, 8800 + M, device=DEV)
    st["outer_mom"][:, :P].normal_(0.0, 1e-3, generator=st["gen"])
    plant(st, case, P)
    h = host_copy(st)
    scratch = torch.zeros(64, dtype=torch.int32, device=DEV)
    for variant in (0, 1, 2):
        dv = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in st.items()}
        hv = {k: (None if v is None else v.copy()) for k, v in h.items()}
        state = binding.State.from_dict(dv, comm_scratch=scratch)
        state.outer_quantized(variant, comm, X, Y)
        oracle.outer_step(variant, M=M, P=P, stride=st["stride"], eta=0.7, mu=0.9, theta=hv["theta"], start=hv["start"],
                          outer_mom=hv["outer_mom"], delta_prev_local=hv["delta_prev_local"],
                          delta_prev_avg=hv["delta_prev_avg"], comm=comm, exp_bits=X, man_bits=Y, nthreads=4)
        torch.cuda.synchronize()
        assert_state_equal(dv, hv, what=f"{case} {fmt} variant {variant} M={M}")
        if case in ("nan", "inf") and comm == binding.COMM_EXMY and variant != 0:
            assert np.isnan(to_numpy(dv["delta_prev_avg"])[:P]).all()       # the whole mean is poisoned
        state.close()


@pytest.mark.parametrize("case", ["idle", "subnormal", "nan", "inf"])
@pytest.mark.parametrize("theta_kind", [1, 2])
def test_fused_quantised_step_edge_values_bf16_storage(oracle, case, theta_kind):
    """The same edges with theta stored as bf16 (Delta_m is formed from the stored value)."""
    M, P = 4, 5_003
    st = inputs.make_outer_state(M, P, 8900, device=DEV, theta_kind=theta_kind)
    val = st["master"] if theta_kind == 2 else st["theta"]
    if case == "idle":
        st["start"][0, :P] = val[0, :P].float()
    elif case == "subnormal":
        st["start"][1, :P] = 0.0
        val[1, :P] = 2.0 ** -130                          # a bf16 (and fp32) subnormal
        val[1, 0] = -0.0
    elif case == "nan":
        val[2, 17] = float("nan")
    else:
        val[3, 99] = float("inf")
    if theta_kind == 2:
        st["theta"].copy_(st["master"])
    h = host_copy(st)
    scratch = torch.zeros(64, dtype=torch.int32, device=DEV)
    state = binding.State.from_dict(st, comm_scratch=scratch)
    for step in range(2):
        state.outer_quantized(binding.EAGER, binding.COMM_EXMY, 4, 3)
        oracle.outer_step(2, M=M, P=P, stride=st["stride"], eta=0.7, mu=0.9, theta=h["theta"], start=h["start"],
                          outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                          delta_prev_avg=h["delta_prev_avg"], master=h["master"], theta_kind=theta_kind,
                          comm=oracle.COMM_EXMY, exp_bits=4, man_bits=3)
        torch.cuda.synchronize()
        assert_state_equal(st, h, what=f"{case} kind {theta_kind} step {step + 1}")
    state.close()


@pytest.mark.parametrize("case", ["idle", "subnormal", "nan", "inf"])
@pytest.mark.parametrize("fmt", [(4, 3), (2, 1), (3, 0)])
@pytest.mark.parametrize("variant,M,P", [(2, 3, 2_003), (0, 2, 1_001), (1, 4, 514)])
def test_worker_pair_edge_values(oracle, case, fmt, variant, M, P):
    """M one-replica workers: send codes + maximum, gather, apply.  Wire bytes and maximum
    words equal the oracle's encoder, the updated state equals the fused quantised oracle."""
    X, Y = fmt
    st = inputs.make_outer_state(M, P, 9100 + M, device=DEV)
    plant(st, case, P)
    stride = st["stride"]
    h = host_copy(st)
    states = [binding.State(M=1, P=P, stride=stride, theta=st["theta"][m], start=st["start"][m],
                            outer_mom=st["outer_mom"][m],
                            delta_prev_local=st["delta_prev_local"][m].clone() if variant == 2 else None, have_prev=0)
              for m in range(M)]
    nbytes = (binding.wire_payload_bytes(P, X, Y) + 15) // 16 * 16
    prev = None
    for k in range(2):                                   # k = 0 records (delayed / eager), k = 1 applies
        new = dict(gathered=torch.zeros((M, nbytes), dtype=torch.uint8, device=DEV),
                   amaxes=torch.zeros(M, dtype=torch.int32, device=DEV))
        if k:                                            # a fresh phase, with the edge planted again
            inputs.inner_phase_standin(st)
            plant(st, case, P)
            h["theta"], h["start"] = to_numpy(st["theta"]), to_numpy(st["start"])
        with np.errstate(invalid="ignore"):                 # inf - inf in the planted cases
            d_before = h["start"] - h["theta"]
        for m in range(M):
            if variant == 0:
                states[m].worker_quantized_send(X, Y, new["gathered"][m], new["amaxes"][m:m + 1])
            else:
                states[m].worker_quantized_apply(variant, M, X, Y, None if prev is None else prev["gathered"],
                                                 None if prev is None else prev["amaxes"], new["gathered"][m],
                                                 new["amaxes"][m:m + 1])
        if variant == 0:
            for m in range(M):
                states[m].worker_quantized_apply(0, M, X, Y, new["gathered"], new["amaxes"], None, None)
        prev = new
        torch.cuda.synchronize()
        for m in range(M):
            want, amax = oracle.wire_encode(np.ascontiguousarray(d_before[m, :P]), X, Y)
            np.testing.assert_array_equal(new["gathered"][m].cpu().numpy()[:len(want)], want)
            got_amax = new["amaxes"][m:m + 1].cpu().numpy().view(np.float32)
            assert (bits(got_amax) == bits(np.array([amax], np.float32))).all(), (m, got_amax, amax)
        oracle.outer_step(variant, M=M, P=P, stride=stride, eta=0.7, mu=0.9, theta=h["theta"], start=h["start"],
                          outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                          delta_prev_avg=h["delta_prev_avg"], bootstrap=(variant != 0 and k == 0),
                          comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y)
        got = dict(theta=st["theta"], start=st["start"], outer_mom=st["outer_mom"])
        assert_state_equal(got, h, keys=tuple(got), what=f"worker pair {case} {fmt} variant {variant} step {k + 1}")
    for s_ in states:
        s_.close()
