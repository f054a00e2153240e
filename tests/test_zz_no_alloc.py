"""diloco_outer_quantized_static: the quantised outer step for callers that cannot hand the
library a scratch buffer (their memory pool owns the whole GPU, or they must not allocate
where they run), so the per-replica maxima are reduced into an array inside the library.

Checked through the C ABI against the ordinary entry point, which takes its scratch from the
caller, and against the CPU oracle: same seeded state, two calls in a row on each side, every
buffer bit-identical after each call (the bar all parity tests here use).  The file name
makes pytest collect it last.
"""
import pytest
import torch

from paper_2502_12996_b200 import binding, inputs
from gpu_util import assert_state_equal, host_copy, to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("theta", "start", "delta_prev_local", "delta_prev_avg", "outer_mom")


def clone_state(st):
    return {k: (v.clone() if torch.is_tensor(v) else v) for k, v in st.items()}


def same_bits(a, b):
    view = torch.int16 if a.dtype == torch.bfloat16 else torch.int32
    return torch.equal(a.view(view), b.view(view))


@pytest.mark.parametrize("M,P,theta_kind,fmt", [(4, 300_003, 0, (binding.COMM_EXMY, 4, 3)),
                                                (16, 40_001, 1, (binding.COMM_EXMY, 2, 1)),
                                                (64, 3_001, 0, (binding.COMM_EXMY, 5, 2)),
                                                (2, 70_001, 0, (binding.COMM_BF16, 0, 0))])
def test_static_scratch_entry_matches_caller_scratch_entry_and_oracle(oracle, M, P, theta_kind, fmt):
    torch.cuda.set_device(0)
    ref = inputs.make_outer_state(M, P, 4242 + M, device=DEV, theta_kind=theta_kind)
    got = clone_state(ref)
    h = host_copy(ref)
    scratch = torch.zeros(64, dtype=torch.int32, device=DEV)
    s_ref = binding.State.from_dict(ref, have_prev=0, comm_scratch=scratch)
    s_got = binding.State.from_dict(got, have_prev=0)              # no scratch buffer at all
    for call in range(2):                                          # t = H bootstrap, then a regular eager step
        if call:
            inputs.inner_phase_standin(ref)
            got["theta"].copy_(ref["theta"])
            h["theta"] = to_numpy(ref["theta"])
        s_ref.outer_quantized(binding.EAGER, *fmt)
        s_got.outer_quantized_static(binding.EAGER, *fmt)
        oracle.outer_step(oracle.EAGER, M=M, P=P, stride=ref["stride"], eta=0.7, mu=0.9, theta=h["theta"],
                          start=h["start"], outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                          delta_prev_avg=h["delta_prev_avg"], theta_kind=theta_kind, bootstrap=(call == 0),
                          comm=fmt[0], exp_bits=fmt[1], man_bits=fmt[2], nthreads=4)
        torch.cuda.synchronize()
        for k in KEYS:
            assert same_bits(got[k], ref[k]), f"{k} differs after call {call + 1}"
        assert_state_equal(got, h, keys=KEYS, what=f"static-scratch entry vs oracle, call {call + 1}")
    assert s_got.get_counters() == s_ref.get_counters() == (0, 2, 1)
    s_ref.close()
    s_got.close()


def test_two_states_share_the_array_back_to_back_on_one_stream(oracle):
    """Every state on a device reduces into the same array.  Calls ordered on one stream do not
    disturb one another: two states of different shapes stepped alternately equal the oracle."""
    torch.cuda.set_device(0)
    shapes = [(8, 20_001, (binding.COMM_EXMY, 4, 3)), (3, 50_003, (binding.COMM_EXMY, 2, 1))]
    sts = [inputs.make_outer_state(M, P, 4300 + M, device=DEV) for M, P, _ in shapes]
    hs = [host_copy(st) for st in sts]
    states = [binding.State.from_dict(st) for st in sts]
    for rnd in range(2):
        for st, h, state, (M, P, fmt) in zip(sts, hs, states, shapes):
            if rnd:
                inputs.inner_phase_standin(st)
                h["theta"] = to_numpy(st["theta"])
            state.outer_quantized_static(binding.EAGER, *fmt)      # no synchronisation between the calls
        torch.cuda.synchronize()
        for st, h, (M, P, fmt) in zip(sts, hs, shapes):
            oracle.outer_step(oracle.EAGER, M=M, P=P, stride=st["stride"], eta=0.7, mu=0.9, theta=h["theta"],
                              start=h["start"], outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                              delta_prev_avg=h["delta_prev_avg"], comm=fmt[0], exp_bits=fmt[1], man_bits=fmt[2])
            assert_state_equal(st, h, keys=KEYS, what=f"shared array, round {rnd + 1}, M={M}")
    for s in states:
        s.close()


def test_static_scratch_entry_rejects_bad_arguments():
    torch.cuda.set_device(0)
    st = inputs.make_outer_state(2, 1000, 1, device=DEV)
    state = binding.State.from_dict(st)
    with pytest.raises(binding.DilocoError) as e:
        state.outer_quantized_static(binding.EAGER, binding.COMM_EXMY, 6, 3)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DilocoError) as e:
        state.outer_quantized_static(5, binding.COMM_BF16)
    assert e.value.status == binding.ERR_INVALID_ARG
    assert binding.load_library().diloco_outer_quantized_static(None, 2, 1, 0, 0, None) == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
