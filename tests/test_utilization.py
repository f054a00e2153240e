"""The compute-utilisation calculator of libdiloco (host only: no GPU needed), pinned on what
the paper prints: the tolerated communication latencies of Table 2 (500M-parameter model, one
step in 0.08 s, H = 30: 0.08 s for 1-inner-step overlap, 2.4 s for 1-outer-step, 4.8 s for
2-outer-steps, 0 without overlap), the definition of compute utilisation in the caption of
Figure 4 (0.8 = 80 % of the time computing, 20 % communicating), and closed forms.  The
paper's Table 4 comes from a DAG simulator specified elsewhere and is not reproduced."""
import math

import pytest

from paper_2502_12996_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def lib():
    build.build_library()
    return binding.load_library()


BASE = dict(P=500_000_000, bits_per_param=32, M=2, H=30, step_time_s=0.08)


def cu(**kw):
    args = dict(BASE, bandwidth_bit_s=1e9)
    args.update(kw)
    return binding.compute_utilization(**args)


def test_tolerated_latencies_of_table_2():
    assert cu(overlap_outer_steps=0)["tolerated_latency_s"] == 0.0
    assert cu(overlap_outer_steps=0, overlap_inner_steps=1)["tolerated_latency_s"] == pytest.approx(0.08, abs=1e-15)
    assert cu(overlap_outer_steps=1)["tolerated_latency_s"] == pytest.approx(2.4, abs=1e-12)
    assert cu(overlap_outer_steps=2)["tolerated_latency_s"] == pytest.approx(4.8, abs=1e-12)


def test_full_utilisation_exactly_while_communication_fits_the_overlap():
    """comm time <= D * H * step time  <=>  utilisation 1."""
    bits = BASE["P"] * 32
    for D, lat in ((1, 2.4), (2, 4.8)):
        w_edge = bits / lat
        assert cu(overlap_outer_steps=D, bandwidth_bit_s=w_edge * 1.0001)["compute_utilization"] == 1.0
        r = cu(overlap_outer_steps=D, bandwidth_bit_s=w_edge * 0.5)
        assert r["comm_time_s"] == pytest.approx(2 * lat) and r["exposed_comm_time_s"] == pytest.approx(lat)
        assert r["compute_utilization"] == pytest.approx(2.4 / (2.4 + lat))
        assert binding.bandwidth_for_utilization(1.0, overlap_outer_steps=D, **BASE) == pytest.approx(w_edge)


def test_definition_of_utilisation_without_overlap():
    """Blocking all-reduce: the share of time spent computing, e.g. 0.8 = 80 % compute, 20 % communication."""
    compute = 30 * 0.08
    comm = compute / 4                                       # 20 % of the total
    r = cu(overlap_outer_steps=0, bandwidth_bit_s=BASE["P"] * 32 / comm)
    assert r["compute_utilization"] == pytest.approx(0.8)
    assert r["compute_time_s"] == pytest.approx(compute) and r["exposed_comm_time_s"] == pytest.approx(comm)
    assert math.isinf(binding.bandwidth_for_utilization(1.0, overlap_outer_steps=0, **BASE))
    assert cu(overlap_outer_steps=0, bandwidth_bit_s=math.inf)["compute_utilization"] == 1.0


def test_monotone_in_bandwidth_and_consistent_inverse():
    prev = 0.0
    for k in range(-2, 12):
        u = cu(bandwidth_bit_s=10.0 ** (6 + k / 2), overlap_outer_steps=1)["compute_utilization"]
        assert u >= prev
        prev = u
    assert prev == 1.0
    for D, tau in ((0, 0), (0, 1), (1, 0), (2, 0)):
        for target in (0.5, 0.8, 0.9, 0.95, 0.99):
            w = binding.bandwidth_for_utilization(target, overlap_outer_steps=D, overlap_inner_steps=tau, **BASE)
            got = cu(overlap_outer_steps=D, overlap_inner_steps=tau, bandwidth_bit_s=w)["compute_utilization"]
            assert got == pytest.approx(target, rel=1e-12)
            assert cu(overlap_outer_steps=D, overlap_inner_steps=tau, bandwidth_bit_s=w * 0.99)["compute_utilization"] < target
    # more overlap never needs more bandwidth, a narrower wire needs proportionally less
    w = [binding.bandwidth_for_utilization(0.95, overlap_outer_steps=D, **BASE) for D in (0, 1, 2)]
    assert w[0] > w[1] > w[2]
    narrow = dict(BASE, bits_per_param=4)
    assert binding.bandwidth_for_utilization(0.95, overlap_outer_steps=1, **narrow) == pytest.approx(w[1] / 8)


def test_wire_width_from_the_library_and_ring_factor():
    P = 1_000_001
    bits = 8 * binding.wire_payload_bytes(P, 2, 1) / P       # 4-bit codes, two per byte
    assert bits == pytest.approx(4.0, rel=1e-5)
    r = binding.compute_utilization(P=P, bits_per_param=bits, M=4, H=100, step_time_s=0.1, bandwidth_bit_s=1e6, ring=True)
    assert r["wire_bits"] == pytest.approx(8 * binding.wire_payload_bytes(P, 2, 1) * 2 * 3 / 4)
    one = binding.compute_utilization(P=P, bits_per_param=32, M=1, H=100, step_time_s=0.1, bandwidth_bit_s=1.0, ring=True)
    assert one["wire_bits"] == 0.0 and one["compute_utilization"] == 1.0     # a single worker exchanges nothing


@pytest.mark.parametrize("kw", [dict(P=0), dict(M=0), dict(H=0), dict(step_time_s=0.0), dict(bits_per_param=-1),
                                dict(bandwidth_bit_s=0.0), dict(overlap_outer_steps=-1), dict(overlap_inner_steps=31),
                                dict(overlap_outer_steps=1, overlap_inner_steps=1), dict(bandwidth_bit_s=float("nan"))])
def test_bad_arguments(kw):
    with pytest.raises(binding.DilocoError) as e:
        cu(**kw)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DilocoError):
        binding.bandwidth_for_utilization(1.5, **BASE)
