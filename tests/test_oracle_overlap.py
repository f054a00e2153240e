"""Pins for the oracle's D-outer-steps overlap (Section 3, "Two-outer-steps overlap").

The paper prints no formula for D = 2, so the reading (line 11 of Algorithm 3 with t-H replaced
by t-DH) cannot be pinned to the paper; what is pinned here is that the oracle implements that
reading: against an exact-rational evaluation that keeps the whole gradient history in plain
lists (no ring, and the eager gradient in the "fresh local + stale non-local" form), that D = 1
is the ordinary step, and that the first D steps apply nothing.
"""
from fractions import Fraction

import numpy as np
import pytest


def make(rng, D, M, P, dtype=np.float64):
    s0 = rng.normal(0, 0.02, size=P)
    st = dict(start=np.tile(s0, (M, 1)).astype(dtype), outer_mom=np.zeros((M, P), dtype),
              delta_prev_local=np.zeros((D, M, P), dtype), delta_prev_avg=np.zeros((D, P), dtype))
    st["theta"] = (st["start"] + rng.normal(0, 1e-3, (M, P))).astype(dtype)
    return st


def run(oracle, variant, st, steps, moves, eta=0.7, mu=0.9, have=0):
    M, P = st["start"].shape
    for k in range(steps):
        if k:
            st["theta"][:] = st["start"] + moves[k - 1]
        have = oracle.outer_step_overlap(variant, k, have, M=M, P=P, stride=P, eta=eta, mu=mu, theta=st["theta"],
                                         start=st["start"], outer_mom=st["outer_mom"],
                                         delta_prev_local=st["delta_prev_local"], delta_prev_avg=st["delta_prev_avg"])
    return have


def rational_history(variant, D, M, P, eta, mu, start, theta0, moves, steps):
    F = Fraction
    start = [[F(float(x)) for x in r] for r in start]
    theta = [[F(float(x)) for x in r] for r in theta0]
    mom = [[F(0)] * P for _ in range(M)]
    hist_local, hist_mean = [], []                  # one entry per outer step, never overwritten
    for k in range(steps):
        if k:
            theta = [[start[m][i] + F(float(moves[k - 1][m][i])) for i in range(P)] for m in range(M)]
        d = [[start[m][i] - theta[m][i] for i in range(P)] for m in range(M)]
        mean = [sum(d[m][i] for m in range(M)) / M for i in range(P)]
        if k >= D:                                   # the all-reduce of step k-D has arrived
            old_l, old_m = hist_local[k - D], hist_mean[k - D]
            for m in range(M):
                for i in range(P):
                    if variant == 1:
                        g = old_m[i]
                    else:
                        g = (d[m][i] + sum(old_l[q][i] for q in range(M) if q != m)) / M
                    mom[m][i] = mu * mom[m][i] + g
                    start[m][i] = start[m][i] - eta * (g + mu * mom[m][i])
            theta = [row[:] for row in start]
        else:
            start = [row[:] for row in theta]        # nothing arrived: keep the local progress
        hist_local.append(d)
        hist_mean.append(mean)
    return start, mom


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("D,M", [(1, 2), (2, 2), (2, 3), (3, 4)])
def test_against_rational_history(oracle, variant, D, M):
    rng = np.random.default_rng(10 * D + M + variant)
    P, steps = 6, 2 * D + 3
    st = make(rng, D, M, P)
    moves = rng.normal(0, 1e-3, size=(steps - 1, M, P))
    start0, theta0 = st["start"].copy(), st["theta"].copy()
    have = run(oracle, variant, st, steps, moves)
    assert have == D
    want_start, want_mom = rational_history(variant, D, M, P, Fraction(0.7), Fraction(0.9), start0, theta0, moves, steps)
    np.testing.assert_allclose(st["start"], np.array(want_start, dtype=np.float64), rtol=0, atol=1e-15)
    np.testing.assert_allclose(st["outer_mom"], np.array(want_mom, dtype=np.float64), rtol=0, atol=1e-15)


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_one_generation_is_the_ordinary_step(oracle, variant):
    rng = np.random.default_rng(3)
    M, P, steps = 4, 64, 4
    a = make(rng, 1, M, P, np.float32)
    b = {k: v.copy() for k, v in a.items()}
    moves = rng.normal(0, 1e-3, size=(steps - 1, M, P)).astype(np.float32)
    run(oracle, variant, a, steps, moves)
    for k in range(steps):
        if k:
            b["theta"][:] = b["start"] + moves[k - 1]
        oracle.outer_step(variant, M=M, P=P, stride=P, eta=0.7, mu=0.9, theta=b["theta"], start=b["start"],
                          outer_mom=b["outer_mom"], delta_prev_local=b["delta_prev_local"][0],
                          delta_prev_avg=b["delta_prev_avg"][0], bootstrap=(variant != 0 and k == 0))
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_first_D_steps_only_record(oracle):
    rng = np.random.default_rng(4)
    D, M, P = 2, 3, 16
    st = make(rng, D, M, P, np.float32)
    moves = rng.normal(0, 1e-3, size=(D, M, P)).astype(np.float32)
    thetas = []
    have = 0
    for k in range(D):
        if k:
            st["theta"][:] = st["start"] + moves[k - 1]
        thetas.append(st["theta"].copy())
        d = st["start"] - st["theta"]
        have = oracle.outer_step_overlap(2, k, have, M=M, P=P, stride=P, eta=0.7, mu=0.9, theta=st["theta"],
                                         start=st["start"], outer_mom=st["outer_mom"],
                                         delta_prev_local=st["delta_prev_local"], delta_prev_avg=st["delta_prev_avg"])
        np.testing.assert_array_equal(st["theta"], thetas[-1])
        np.testing.assert_array_equal(st["start"], thetas[-1])
        np.testing.assert_array_equal(st["delta_prev_local"][k], d)
        assert not st["outer_mom"].any()
    assert have == D


# ---------------------------------------------------------------- fragments on their own schedules
def _frag_state(rng, D, M, P):
    f = np.float32
    s0 = rng.normal(0, 0.02, P)
    st = dict(start=np.tile(s0, (M, 1)).astype(f), outer_mom=rng.normal(0, 1e-3, (M, P)).astype(f),
              delta_prev_local=rng.normal(0, 1e-3, (D, M, P)).astype(f))
    st["theta"] = (st["start"] + rng.normal(0, 1e-3, (M, P))).astype(f)
    st["delta_prev_avg"] = st["delta_prev_local"].mean(1).astype(f)
    return st


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("D", [1, 2])
def test_fragments_stepped_together_equal_the_whole_vector(oracle, variant, D):
    """All fragments of a partition stepped at the same outer step, in any order, give the bits
    of one whole-vector step (slice independence, now through the fragment helper)."""
    rng = np.random.default_rng(70 + D)
    M, P = 3, 96
    a = _frag_state(rng, D, M, P)
    b = {k: v.copy() for k, v in a.items()}
    cuts = [(64, 32), (0, 40), (40, 24)]
    have_a, have_b = 0, [0, 0, 0]
    for k in range(2 * D + 1):
        if k:
            noise = rng.normal(0, 1e-3, (M, P)).astype(np.float32)
            a["theta"] = a["start"] + noise
            b["theta"] = b["start"] + noise
        have_a = oracle.outer_step_overlap(variant, k, have_a, M=M, P=P, stride=P, eta=0.7, mu=0.9, **a)
        for f, (off, ln) in enumerate(cuts):
            have_b[f] = oracle.outer_step_fragment(variant, k, have_b[f], off, ln, M=M, eta=0.7, mu=0.9, **b)
        for key in a:
            np.testing.assert_array_equal(a[key], b[key], err_msg=f"{key} step {k}")
        assert have_b == [have_a] * 3


def test_a_fragment_step_touches_only_its_fragment_and_schedules_commute(oracle):
    """A step of one fragment leaves every index outside it untouched, bit for bit, so steps of
    different fragments commute: a staggered schedule equals the same steps taken fragment by
    fragment."""
    rng = np.random.default_rng(75)
    D, M, P = 2, 2, 128
    st = _frag_state(rng, D, M, P)
    thetas = [(st["start"] + rng.normal(0, 1e-3, (M, P))).astype(np.float32) for _ in range(6)]
    cuts = [(0, 32), (32, 64), (96, 32)]
    schedule = [(t, f) for t in range(6) for f in range(3) if t % 3 == f]            # staggered: fragment f at t = f mod 3

    def run(order):
        s = {k: v.copy() for k, v in st.items()}
        have, count = [0, 0, 0], [0, 0, 0]
        for t, f in order:
            s["theta"] = thetas[t].copy()
            off, ln = cuts[f]
            before = {k: v.copy() for k, v in s.items()}
            have[f] = oracle.outer_step_fragment(2, count[f], have[f], off, ln, M=M, eta=0.7, mu=0.9, **s)
            count[f] += 1
            outside = np.ones(P, bool)
            outside[off:off + ln] = False
            for key in s:
                np.testing.assert_array_equal(s[key][..., outside], before[key][..., outside])
        return s

    a = run(schedule)
    # theta is an input of each step (set from the same list), so compare what the steps own
    b = run(sorted(schedule, key=lambda tf: (tf[1], tf[0])))
    for key in ("start", "outer_mom", "delta_prev_local", "delta_prev_avg"):
        np.testing.assert_array_equal(a[key], b[key], err_msg=key)


def test_quantised_fragment_takes_its_scale_from_the_fragment(oracle):
    """A fragment is what one exchange carries, so its EXMY scale is the maximum over the
    fragment's own indices: the step equals the whole-vector quantised step of the slice taken on
    its own, and differs from a step whose scale came from a larger outer gradient elsewhere."""
    rng = np.random.default_rng(77)
    D, M, P = 1, 2, 96
    st = _frag_state(rng, D, M, P)
    st["theta"][0, 80] = st["start"][0, 80] - 1.0             # a huge outer gradient outside the fragment [0, 64)
    a = {k: v.copy() for k, v in st.items()}
    oracle.outer_step_fragment(2, 0, 1, 0, 64, M=M, eta=0.7, mu=0.9, comm=oracle.COMM_EXMY, exp_bits=2, man_bits=1, **a)
    b = {k: np.ascontiguousarray(v[..., :64]) for k, v in st.items()}
    oracle.outer_step(2, M=M, P=64, stride=64, eta=0.7, mu=0.9, comm=oracle.COMM_EXMY, exp_bits=2, man_bits=1,
                      theta=b["theta"], start=b["start"], outer_mom=b["outer_mom"],
                      delta_prev_local=b["delta_prev_local"][0], delta_prev_avg=b["delta_prev_avg"][0])
    for key in a:
        np.testing.assert_array_equal(a[key][..., :64], b[key], err_msg=key)
        np.testing.assert_array_equal(a[key][..., 64:], st[key][..., 64:], err_msg=key)   # the rest untouched
    c = {k: v.copy() for k, v in st.items()}
    oracle.outer_step(2, M=M, P=P, stride=P, eta=0.7, mu=0.9, comm=oracle.COMM_EXMY, exp_bits=2, man_bits=1,
                      theta=c["theta"], start=c["start"], outer_mom=c["outer_mom"],
                      delta_prev_local=c["delta_prev_local"][0], delta_prev_avg=c["delta_prev_avg"][0])
    assert not np.array_equal(c["delta_prev_avg"][0, :64], a["delta_prev_avg"][0, :64])   # the whole-vector scale is coarser
