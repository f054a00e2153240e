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
