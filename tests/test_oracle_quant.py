"""Pins for the oracle's quantised outer-gradient communication (Section 3, "Quantized
Communication": float32, bfloat16, float8 and float4 "using EXMY").

The rounding function is pinned by brute force over every code of a format (nearest value,
ties to the even code), by the well-known value tables of 4-bit E2M1, and by torch's own
float8 conversions where the formats coincide; the step is pinned by a numpy restatement
that uses the brute-force quantiser, by exactness when nothing needs rounding, and by the
fact that only the all-reduce operand changes.
"""
import itertools

import numpy as np
import pytest
import torch

FORMATS = [(2, 1), (3, 0), (4, 3), (5, 2), (3, 2), (2, 3), (1, 2)]


def all_values(X, Y):
    """Every non-negative value of EXMY(X, Y) with its code, from the definition: bias
    2^(X-1)-1, exponent field 0 = subnormal, no infinities or NaNs."""
    bias = (1 << (X - 1)) - 1
    out = []
    for e in range(1 << X):
        for m in range(1 << Y):
            v = (m / (1 << Y)) * 2.0 ** (1 - bias) if e == 0 else (1 + m / (1 << Y)) * 2.0 ** (e - bias)
            out.append((v, (e << Y) | m))
    return out


def brute_round(y, table):
    a = abs(y)
    best = min(table, key=lambda vc: (abs(vc[0] - a), vc[1] & 1))   # nearest, then even code
    return np.sign(y) * best[0]


def test_e2m1_value_table(oracle):
    """The 4-bit float with 2 exponent and 1 mantissa bits: 0, 0.5, 1, 1.5, 2, 3, 4, 6."""
    assert [v for v, _ in all_values(2, 1)] == [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    assert oracle.exmy_max(2, 1) == 6 and oracle.exmy_max(3, 0) == 16
    assert oracle.exmy_max(4, 3) == 480 and oracle.exmy_max(5, 2) == 114688
    for v, _ in all_values(2, 1):
        assert oracle.exmy_round(v, 2, 1) == v and oracle.exmy_round(-v, 2, 1) == -v


@pytest.mark.parametrize("X,Y", FORMATS)
def test_rounding_against_brute_force(oracle, X, Y):
    table = all_values(X, Y)
    top = table[-1][0]
    assert oracle.exmy_max(X, Y) == top
    rng = np.random.default_rng(X * 10 + Y)
    ys = np.concatenate([rng.uniform(-1.05 * top, 1.05 * top, 1500), rng.normal(0, top / 50, 1500),
                         rng.normal(0, table[1][0] * 2, 500), [0.0, top, -top, 2 * top, -3 * top]])
    # every midpoint between neighbours (the ties) and values one fp32 ulp to either side
    vals = [v for v, _ in table]
    mids = [(a + b) / 2 for a, b in zip(vals[:-1], vals[1:])]
    ys = np.concatenate([ys, mids, np.nextafter(np.float32(mids), np.float32(0)).astype(np.float64),
                         np.nextafter(np.float32(mids), np.float32(1e9)).astype(np.float64)])
    for y in ys.astype(np.float32).astype(np.float64):
        assert oracle.exmy_round(float(y), X, Y) == brute_round(float(y), table), (y, X, Y)


def test_rounding_matches_torch_float8_where_formats_coincide(oracle):
    """torch's e4m3fn and e5m2 reserve their top codes (NaN / inf); below those the value
    sets and the round-to-nearest-even rule are the same."""
    rng = np.random.default_rng(0)
    for dt, X, Y, limit in ((torch.float8_e4m3fn, 4, 3, 448.0), (torch.float8_e5m2, 5, 2, 57344.0)):
        y = np.concatenate([rng.uniform(-limit, limit, 4000), rng.normal(0, 1, 4000), rng.normal(0, 1e-2, 2000)])
        y = y.astype(np.float32)
        want = torch.tensor(y).to(dt).float().numpy()
        got = np.array([oracle.exmy_round(float(v), X, Y) for v in y], dtype=np.float32)
        np.testing.assert_array_equal(got, want)


def state(rng, M, P, dtype=np.float32):
    s0 = rng.normal(0, 0.02, size=P)
    st = dict(start=np.tile(s0, (M, 1)).astype(dtype), delta_prev_local=rng.normal(0, 1e-3, (M, P)).astype(dtype),
              outer_mom=rng.normal(0, 1e-3, (M, P)).astype(dtype))
    st["theta"] = (st["start"] + rng.normal(0, 1e-3, (M, P))).astype(dtype)
    st["delta_prev_avg"] = st["delta_prev_local"].mean(0).astype(dtype)
    return st


def run(oracle, variant, st, eta=0.7, mu=0.9, **kw):
    M, P = st["start"].shape
    oracle.outer_step(variant, M=M, P=P, stride=P, eta=eta, mu=mu, theta=st["theta"], start=st["start"],
                      outer_mom=st["outer_mom"], delta_prev_local=st["delta_prev_local"],
                      delta_prev_avg=st["delta_prev_avg"], **kw)


@pytest.mark.parametrize("X,Y", [(2, 1), (3, 0), (4, 3), (5, 2)])
@pytest.mark.parametrize("variant", [0, 1, 2])
def test_quantised_step_against_numpy_restatement(oracle, variant, X, Y):
    """Only line 8's operand is rounded: Delta = (1/M) sum_m scale_m * Q(Delta_m / scale_m)
    with scale_m = max|Delta_m| / max(EXMY); everything local keeps full precision."""
    rng = np.random.default_rng(5 + X)
    M, P = 4, 257
    st = state(rng, M, P)
    before = {k: v.copy() for k, v in st.items()}
    scales = np.zeros(M, np.float32)
    run(oracle, variant, st, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y, scales_out=scales)
    table = all_values(X, Y)
    f = np.float32
    d = before["start"] - before["theta"]                                  # fp32
    want_scale = (np.abs(d).max(1) / f(table[-1][0])).astype(f)
    np.testing.assert_array_equal(scales, want_scale)
    q = np.empty_like(d)
    for m in range(M):
        y = (d[m] / want_scale[m]).astype(f)
        q[m] = (np.array([brute_round(float(v), table) for v in y], dtype=f) * want_scale[m]).astype(f)
    acc = q[0].copy()
    for m in range(1, M):
        acc = (acc + q[m]).astype(f)
    mean = (acc / f(M)).astype(f)
    # replay OuterOpt with that mean (the full-precision step is pinned elsewhere)
    ref = {k: v.copy() for k, v in before.items()}
    if variant == 0:
        # standard consumes the new mean directly: feed it through a one-replica-per-row trick:
        g = np.tile(mean, (M, 1))
    elif variant == 1:
        g = np.tile(before["delta_prev_avg"], (M, 1))
    else:
        g = (((d - before["delta_prev_local"]).astype(f) / f(M)).astype(f) + before["delta_prev_avg"]).astype(f)
    b = ((f(0.9) * before["outer_mom"]).astype(f) + g).astype(f)
    u = (f(0.7) * (g + (f(0.9) * b).astype(f)).astype(f)).astype(f)
    n = (before["start"] - u).astype(f)
    np.testing.assert_array_equal(st["outer_mom"], b)
    np.testing.assert_array_equal(st["start"], n)
    np.testing.assert_array_equal(st["theta"], n)
    if variant != 0:
        np.testing.assert_array_equal(st["delta_prev_avg"], mean)
    if variant == 2:
        np.testing.assert_array_equal(st["delta_prev_local"], d)            # full precision, not the wire value


def test_bf16_wire_format(oracle):
    rng = np.random.default_rng(9)
    M, P = 3, 200
    st = state(rng, M, P)
    d = st["start"] - st["theta"]
    q = torch.tensor(d).to(torch.bfloat16).float().numpy()
    acc = q[0].copy()
    for m in range(1, M):
        acc = acc + q[m]
    run(oracle, 2, st, comm=oracle.COMM_BF16)
    np.testing.assert_array_equal(st["delta_prev_avg"], acc / np.float32(M))
    np.testing.assert_array_equal(st["delta_prev_local"], d)


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_f32_wire_is_the_plain_step(oracle, variant):
    rng = np.random.default_rng(10)
    a = state(rng, 4, 300)
    b = {k: v.copy() for k, v in a.items()}
    run(oracle, variant, a)
    run(oracle, variant, b, comm=oracle.COMM_F32)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_nothing_to_round_means_nothing_changes(oracle):
    """Outer gradients that are already E2M1 numbers times a power-of-two scale pass through
    the wire unchanged, so the quantised and the plain step agree bit for bit."""
    rng = np.random.default_rng(11)
    M, P = 4, 128
    vals = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], np.float32)
    d = (rng.choice(vals, size=(M, P)) * rng.choice([-1, 1], size=(M, P))).astype(np.float32) / 64
    d[:, 0] = 6 / 64                                            # every replica attains the maximum
    st = state(rng, M, P)
    st["start"] = np.round(st["start"] * 256).astype(np.float32) / 256      # keep start - d exact
    st["theta"] = st["start"] - d
    a = {k: v.copy() for k, v in st.items()}
    b = {k: v.copy() for k, v in st.items()}
    run(oracle, 2, a)
    run(oracle, 2, b, comm=oracle.COMM_EXMY, exp_bits=2, man_bits=1)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_quantisation_error_bound_and_zero_gradient(oracle):
    """|Q(x) - x| <= half the spacing at the top binade = amax * 2^-(Y+1) / (2 - 2^-Y) ... and an
    all-zero outer gradient (replica did not move) stays zero with scale 1."""
    rng = np.random.default_rng(12)
    M, P, X, Y = 2, 4096, 4, 3
    st = state(rng, M, P, np.float64)
    st["theta"][1] = st["start"][1]                             # replica 1 did not move
    d = st["start"] - st["theta"]
    plain = {k: v.copy() for k, v in st.items()}
    scales = np.zeros(M)
    run(oracle, 1, st, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y, scales_out=scales)
    run(oracle, 1, plain)
    assert scales[1] == 1.0
    amax = np.abs(d[0]).max()
    bound = amax / 480.0 * 2.0 ** (8 - 3) / 2                  # half the top-binade spacing, in Delta units
    err = np.abs(st["delta_prev_avg"] - plain["delta_prev_avg"]) * M
    assert err.max() <= bound * (1 + 1e-12) and err.max() > 0


def test_first_outer_step_records_wire_mean(oracle):
    rng = np.random.default_rng(13)
    M, P = 4, 100
    st = state(rng, M, P)
    before = {k: v.copy() for k, v in st.items()}
    run(oracle, 2, st, comm=oracle.COMM_BF16, bootstrap=True)
    d = before["start"] - before["theta"]
    q = torch.tensor(d).to(torch.bfloat16).float().numpy()
    acc = q[0].copy()
    for m in range(1, M):
        acc = acc + q[m]
    np.testing.assert_array_equal(st["delta_prev_avg"], acc / np.float32(M))
    np.testing.assert_array_equal(st["delta_prev_local"], d)
    np.testing.assert_array_equal(st["theta"], before["theta"])
    np.testing.assert_array_equal(st["start"], before["theta"])


def test_bad_formats_rejected(oracle):
    st = state(np.random.default_rng(1), 2, 8)
    for X, Y in ((0, 3), (6, 1), (4, 4), (2, -1)):
        with pytest.raises(ValueError):
            run(oracle, 2, st, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y)


# ---------------------------------------------------------------- wire bytes
@pytest.mark.parametrize("X,Y", [(4, 3), (5, 2), (2, 1), (3, 0), (3, 2)])
def test_wire_bytes_against_brute_force_codes(oracle, X, Y):
    """The payload is the code sign|exponent|mantissa of the rounded, scaled element; 4-bit
    codes two per byte, low nibble first.  Codes come from the enumerated value table."""
    rng = np.random.default_rng(20 + X)
    P = 1001
    d = rng.normal(0, 1e-3, P).astype(np.float32)
    d[7] = 0.0
    payload, amax = oracle.wire_encode(d, X, Y)
    table = all_values(X, Y)
    assert amax == np.abs(d).max()
    scale = np.float32(amax) / np.float32(table[-1][0])
    codes = []
    for v in (d / scale).astype(np.float32):
        a = abs(float(v))
        val, code = min(table, key=lambda vc: (abs(vc[0] - a), vc[1] & 1))
        codes.append(code | ((1 if np.signbit(v) else 0) << (X + Y)))
    codes = np.array(codes, dtype=np.uint8)
    if X + Y + 1 <= 4:
        padded = np.concatenate([codes, np.zeros(P % 2, np.uint8)])
        want = padded[0::2] | (padded[1::2] << 4)
    else:
        want = codes
    np.testing.assert_array_equal(payload, want)


@pytest.mark.parametrize("X,Y", [(4, 3), (2, 1), (3, 0)])
def test_wire_round_trip_is_the_quantised_mean_of_the_step(oracle, X, Y):
    """Decoding the workers' payloads and summing them in order gives exactly M times the mean
    that the fused quantised step records."""
    rng = np.random.default_rng(30 + X)
    M, P = 4, 777
    st = state(rng, M, P)
    d = st["start"] - st["theta"]
    rows, amaxes = [], []
    for m in range(M):
        p, a = oracle.wire_encode(d[m], X, Y)
        rows.append(p)
        amaxes.append(a)
    total = oracle.wire_decode_sum(np.stack(rows), np.array(amaxes, np.float32), P, X, Y)
    run(oracle, 2, st, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y)
    np.testing.assert_array_equal(total / np.float32(M), st["delta_prev_avg"])


# ---------------------------------------------------------------- non-finite and vanishing outer gradients
@pytest.mark.parametrize("bad", [np.nan, np.inf, -np.inf])
def test_non_finite_outer_gradient_poisons_the_replicas_scaled_contribution(oracle, bad):
    """EXMY wire: max|Delta_m| propagates NaN and infinity, so the replica's scale is NaN or
    infinite and every element it sends decodes to NaN (x / NaN, 0 * inf): the recorded mean
    is NaN at EVERY index, not a clamped finite number.  The local, full-precision terms are
    untouched: delta_prev_local holds the raw Delta_m.  bf16 wire (no scale): only the bad
    index is non-finite."""
    rng = np.random.default_rng(40)
    M, P = 3, 64
    st = state(rng, M, P)
    st["theta"][1, 5] = bad                                    # Delta_1[5] = start - theta = -bad (or NaN)
    d = st["start"] - st["theta"]
    a = {k: v.copy() for k, v in st.items()}
    scales = np.zeros(M, np.float32)
    run(oracle, 2, a, comm=oracle.COMM_EXMY, exp_bits=4, man_bits=3, bootstrap=True, scales_out=scales)
    assert np.isfinite(scales[0]) and np.isfinite(scales[2]) and not np.isfinite(scales[1])
    assert np.isnan(scales[1]) == np.isnan(bad)
    assert np.isnan(a["delta_prev_avg"]).all()
    np.testing.assert_array_equal(a["delta_prev_local"], d)   # NaN == NaN positionally in this assert
    b = {k: v.copy() for k, v in st.items()}
    run(oracle, 2, b, comm=oracle.COMM_BF16, bootstrap=True)
    finite = np.isfinite(b["delta_prev_avg"])
    assert not finite[5] and finite.sum() == P - 1
    # the rounding itself: NaN stays NaN, infinities saturate to the largest value
    assert np.isnan(oracle.exmy_round(float("nan"), 4, 3))
    assert oracle.exmy_round(float("inf"), 4, 3) == 480.0 and oracle.exmy_round(float("-inf"), 2, 1) == -6.0


def test_scale_that_underflows_is_one_and_the_replica_sends_zeros(oracle):
    """fp32 outer gradients so small that max|Delta_m| / max(EXMY) underflows to zero: the
    scale is 1 (as for a replica that did not move), every element rounds to a zero of its own
    sign, and the mean equals the mean of the other replicas' wire values divided by M."""
    rng = np.random.default_rng(41)
    M, P, X, Y = 2, 128, 4, 3
    st = state(rng, M, P)
    tiny = (rng.integers(-3, 4, P) * np.float32(1e-45)).astype(np.float32)   # multiples of the smallest subnormal
    tiny[0] = np.float32(-0.0)
    assert np.float32(np.abs(tiny).max()) / np.float32(480.0) == 0.0
    st["start"][1] = 0.0
    st["theta"][1] = -tiny                                     # Delta_1 = 0 - (-tiny) = tiny, exactly
    ref = {k: v.copy() for k, v in st.items()}
    ref["theta"][1] = ref["start"][1]                          # the same replica, not moved at all
    scales = np.zeros(M, np.float32)
    run(oracle, 1, st, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y, bootstrap=True, scales_out=scales)
    run(oracle, 1, ref, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y, bootstrap=True)
    assert scales[1] == 1.0
    np.testing.assert_array_equal(st["delta_prev_avg"], ref["delta_prev_avg"])
    # a subnormal scale that does not underflow is kept: amax = 2^-120, scale = 2^-120 / 480 > 0
    st2 = state(rng, M, P)
    st2["start"][1] = 0.0
    st2["theta"][1] = 0.0
    st2["theta"][1, 3] = -np.float32(2.0 ** -120)
    run(oracle, 1, st2, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y, bootstrap=True, scales_out=scales)
    assert scales[1] == np.float32(2.0 ** -120) / np.float32(480.0) and 0 < scales[1] < 1.2e-38


def test_wire_bytes_of_non_finite_outer_gradients(oracle):
    """Every code is finite, so a NaN travels as code 0 next to a NaN (or infinite) maximum
    word; decoding such a payload gives NaN everywhere (0 * NaN, 0 * inf), exactly what the
    fused quantised step records."""
    X, Y, P = 4, 3, 9
    d = np.linspace(-1e-3, 1e-3, P).astype(np.float32)
    d[4] = np.nan
    payload, amax = oracle.wire_encode(d, X, Y)
    assert np.isnan(amax) and (payload == 0).all()             # x / NaN is NaN for every element
    d[4] = np.inf
    payload, amax = oracle.wire_encode(d, X, Y)
    assert np.isinf(amax) and payload[4] == 0                  # inf / inf
    assert set(payload[np.arange(P) != 4]) <= {0x00, 0x80}     # finite / inf = a signed zero
    other = np.full(P, 1e-3, np.float32)
    p2, a2 = oracle.wire_encode(other, X, Y)
    total = oracle.wire_decode_sum(np.stack([p2, payload]), np.array([a2, amax], np.float32), P, X, Y)
    assert np.isnan(total).all()                               # 0 * inf
    # ... which is the mean the fused quantised step records for the same two outer gradients
    st = dict(start=np.zeros((2, P), np.float32), theta=-np.stack([other, d]),
              delta_prev_local=np.zeros((2, P), np.float32), delta_prev_avg=np.zeros(P, np.float32),
              outer_mom=np.zeros((2, P), np.float32))
    run(oracle, 2, st, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y, bootstrap=True)
    assert np.isnan(st["delta_prev_avg"]).all()
