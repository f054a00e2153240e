"""Pins for the CPU oracle of the outer step: nothing here touches the CUDA path.

Each test fixes the oracle to something other than itself: hand-worked values
(tests/golden), exact rational evaluation of the paper's SECOND form of the eager gradient,
library routines (torch.optim.SGD with nesterov=True), closed forms and the structural
facts Section 2 states (eager differs from naive delayed only in line 11; replicas stay
equal under the standard step; nothing is applied at t = H).
"""
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest
import torch

GOLDEN = Path(__file__).parent / "golden" / "outer_worked_example.txt"
VARIANTS = {"standard": 0, "delayed": 1, "eager": 2}


def read_golden(path):
    out = {}
    for line in path.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = line.split(":")
        out[key.strip()] = [float(x) for x in val.split()]
    return out


def random_state(rng, M, P, stride=None, dtype=np.float32):
    stride = P if stride is None else stride
    s0 = rng.normal(0, 0.02, size=P)
    st = dict(
        start=np.zeros((M, stride), dtype), theta=np.zeros((M, stride), dtype),
        delta_prev_local=np.zeros((M, stride), dtype), delta_prev_avg=np.zeros(stride, dtype),
        outer_mom=np.zeros((M, stride), dtype))
    st["start"][:, :P] = s0
    st["theta"][:, :P] = s0 + rng.normal(0, 1e-3, size=(M, P))
    st["delta_prev_local"][:, :P] = rng.normal(0, 1e-3, size=(M, P))
    st["delta_prev_avg"][:P] = st["delta_prev_local"][:, :P].astype(np.float64).mean(0)
    st["outer_mom"][:, :P] = rng.normal(0, 1e-3, size=(M, P))
    return st


def clone(st):
    return {k: v.copy() for k, v in st.items()}


def step(oracle, variant, st, M, P, eta, mu, stride=None, **kw):
    stride = st["start"].shape[1] if stride is None else stride
    oracle.outer_step(variant, M=M, P=P, stride=stride, eta=eta, mu=mu, theta=st["theta"], start=st["start"],
                      outer_mom=st["outer_mom"], delta_prev_local=st["delta_prev_local"],
                      delta_prev_avg=st["delta_prev_avg"], **kw)


# ---------------------------------------------------------------- hand-worked example
@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("name", ["standard", "delayed", "eager"])
def test_worked_example(oracle, name, dtype):
    g = read_golden(GOLDEN)
    M, P = int(g["M"][0]), int(g["P"][0])
    arr = lambda k, shape: np.array(g[k], dtype).reshape(shape)
    st = dict(start=arr("start", (M, P)), theta=arr("theta", (M, P)),
              delta_prev_local=arr("delta_prev_local", (M, P)), delta_prev_avg=arr("delta_prev_avg", (P,)),
              outer_mom=np.zeros((M, P), dtype))
    for k in (1, 2):
        if k == 2:
            st["theta"] += arr("inner_phase_2", (M, P))
        step(oracle, VARIANTS[name], st, M, P, g["eta"][0], g["mu"][0])
        np.testing.assert_array_equal(st["theta"], arr(f"{name}_theta_{k}", (M, P)))
        np.testing.assert_array_equal(st["start"], st["theta"])
        np.testing.assert_array_equal(st["outer_mom"], arr(f"{name}_mom_{k}", (M, P)))
        if name != "standard":
            np.testing.assert_array_equal(st["delta_prev_avg"], arr(f"mean_step{k}", (P,)))


# ---------------------------------------------------------------- exact rational brute force
def rational_reference(variant, M, P, eta, mu, start, theta, dpl, dpa, mom, steps, moves):
    """Algorithms 1-3 in exact rationals.  The eager gradient is evaluated in the paper's
    SECOND form, (1/M)(Delta_m + sum_{m' != m} stale Delta_m'), which needs every stale local
    gradient and therefore differs structurally from line 11 that the oracle implements."""
    F = Fraction
    start = [[F(x) for x in r] for r in start]
    theta = [[F(x) for x in r] for r in theta]
    dpl = [[F(x) for x in r] for r in dpl]
    dpa = [F(x) for x in dpa]
    mom = [[F(x) for x in r] for r in mom]
    eta, mu = F(eta), F(mu)
    for k in range(steps):
        if k > 0:
            for m in range(M):
                for i in range(P):
                    theta[m][i] += F(moves[k - 1][m][i])
        for i in range(P):
            d = [start[m][i] - theta[m][i] for m in range(M)]
            mean = sum(d) / M
            for m in range(M):
                if variant == 0:
                    g = mean
                elif variant == 1:
                    g = dpa[i]
                else:
                    g = (d[m] + sum(dpl[q][i] for q in range(M) if q != m)) / M
                mom[m][i] = mu * mom[m][i] + g
                start[m][i] = start[m][i] - eta * (g + mu * mom[m][i])
                theta[m][i] = start[m][i]
            for m in range(M):
                dpl[m][i] = d[m]                 # stale values were needed by every replica above
            dpa[i] = mean
    return theta, mom, dpl, dpa


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("M", [1, 2, 3, 4])
def test_rational_brute_force_f64(oracle, variant, M):
    """General inputs, P = 16, 4 steps: the double oracle agrees with exact rationals to
    rounding (a dropped term, wrong sign or wrong index would be off by ~1e-3)."""
    rng = np.random.default_rng(100 + 10 * variant + M)
    P, steps, eta, mu = 16, 4, 0.7, 0.9
    st = random_state(rng, M, P, dtype=np.float64)
    moves = rng.normal(0, 1e-3, size=(steps - 1, M, P))
    ref = rational_reference(variant, M, P, eta, mu, st["start"], st["theta"], st["delta_prev_local"],
                             st["delta_prev_avg"], st["outer_mom"], steps, moves)
    for k in range(steps):
        if k > 0:
            st["theta"] += moves[k - 1]
        step(oracle, variant, st, M, P, eta, mu)
    np.testing.assert_allclose(st["theta"], np.array(ref[0], dtype=np.float64), rtol=0, atol=1e-15)
    np.testing.assert_allclose(st["outer_mom"], np.array(ref[1], dtype=np.float64), rtol=0, atol=1e-15)
    if variant == 2:
        np.testing.assert_allclose(st["delta_prev_local"], np.array(ref[2], dtype=np.float64), rtol=0, atol=1e-16)
    if variant != 0:
        np.testing.assert_allclose(st["delta_prev_avg"], np.array(ref[3], dtype=np.float64), rtol=0, atol=1e-16)


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_rational_brute_force_f32_exact_on_dyadics(oracle, variant):
    """Inputs on a coarse dyadic grid with eta = mu = 1/2, M = 4: every intermediate is exact
    in fp32, so the fp32 oracle must equal the rational result bit for bit."""
    rng = np.random.default_rng(7 + variant)
    M, P, steps = 4, 16, 3
    q = lambda shape: rng.integers(-8, 9, size=shape) / 8.0
    dpl = q((M, P))
    st = dict(start=np.repeat(q((1, P)), M, 0), delta_prev_local=dpl, delta_prev_avg=dpl.mean(0),
              outer_mom=q((M, P)) / 2)
    st["theta"] = st["start"] + q((M, P))
    moves = q((steps - 1, M, P))
    ref = rational_reference(variant, M, P, 0.5, 0.5, st["start"], st["theta"], st["delta_prev_local"],
                             st["delta_prev_avg"], st["outer_mom"], steps, moves)
    st = {k: np.ascontiguousarray(v, dtype=np.float32) for k, v in st.items()}
    for k in range(steps):
        if k > 0:
            st["theta"] += moves[k - 1].astype(np.float32)
        step(oracle, variant, st, M, P, 0.5, 0.5)
    np.testing.assert_array_equal(st["theta"], np.array(ref[0], dtype=np.float64).astype(np.float32))
    np.testing.assert_array_equal(st["outer_mom"], np.array(ref[1], dtype=np.float64).astype(np.float32))


# ---------------------------------------------------------------- library routine: Nesterov SGD
@pytest.mark.parametrize("eta,mu", [(0.7, 0.9), (0.4, 0.9), (1.0, 0.0)])
def test_standard_equals_torch_sgd_nesterov(oracle, eta, mu):
    """Algorithm 1 line 10 with OuterOpt = SGD(nesterov=True): the outer parameters are the
    optimiser's parameter, the averaged outer gradient its gradient."""
    rng = np.random.default_rng(3)
    M, P, steps = 4, 257, 6
    st = random_state(rng, M, P, dtype=np.float64)
    st["outer_mom"][:] = 0
    param = torch.tensor(st["start"][0].copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([param], lr=eta, momentum=mu, nesterov=(mu > 0))
    for k in range(steps):
        if k > 0:
            st["theta"] = st["start"] + rng.normal(0, 1e-3, size=(M, P))
        mean = (st["start"] - st["theta"]).mean(0)
        param.grad = torch.tensor(mean)
        opt.step()
        step(oracle, 0, st, M, P, eta, mu)
        for m in range(M):
            np.testing.assert_allclose(st["theta"][m], param.detach().numpy(), rtol=0, atol=1e-15)


def test_delayed_equals_torch_sgd_fed_with_previous_mean(oracle):
    """Algorithm 2: the optimiser sees the PREVIOUS phase's mean, one step late."""
    rng = np.random.default_rng(4)
    M, P, steps, eta, mu = 3, 64, 5, 0.4, 0.9
    st = random_state(rng, M, P, dtype=np.float64)
    st["outer_mom"][:] = 0
    param = torch.tensor(st["start"][0].copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([param], lr=eta, momentum=mu, nesterov=True)
    in_flight = st["delta_prev_avg"].copy()
    for k in range(steps):
        if k > 0:
            st["theta"] = st["start"] + rng.normal(0, 1e-3, size=(M, P))
        new_mean = (st["start"] - st["theta"]).mean(0)
        param.grad = torch.tensor(in_flight)
        opt.step()
        step(oracle, 1, st, M, P, eta, mu)
        in_flight = new_mean
        np.testing.assert_allclose(st["theta"][1], param.detach().numpy(), rtol=0, atol=1e-15)
        np.testing.assert_allclose(st["delta_prev_avg"], new_mean, rtol=0, atol=1e-16)


# ---------------------------------------------------------------- special cases the paper fixes
def test_unit_lr_zero_momentum_is_replica_averaging(oracle):
    """eta = 1, mu = 0: OuterOpt(s, Delta) = s - mean(s - theta_m) = mean(theta_m)."""
    rng = np.random.default_rng(5)
    M, P = 4, 1000
    for dtype, tol in ((np.float64, 1e-16), (np.float32, 4 * 2.0 ** -24 * 0.1)):
        st = random_state(rng, M, P, dtype=dtype)
        want = st["theta"].astype(np.float64).mean(0)
        step(oracle, 0, st, M, P, 1.0, 0.0)
        for m in range(M):
            np.testing.assert_allclose(st["theta"][m], want, rtol=0, atol=tol)
        np.testing.assert_array_equal(st["theta"], st["start"])


@pytest.mark.parametrize("M", [1, 2, 4, 8])
def test_eager_equals_delayed_when_local_gradient_repeats(oracle, M):
    """Only line 11 differs between Algorithms 2 and 3; if Delta_m^(t) = Delta_m^(t-H) the
    fresh-minus-stale term is exactly zero and the two must agree bit for bit (fp32)."""
    rng = np.random.default_rng(6 + M)
    P = 513
    a = random_state(rng, M, P)
    a["delta_prev_local"][:] = a["start"] - a["theta"]          # computed in fp32, one rounding
    b = clone(a)
    step(oracle, 2, a, M, P, 0.7, 0.9)
    step(oracle, 1, b, M, P, 0.7, 0.9)
    for k in ("theta", "start", "outer_mom", "delta_prev_avg"):
        np.testing.assert_array_equal(a[k], b[k])


def test_single_replica(oracle):
    """M = 1: the mean is the local gradient; eager's line 11 collapses to the fresh Delta_1
    (stale terms cancel); standard with eta = 1, mu = 0 returns the post-inner parameters."""
    rng = np.random.default_rng(8)
    P = 300
    st = random_state(rng, 1, P, dtype=np.float64)
    st["delta_prev_avg"][:] = st["delta_prev_local"][0]          # mean over one replica
    e, s = clone(st), clone(st)
    post_inner = st["theta"].copy()
    step(oracle, 2, e, 1, P, 0.7, 0.9)
    step(oracle, 0, s, 1, P, 0.7, 0.9)
    np.testing.assert_allclose(e["theta"], s["theta"], rtol=0, atol=1e-17)
    np.testing.assert_allclose(e["outer_mom"], s["outer_mom"], rtol=0, atol=1e-17)
    ident = clone(st)
    step(oracle, 0, ident, 1, P, 1.0, 0.0)
    np.testing.assert_allclose(ident["theta"], post_inner, rtol=0, atol=1e-17)


def test_eager_gradient_two_forms_and_mean_identity(oracle):
    """Section 2.3: line 11 equals the average of the fresh local and the stale non-local
    gradients; summing line 11 over m gives (1/M)(Delta - stale Delta) + stale Delta."""
    rng = np.random.default_rng(9)
    for M in (2, 3, 4, 16):
        P = 128
        st = random_state(rng, M, P, dtype=np.float64)
        kw = dict(M=M, P=P, stride=P, theta=st["theta"], start=st["start"], delta_prev_local=st["delta_prev_local"])
        a = oracle.eager_gradient("a", delta_prev_avg=st["delta_prev_avg"], **kw)
        b = oracle.eager_gradient("b", **kw)
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-17)
        d = st["start"] - st["theta"]
        want_mean = (d.mean(0) - st["delta_prev_avg"]) / M + st["delta_prev_avg"]
        np.testing.assert_allclose(a.mean(0), want_mean, rtol=0, atol=1e-17)
        # and it is what the eager step actually applies: with mu = 0, eta = 1 the step is s - g
        applied = clone(st)
        step(oracle, 2, applied, M, P, 1.0, 0.0)
        np.testing.assert_allclose(st["start"] - applied["theta"], a, rtol=0, atol=1e-17)


def test_momentum_closed_form(oracle):
    """Constant gradient g for k steps: b_k = g (1 - mu^k)/(1 - mu), step_k = eta (g + mu b_k)."""
    M, P, eta, mu, g = 2, 8, 0.4, 0.9, 0.125
    st = dict(start=np.full((M, P), 3.0), theta=None, delta_prev_local=np.zeros((M, P)),
              delta_prev_avg=np.zeros(P), outer_mom=np.zeros((M, P)))
    total = 0.0
    for k in range(1, 8):
        st["theta"] = st["start"] - g                            # every replica moved by -g
        before = st["start"].copy()
        step(oracle, 0, st, M, P, eta, mu)
        bk = g * (1 - mu ** k) / (1 - mu)
        np.testing.assert_allclose(st["outer_mom"], bk, rtol=1e-14)
        np.testing.assert_allclose(before - st["start"], eta * (g + mu * bk), rtol=1e-13)


@pytest.mark.parametrize("variant", [1, 2])
def test_first_outer_step_applies_nothing(oracle, variant):
    """t = H: the 'if t > H' branch is skipped.  theta and momentum are untouched, the mean
    and (eager) the local gradients are recorded, the current parameters become the start."""
    rng = np.random.default_rng(10)
    M, P = 4, 200
    st = random_state(rng, M, P)
    before = clone(st)
    step(oracle, variant, st, M, P, 0.7, 0.9, bootstrap=True)
    np.testing.assert_array_equal(st["theta"], before["theta"])
    np.testing.assert_array_equal(st["outer_mom"], before["outer_mom"])
    np.testing.assert_array_equal(st["start"], before["theta"])
    d = before["start"] - before["theta"]
    acc = d[0].copy()
    for m in range(1, M):
        acc = acc + d[m]
    np.testing.assert_array_equal(st["delta_prev_avg"], acc / np.float32(M))
    if variant == 2:
        np.testing.assert_array_equal(st["delta_prev_local"], d)
    else:
        np.testing.assert_array_equal(st["delta_prev_local"], before["delta_prev_local"])


def test_replicas_stay_identical_under_standard_and_delayed_momentum(oracle):
    """Standard DiLoCo re-synchronises: all theta_m equal after every step.  Under naive
    delayed every replica consumes the same gradient sequence, so the momenta stay equal."""
    rng = np.random.default_rng(11)
    M, P = 4, 100
    for variant in (0, 1):
        st = random_state(rng, M, P)
        st["outer_mom"][:] = 0
        for k in range(4):
            if k:
                st["theta"][:] = st["start"] + rng.normal(0, 1e-3, size=(M, P)).astype(np.float32)
            step(oracle, variant, st, M, P, 0.7, 0.9)
            for m in range(1, M):
                np.testing.assert_array_equal(st["outer_mom"][m], st["outer_mom"][0])
                np.testing.assert_array_equal(st["theta"][m], st["theta"][0])


def test_eager_replicas_diverge(oracle):
    """Section 2.2 item 1: under delayed/eager the per-worker parameters are never
    synchronised; with different local gradients the eager replicas must differ."""
    rng = np.random.default_rng(12)
    st = random_state(rng, 2, 50)
    step(oracle, 2, st, 2, 50, 0.7, 0.9)
    assert np.abs(st["theta"][0] - st["theta"][1]).max() > 1e-5


def test_padding_untouched_and_slice_independence(oracle):
    """Elements i >= P are never written; running on a sub-range of indices gives the same
    bits as the full run (every index is independent)."""
    rng = np.random.default_rng(13)
    M, P, stride = 3, 1000, 1024
    for variant in (0, 1, 2):
        st = random_state(rng, M, P, stride)
        for v in st.values():
            v[..., P:] = 777.0
        full = clone(st)
        step(oracle, variant, full, M, P, 0.7, 0.9)
        for v in full.values():
            assert (v[..., P:] == 777.0).all()
        a, b = 137, 811
        part = {k: np.ascontiguousarray(v[..., a:b]) for k, v in st.items()}
        step(oracle, variant, part, M, b - a, 0.7, 0.9, stride=b - a)
        for k in part:
            np.testing.assert_array_equal(part[k], full[k][..., a:b])


def test_thread_count_does_not_change_bits(oracle):
    rng = np.random.default_rng(14)
    M, P = 4, 50_000
    a = random_state(rng, M, P)
    b = clone(a)
    step(oracle, 2, a, M, P, 0.7, 0.9, nthreads=1)
    step(oracle, 2, b, M, P, 0.7, 0.9, nthreads=4)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_f32_tracks_f64(oracle):
    """The fp32 oracle is the double oracle up to fp32 rounding (a few ulp of the 0.02-sized
    parameters over 3 steps)."""
    rng = np.random.default_rng(15)
    M, P = 4, 4096
    for variant in (0, 1, 2):
        d = random_state(rng, M, P, dtype=np.float64)
        f = {k: v.astype(np.float32) for k, v in d.items()}
        d = {k: v.astype(np.float64) for k, v in f.items()}
        for _ in range(3):
            step(oracle, variant, d, M, P, 0.7, 0.9)
            step(oracle, variant, f, M, P, 0.7, 0.9)
            noise = rng.normal(0, 1e-3, size=(M, P)).astype(np.float32)
            d["theta"] = d["start"] + noise
            f["theta"] = f["start"] + noise
        np.testing.assert_allclose(f["start"], d["start"], rtol=0, atol=2e-7)


# ---------------------------------------------------------------- bf16 storage
def test_bf16_rounding_matches_torch(oracle):
    rng = np.random.default_rng(16)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-3, 2000), [0.0, -0.0, 1.0, 3.0e38, 1e-40]])
    x = x.astype(np.float32)
    # exact ties: mantissa low half = 0x8000, both parities of the kept lsb
    ties = np.array([0x3f808000, 0x3f818000, 0xbf808000, 0x3f80ffff, 0x3f808001], dtype=np.uint32).view(np.float32)
    x = np.concatenate([x, ties])
    want = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16(float(v)) for v in x], dtype=np.uint16)
    np.testing.assert_array_equal(got, want)
    back = np.array([oracle.bf16_to_f32(int(h)) for h in want], dtype=np.float32)
    np.testing.assert_array_equal(back, torch.tensor(x).to(torch.bfloat16).float().numpy())


@pytest.mark.parametrize("kind", [1, 2])
def test_bf16_storage_modes(oracle, kind):
    """bf16 theta: Delta_m is formed from the stored (rounded) value and the new theta is the
    fp32 result rounded to nearest even.  Master mode: Delta_m comes from the fp32 master and
    both copies are written.  Checked against the native fp32 run on the same values."""
    rng = np.random.default_rng(17)
    M, P = 4, 2048
    st = random_state(rng, M, P)
    theta_bf = torch.tensor(st["theta"]).to(torch.bfloat16)
    bits = theta_bf.view(torch.int16).numpy().view(np.uint16).copy()
    ref = clone(st)
    if kind == 1:
        ref["theta"] = theta_bf.float().numpy().copy()           # what is stored is what counts
        master = None
    else:
        master = st["theta"].copy()
    step(oracle, 2, ref, M, P, 0.7, 0.9)
    got = clone(st)
    got["theta"] = bits
    oracle.outer_step(2, M=M, P=P, stride=P, eta=0.7, mu=0.9, theta=got["theta"], start=got["start"],
                      outer_mom=got["outer_mom"], delta_prev_local=got["delta_prev_local"],
                      delta_prev_avg=got["delta_prev_avg"], master=master, theta_kind=kind)
    for k in ("start", "outer_mom", "delta_prev_local", "delta_prev_avg"):
        np.testing.assert_array_equal(got[k], ref[k])
    want_bits = torch.tensor(ref["start"]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got["theta"], want_bits)
    if kind == 2:
        np.testing.assert_array_equal(master, ref["start"])
