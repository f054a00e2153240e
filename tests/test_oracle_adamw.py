"""Pins for the CPU oracle of the inner AdamW step (InnerOpt of Algorithms 1-3, line 5).

Pinned against torch.optim.AdamW on CPU (a library routine), closed forms for constant and
zero gradients, hand-computed dyadic values, and the storage modes against the native run.
"""
import numpy as np
import pytest
import torch

HP = dict(lr=4e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1)


def run(oracle, theta, grads_seq, adam_m, adam_v, k0=1, hp=HP, **kw):
    M, stride = adam_m.shape
    P = kw.pop("P", stride)
    for j, g in enumerate(grads_seq):
        oracle.inner_adamw(M=M, P=P, stride=stride, gstride=g.shape[1], k=k0 + j, theta=theta, grads=g,
                           adam_m=adam_m, adam_v=adam_v, **hp, **kw)


@pytest.mark.parametrize("dtype,tol", [(np.float64, 1e-12), (np.float32, 2e-6)])
def test_matches_torch_adamw(oracle, dtype, tol):
    """120 steps, P = 1024, 2 replicas, against torch.optim.AdamW (amsgrad off) in the same
    precision.  Relative tolerance covers the different operation order inside torch."""
    rng = np.random.default_rng(0)
    M, P, steps = 2, 1024, 120
    theta = rng.normal(0, 0.02, size=(M, P)).astype(dtype)
    tdt = torch.float64 if dtype == np.float64 else torch.float32
    params = [torch.tensor(theta[m].copy(), dtype=tdt, requires_grad=True) for m in range(M)]
    opt = torch.optim.AdamW(params, lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]), eps=HP["eps"],
                            weight_decay=HP["wd"], amsgrad=False)
    am, av = np.zeros((M, P), dtype), np.zeros((M, P), dtype)
    for k in range(1, steps + 1):
        g = rng.normal(0, 1e-2, size=(M, P)).astype(dtype)
        for m in range(M):
            params[m].grad = torch.tensor(g[m], dtype=tdt)
        opt.step()
        run(oracle, theta, [g], am, av, k0=k)
    for m in range(M):
        want = params[m].detach().numpy()
        np.testing.assert_allclose(theta[m], want, rtol=tol, atol=tol * 0.05)   # abs: 0.02-sized parameters, 120 steps
        st = opt.state[params[m]]
        np.testing.assert_allclose(am[m], st["exp_avg"].numpy(), rtol=tol * 10, atol=tol * 1e-3)   # moments ~3e-3, cancel near zero
        np.testing.assert_allclose(av[m], st["exp_avg_sq"].numpy(), rtol=tol * 10, atol=tol * 1e-5)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_hand_computed_dyadic_steps(oracle, dtype):
    """The hand-worked steps of tests/golden/adamw_worked_example.txt (derivation in the file);
    all values exact in fp32."""
    from pathlib import Path
    g = {}
    for line in (Path(__file__).parent / "golden" / "adamw_worked_example.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            key, val = line.split(":")
            g[key.strip()] = float(val)
    hp = dict(lr=g["lr"], beta1=g["beta1"], beta2=g["beta2"], eps=g["eps"], wd=g["wd"])
    theta = np.full((1, 4), g["theta0"], dtype)
    grad = np.full((1, 4), g["g"], dtype)
    am, av = np.zeros((1, 4), dtype), np.zeros((1, 4), dtype)
    for k in (1, 2):
        run(oracle, theta, [grad], am, av, k0=k, hp=hp)
        np.testing.assert_array_equal(theta, g[f"theta_{k}"])
        np.testing.assert_array_equal(am, g[f"m_{k}"])
        np.testing.assert_array_equal(av, g[f"v_{k}"])


def test_zero_gradient_is_pure_decay(oracle):
    """g = 0: the Adam term vanishes (0 / (0 + eps)), theta_k = theta_0 (1 - lr wd)^k."""
    theta = np.full((1, 8), 2.0)
    g = np.zeros((1, 8))
    am, av = np.zeros((1, 8)), np.zeros((1, 8))
    run(oracle, theta, [g] * 10, am, av)
    np.testing.assert_allclose(theta, 2.0 * (1 - HP["lr"] * HP["wd"]) ** 10, rtol=1e-14)


def test_first_step_is_sign_descent(oracle):
    """wd = 0, eps tiny, k = 1: mhat = g, vhat = g^2, so theta_1 = theta_0 - lr sign(g)."""
    rng = np.random.default_rng(1)
    g = rng.normal(0, 1e-2, size=(1, 64))
    theta = rng.normal(0, 1, size=(1, 64))
    want = theta - 1e-3 * np.sign(g)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-30, wd=0.0)
    run(oracle, theta, [g], np.zeros((1, 64)), np.zeros((1, 64)), hp=hp)
    np.testing.assert_allclose(theta, want, rtol=0, atol=1e-15)


def test_weight_decay_is_decoupled(oracle):
    """The decay term lr*wd*theta is added outside the adaptive ratio: two runs that differ
    only in wd differ by exactly that term on the first step."""
    rng = np.random.default_rng(2)
    g = rng.normal(0, 1e-2, size=(1, 32))
    t0 = rng.normal(0, 1, size=(1, 32))
    a, b = t0.copy(), t0.copy()
    run(oracle, a, [g], np.zeros((1, 32)), np.zeros((1, 32)), hp=dict(HP, wd=0.0))
    run(oracle, b, [g], np.zeros((1, 32)), np.zeros((1, 32)), hp=dict(HP, wd=0.1))
    np.testing.assert_allclose(a - b, HP["lr"] * 0.1 * t0, rtol=1e-9)


def test_step_counter_drives_bias_correction(oracle):
    """Running step k with the wrong k changes the result (bias correction is on), and a
    resumed run (moments + counter restored) continues bit for bit."""
    rng = np.random.default_rng(3)
    M, P = 2, 512
    gs = [rng.normal(0, 1e-2, size=(M, P)).astype(np.float32) for _ in range(6)]
    t0 = rng.normal(0, 0.02, size=(M, P)).astype(np.float32)
    a, am, av = t0.copy(), np.zeros((M, P), np.float32), np.zeros((M, P), np.float32)
    run(oracle, a, gs, am, av)
    b, bm, bv = t0.copy(), np.zeros((M, P), np.float32), np.zeros((M, P), np.float32)
    run(oracle, b, gs[:2], bm, bv, k0=1)
    b2, bm2, bv2 = b.copy(), bm.copy(), bv.copy()                # "checkpoint"
    run(oracle, b2, gs[2:], bm2, bv2, k0=3)
    np.testing.assert_array_equal(a, b2)
    wrong = b.copy()
    run(oracle, wrong, gs[2:], bm.copy(), bv.copy(), k0=1)
    assert np.abs(wrong - a).max() > 1e-6


def to_bf16_bits(x):
    return torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()


def from_bf16_bits(b):
    return torch.tensor(b.view(np.int16)).view(torch.bfloat16).float().numpy()


@pytest.mark.parametrize("theta_kind", [1, 2])
def test_bf16_storage_modes(oracle, theta_kind):
    """bf16 gradients are widened exactly; bf16 theta is re-read as stored each step; the
    master mode carries fp32 and writes a rounded copy.  Checked against the native run fed
    with the same (already rounded) values, step by step."""
    rng = np.random.default_rng(4)
    M, P, stride, steps = 2, 777, 832, 5
    theta0 = np.zeros((M, stride), np.float32)
    theta0[:, :P] = rng.normal(0, 0.02, size=(M, P))
    gs = [to_bf16_bits(np.pad(rng.normal(0, 1e-2, size=(M, P)).astype(np.float32), ((0, 0), (0, stride - P))))
          for _ in range(steps)]
    bits = to_bf16_bits(theta0)
    master = theta0.copy() if theta_kind == 2 else None
    am, av = np.zeros((M, stride), np.float32), np.zeros((M, stride), np.float32)
    rm, rv = am.copy(), av.copy()
    ref = from_bf16_bits(bits) if theta_kind == 1 else theta0.copy()
    for k in range(1, steps + 1):
        oracle.inner_adamw(M=M, P=P, stride=stride, gstride=stride, k=k, theta=bits, grads=gs[k - 1], adam_m=am,
                           adam_v=av, master=master, theta_kind=theta_kind, grad_kind=1, **HP)
        g32 = from_bf16_bits(gs[k - 1])
        oracle.inner_adamw(M=M, P=P, stride=stride, gstride=stride, k=k, theta=ref, grads=g32, adam_m=rm,
                           adam_v=rv, **HP)
        np.testing.assert_array_equal(am, rm)
        np.testing.assert_array_equal(av, rv)
        np.testing.assert_array_equal(bits[:, :P], to_bf16_bits(ref)[:, :P])
        if theta_kind == 1:
            ref = from_bf16_bits(to_bf16_bits(ref))              # next step reads the stored value
        else:
            np.testing.assert_array_equal(master, ref)
    assert (bits[:, P:] == 0).all() and (am[:, P:] == 0).all()   # padding untouched


def test_thread_count_does_not_change_bits(oracle):
    rng = np.random.default_rng(5)
    M, P = 2, 40_000
    g = rng.normal(0, 1e-2, size=(M, P)).astype(np.float32)
    t0 = rng.normal(0, 0.02, size=(M, P)).astype(np.float32)
    outs = []
    for nt in (1, 4):
        t, am, av = t0.copy(), np.zeros((M, P), np.float32), np.zeros((M, P), np.float32)
        oracle.inner_adamw(M=M, P=P, stride=P, gstride=P, k=1, theta=t, grads=g, adam_m=am, adam_v=av,
                           nthreads=nt, **HP)
        outs.append((t, am, av))
    for x, y in zip(*outs):
        np.testing.assert_array_equal(x, y)
