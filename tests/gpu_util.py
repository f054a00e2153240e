"""Helpers shared by the GPU parity tests: move a seeded state between torch (device) and
numpy (oracle), run both sides, compare bit patterns."""
import numpy as np
import torch

from paper_2502_12996_b200 import binding, inputs

KEYS = ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom", "adam_m", "adam_v")


def to_numpy(t):
    """Device tensor -> host numpy array; bf16 as uint16 bit patterns."""
    if t is None or isinstance(t, np.ndarray):
        return t
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).numpy().view(np.uint16).copy()
    return t.contiguous().numpy().copy()


def host_copy(state):
    return {k: to_numpy(state.get(k)) for k in KEYS}


def guarded(shape, dtype, device, guard=1024, fill=None):
    """A tensor carved out of a larger allocation with sentinel-filled guard zones before and
    after it.  Returns (view, check) where check() asserts the guards are intact."""
    n = int(np.prod(shape))
    raw = torch.empty(n + 2 * guard, dtype=dtype, device=device)
    sentinel = 12345.0
    raw.fill_(sentinel)
    view = raw[guard:guard + n].view(*shape)
    if fill is not None:
        view.copy_(fill)

    def check():
        assert bool((raw[:guard] == sentinel).all()) and bool((raw[guard + n:] == sentinel).all()), "guard zone overwritten"
    return view, check


def with_guards(state, device):
    """Re-home every buffer of a state into guarded allocations."""
    checks = []
    for k in KEYS:
        t = state.get(k)
        if t is None:
            continue
        v, c = guarded(tuple(t.shape), t.dtype, device, fill=t)
        state[k] = v
        checks.append(c)
    return checks


def oracle_outer(oracle, variant, h, M, P, stride, eta, mu, theta_kind, bootstrap=False, nthreads=8):
    oracle.outer_step(variant, M=M, P=P, stride=stride, eta=eta, mu=mu, theta=h["theta"], start=h["start"],
                      outer_mom=h["outer_mom"], delta_prev_local=h["delta_prev_local"],
                      delta_prev_avg=h["delta_prev_avg"], master=h["master"], theta_kind=theta_kind,
                      bootstrap=bootstrap, nthreads=nthreads)


def oracle_adamw(oracle, h, grads_np, M, P, stride, gstride, k, hp, theta_kind, grad_kind, nthreads=8):
    oracle.inner_adamw(M=M, P=P, stride=stride, gstride=gstride, lr=hp["lr"], beta1=hp["beta1"], beta2=hp["beta2"],
                       eps=hp["eps"], wd=hp["wd"], k=k, theta=h["theta"], grads=grads_np, adam_m=h["adam_m"],
                       adam_v=h["adam_v"], master=h["master"], theta_kind=theta_kind, grad_kind=grad_kind,
                       nthreads=nthreads)


def bits(a):
    """Bit patterns with +0 and -0 identified (IEEE equal; the sign of zero is not a result) and
    every NaN mapped to one pattern (which NaN an operation returns is not specified by IEEE
    and differs between the host CPU and the GPU)."""
    if a.dtype == np.float32:
        u = a.view(np.uint32).copy()
        u[u == 0x80000000] = 0
        u[(u & 0x7fffffff) > 0x7f800000] = 0x7fc00000
        return u
    if a.dtype == np.uint16:
        u = a.copy()
        u[u == 0x8000] = 0
        u[(u & 0x7fff) > 0x7f80] = 0x7fc0
        return u
    return a


def assert_state_equal(dev_state, h, keys=KEYS, what=""):
    for k in keys:
        if h.get(k) is None:
            continue
        got = to_numpy(dev_state[k])
        want = h[k]
        same = bits(got) == bits(want)
        if not same.all():
            bad = np.argwhere(~same)
            first = tuple(bad[0])
            raise AssertionError(f"{what} {k}: {len(bad)} of {same.size} elements differ, first at {first}: "
                                 f"gpu={got[first]!r} oracle={want[first]!r}")


def sync_theta_from_host(dev_state, h):
    """Copy host theta (and master) back into the device state: used after both sides applied
    the same host-made inner-phase stand-in."""
    for k in ("theta", "master"):
        if h.get(k) is None:
            continue
        src = torch.from_numpy(h[k].view(np.int16) if h[k].dtype == np.uint16 else h[k])
        if h[k].dtype == np.uint16:
            src = src.view(torch.bfloat16)
        dev_state[k].copy_(src.to(dev_state[k].device))
