"""CPU oracle for the DiLoCo outer step (standard / naive delayed / eager) and inner AdamW.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module; it is used
by the test-suite, by the smoke check and by the benchmark's CPU-baseline leg.  The
arithmetic lives in ``diloco_oracle.c`` (plain scalar loops written from Algorithms 1-3 of
the paper); this file only compiles that C file with gcc and marshals numpy arrays into it.

Two precisions are exported, ``f32`` (one IEEE rounding per written operation, the parity
target of the GPU kernels) and ``f64`` (same steps in double, used as truth in tolerance
checks).  Arrays are updated IN PLACE.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "diloco_oracle.c"
_LIB = _HERE / "libdiloco_oracle.so"

STANDARD, DELAYED, EAGER = 0, 1, 2
THETA_NATIVE, THETA_BF16, THETA_MASTER_BF16 = 0, 1, 2
GRAD_NATIVE, GRAD_BF16 = 0, 1
COMM_F32, COMM_BF16, COMM_EXMY = 0, 1, 2

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc: no FMA contraction, no fast-math, OpenMP for the timed leg."""
    if _LIB.exists() and not force and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    common = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-c", str(_SRC)]
    o32, o64 = _HERE / "oracle_f32.o", _HERE / "oracle_f64.o"
    subprocess.check_call(common + ["-DREAL=float", "-DSFX=f32", "-o", str(o32)])
    subprocess.check_call(common + ["-DREAL=double", "-DSFX=f64", "-DORACLE_REAL_IS_DOUBLE", "-o", str(o64)])
    tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
    subprocess.check_call(["gcc", "-shared", "-fopenmp", "-o", str(tmp), str(o32), str(o64), "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
    return _lib


def _prec(arr: np.ndarray):
    if arr.dtype == np.float32:
        return "f32", ctypes.c_float
    if arr.dtype == np.float64:
        return "f64", ctypes.c_double
    raise TypeError(f"oracle works in float32 or float64, got {arr.dtype}")


def _ptr(a, dtype=None):
    if a is None:
        return None
    if not isinstance(a, np.ndarray) or not a.flags["C_CONTIGUOUS"] or not a.flags["WRITEABLE"]:
        raise TypeError("oracle arguments must be writable C-contiguous numpy arrays")
    if dtype is not None and a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a.ctypes.data_as(ctypes.c_void_p)


def _theta_dtype(theta_kind, real):
    return real if theta_kind == THETA_NATIVE else np.uint16


def outer_step(variant, *, M, P, stride, eta, mu, theta, start, outer_mom,
               delta_prev_local=None, delta_prev_avg=None, master=None,
               theta_kind=THETA_NATIVE, bootstrap=False, nthreads=1,
               comm=COMM_F32, exp_bits=0, man_bits=0, scales_out=None):
    """One outer step of Algorithm 1 (STANDARD), 2 (DELAYED) or 3 (EAGER), in place.

    ``theta`` is float32/float64 [M, stride] for THETA_NATIVE, else uint16 bf16 bit patterns;
    the working precision is taken from ``start``.
    """
    sfx, creal = _prec(start)
    real = start.dtype
    if variant == EAGER and delta_prev_local is None:
        raise ValueError("eager needs delta_prev_local")
    if variant != STANDARD and delta_prev_avg is None:
        raise ValueError("delayed/eager need delta_prev_avg")
    if theta_kind == THETA_MASTER_BF16 and master is None:
        raise ValueError("master copy missing")
    fn = getattr(lib(), f"oracle_outer_step_comm_{sfx}")
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                   creal, creal, ctypes.c_int] + [ctypes.c_void_p] * 6 \
                  + [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_int]
    rc = fn(variant, int(bool(bootstrap)), M, P, stride, eta, mu, theta_kind,
            _ptr(theta, _theta_dtype(theta_kind, real)), _ptr(master, real), _ptr(start, real),
            _ptr(delta_prev_local, real), _ptr(delta_prev_avg, real), _ptr(outer_mom, real),
            int(comm), int(exp_bits), int(man_bits), _ptr(scales_out, real), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_outer_step rejected its arguments")


def outer_step_overlap(variant, k, have, *, delta_prev_local=None, delta_prev_avg=None, **kw):
    """Outer step number ``k`` (0-based) of a run whose all-reduce result arrives D outer steps
    late, D = number of generations in ``delta_prev_avg`` [D, stride] (``delta_prev_local`` is
    [D, M, stride]).  D = 1 is Algorithms 2-3 as printed.  For D = 2 ("two-outer-steps"
    overlap, Section 3) the paper prints no formula; the reading taken is line 11 with t-H
    replaced by t-DH:  g_m = (Delta_m^(t) - Delta_m^(t-DH)) / M + Delta^(t-DH)  (PARITY
    UNPINNED against the paper: there is nothing printed to pin it to).  The generations are
    kept in a ring, slot k mod D; the step reads its slot (recorded at step k-D) and then
    overwrites it.  While fewer than D generations have been recorded (``have`` < D) nothing
    can have arrived yet and the step only records.  Returns the new ``have``.
    """
    D = delta_prev_avg.shape[0]
    slot = k % D
    boot = variant != STANDARD and have < D
    outer_step(variant, bootstrap=boot, delta_prev_avg=delta_prev_avg[slot],
               delta_prev_local=None if delta_prev_local is None else delta_prev_local[slot], **kw)
    return min(D, have + 1) if variant != STANDARD else have


def outer_step_fragment(variant, k, have, offset, length, *, M, theta, start, outer_mom, delta_prev_local=None,
                        delta_prev_avg=None, master=None, **kw):
    """Outer step number ``k`` (0-based, counted per fragment) of the fragment made of indices
    [offset, offset + length) of every replica, as Streaming DiLoCo steps parts of the model on
    their own schedules (Section 3).  Every index is independent, so this is outer_step_overlap on
    the slices: they are copied out, stepped, and copied back; nothing outside the fragment is
    read or written.  ``delta_prev_local`` is [D, M, stride], ``delta_prev_avg`` [D, stride];
    ``have`` counts the fragment's recorded generations.  Returns the fragment's new ``have``."""
    sl = slice(offset, offset + length)
    names = dict(theta=theta, start=start, outer_mom=outer_mom, delta_prev_local=delta_prev_local,
                 delta_prev_avg=delta_prev_avg, master=master)
    part = {n: (None if a is None else np.ascontiguousarray(a[..., sl])) for n, a in names.items()}
    have = outer_step_overlap(variant, k, have, M=M, P=length, stride=length, **part, **kw)
    for n, a in names.items():
        if a is not None:
            a[..., sl] = part[n]
    return have


def eager_gradient(form, *, M, P, stride, theta, start, delta_prev_local, delta_prev_avg=None,
                   master=None, theta_kind=THETA_NATIVE):
    """tilde-Delta_m for all m, without applying it: form 'a' = Alg. 3 line 11, 'b' = the
    equivalent average over the fresh local and the stale non-local gradients."""
    sfx, _ = _prec(start)
    real = start.dtype
    out = np.zeros((M, stride), dtype=real)
    if form == "a":
        fn = getattr(lib(), f"oracle_eager_gradient_form_a_{sfx}")
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int] + [ctypes.c_void_p] * 6
        rc = fn(M, P, stride, theta_kind, _ptr(theta, _theta_dtype(theta_kind, real)), _ptr(master, real),
                _ptr(start, real), _ptr(delta_prev_local, real), _ptr(delta_prev_avg, real), _ptr(out))
    else:
        fn = getattr(lib(), f"oracle_eager_gradient_form_b_{sfx}")
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int] + [ctypes.c_void_p] * 5
        rc = fn(M, P, stride, theta_kind, _ptr(theta, _theta_dtype(theta_kind, real)), _ptr(master, real),
                _ptr(start, real), _ptr(delta_prev_local, real), _ptr(out))
    if rc != 0:
        raise ValueError("oracle_eager_gradient rejected its arguments")
    return out


def inner_adamw(*, M, P, stride, gstride, lr, beta1, beta2, eps, wd, k, theta, grads, adam_m, adam_v,
                master=None, theta_kind=THETA_NATIVE, grad_kind=GRAD_NATIVE, nthreads=1):
    """Inner AdamW step number ``k`` (1-based, never reset) for all M replicas, in place."""
    sfx, creal = _prec(adam_m)
    real = adam_m.dtype
    fn = getattr(lib(), f"oracle_inner_adamw_{sfx}")
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                   creal, creal, creal, creal, creal, ctypes.c_int64, ctypes.c_int, ctypes.c_int] \
                  + [ctypes.c_void_p] * 5 + [ctypes.c_int]
    gd = real if grad_kind == GRAD_NATIVE else np.uint16
    rc = fn(M, P, stride, gstride, lr, beta1, beta2, eps, wd, int(k), theta_kind, grad_kind,
            _ptr(theta, _theta_dtype(theta_kind, real)), _ptr(master, real), _ptr(grads, gd),
            _ptr(adam_m, real), _ptr(adam_v, real), int(nthreads))
    if rc != 0:
        raise ValueError("oracle_inner_adamw rejected its arguments")


def exmy_round(y: float, exp_bits: int, man_bits: int) -> float:
    """Nearest EXMY(exp_bits, man_bits) number (ties to the even code, saturating)."""
    fn = lib().oracle_exmy_round_f64
    fn.restype = ctypes.c_double
    fn.argtypes = [ctypes.c_double, ctypes.c_int, ctypes.c_int]
    return float(fn(y, exp_bits, man_bits))


def exmy_max(exp_bits: int, man_bits: int) -> float:
    fn = lib().oracle_exmy_max_f64
    fn.restype = ctypes.c_double
    fn.argtypes = [ctypes.c_int, ctypes.c_int]
    return float(fn(exp_bits, man_bits))


def wire_encode(d: np.ndarray, exp_bits: int, man_bits: int):
    """One worker's quantised outer gradient as wire bytes: (payload uint8 array, amax)."""
    sfx, creal = _prec(d)
    P = d.shape[0]
    packed = exp_bits + man_bits + 1 <= 4
    payload = np.zeros((P + 1) // 2 if packed else P, dtype=np.uint8)
    amax = np.zeros(1, dtype=d.dtype)
    fn = getattr(lib(), f"oracle_wire_encode_{sfx}")
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    if fn(P, _ptr(np.ascontiguousarray(d)), exp_bits, man_bits, _ptr(payload), _ptr(amax)) != 0:
        raise ValueError("oracle_wire_encode rejected its arguments")
    return payload, amax[0]


def wire_decode_sum(payloads: np.ndarray, amaxes: np.ndarray, P: int, exp_bits: int, man_bits: int) -> np.ndarray:
    """Ordered sum over workers of the dequantised payload rows ([M, row bytes] uint8)."""
    sfx, creal = _prec(amaxes)
    M = payloads.shape[0]
    out = np.zeros(P, dtype=amaxes.dtype)
    fn = getattr(lib(), f"oracle_wire_decode_sum_{sfx}")
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                   ctypes.c_int, ctypes.c_void_p]
    if fn(M, P, payloads.strides[0], _ptr(payloads), _ptr(amaxes), exp_bits, man_bits, _ptr(out)) != 0:
        raise ValueError("oracle_wire_decode_sum rejected its arguments")
    return out


def f32_to_bf16(x: float) -> int:
    fn = lib().oracle_f32_to_bf16_f32
    fn.restype = ctypes.c_uint16
    fn.argtypes = [ctypes.c_float]
    return int(fn(x))


def bf16_to_f32(h: int) -> float:
    fn = lib().oracle_bf16_to_f32_f32
    fn.restype = ctypes.c_float
    fn.argtypes = [ctypes.c_uint16]
    return float(fn(h))
