"""ctypes binding of libdiloco.so: the same names as include/diloco.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; this module converts torch
tensors to device pointers and checks status codes.  There is no fallback: if the shared
library has not been built (``python -m paper_2502_12996_b200.build``) loading raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional

PKG = Path(__file__).resolve().parent
LIB_PATH = PKG / "libdiloco.so"

OK, ERR_INVALID_ARG, ERR_MISALIGNED, ERR_BAD_STATE, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_UNSUPPORTED = 0, -1, -2, -3, -4, -5, -6
THETA_F32, THETA_BF16, THETA_MASTER_BF16 = 0, 1, 2
GRAD_F32, GRAD_BF16 = 0, 1
IMPL_AUTO, IMPL_DIRECT, IMPL_BULK, IMPL_SPLIT_R2, IMPL_SPLIT_R4 = 0, 1, 2, 3, 4
IMPL_TENSOR_T256, IMPL_TENSOR_T128, IMPL_TENSOR_T64 = 5, 6, 7
STANDARD, DELAYED, EAGER = 0, 1, 2
COMM_F32, COMM_BF16, COMM_EXMY = 0, 1, 2
MAX_M = 64
MAX_OVERLAP = 4


class Config(ctypes.Structure):
    """diloco_config_t"""
    _fields_ = [("M", ctypes.c_int32), ("H", ctypes.c_int32), ("P", ctypes.c_int64), ("stride", ctypes.c_int64),
                ("outer_lr", ctypes.c_float), ("outer_momentum", ctypes.c_float),
                ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
                ("weight_decay", ctypes.c_float), ("theta_kind", ctypes.c_int32), ("grad_kind", ctypes.c_int32),
                ("have_prev", ctypes.c_int32), ("impl", ctypes.c_int32), ("overlap_steps", ctypes.c_int32),
                ("shared_outer_state", ctypes.c_int32)]


class Buffers(ctypes.Structure):
    """diloco_buffers_t"""
    _fields_ = [("theta", ctypes.c_void_p), ("master", ctypes.c_void_p), ("start", ctypes.c_void_p),
                ("delta_prev_local", ctypes.c_void_p), ("delta_prev_avg", ctypes.c_void_p),
                ("outer_mom", ctypes.c_void_p), ("adam_m", ctypes.c_void_p), ("adam_v", ctypes.c_void_p),
                ("device_status", ctypes.c_void_p), ("comm_scratch", ctypes.c_void_p)]


class CUInput(ctypes.Structure):
    """diloco_cu_input_t"""
    _fields_ = [("P", ctypes.c_int64), ("bits_per_param", ctypes.c_double), ("M", ctypes.c_int32), ("H", ctypes.c_int32),
                ("step_time_s", ctypes.c_double), ("bandwidth_bit_s", ctypes.c_double),
                ("overlap_outer_steps", ctypes.c_int32), ("overlap_inner_steps", ctypes.c_int32), ("ring", ctypes.c_int32)]


class CUOutput(ctypes.Structure):
    """diloco_cu_output_t"""
    _fields_ = [(n, ctypes.c_double) for n in ("wire_bits", "comm_time_s", "tolerated_latency_s", "exposed_comm_time_s",
                                               "compute_time_s", "compute_utilization")]


class DilocoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = status_string(status)
        if status == ERR_CUDA:
            msg += f" (cudaError {last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


_lib = None

SYMBOLS = {
    "diloco_state_init": (ctypes.c_int, [ctypes.POINTER(Config), ctypes.POINTER(Buffers), ctypes.POINTER(ctypes.c_void_p)]),
    "diloco_state_free": (ctypes.c_int, [ctypes.c_void_p]),
    "diloco_inner_adamw": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p]),
    "diloco_outer_standard": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_outer_delayed": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_outer_eager": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_outer_quantized": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]),
    "diloco_outer_quantized_static": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]),
    "diloco_worker_outer_send": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_worker_outer_apply": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_wire_payload_bytes": (ctypes.c_int64, [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]),
    "diloco_worker_quantized_send": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_worker_quantized_apply": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_outer_fragment": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]),
    "diloco_fragments_set": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]),
    "diloco_outer_fragment_step": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]),
    "diloco_outer_fragment_step_quantized": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]),
    "diloco_fragment_get_counters": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int32)]),
    "diloco_fragment_set_counters": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_int32]),
    "diloco_outer_step_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(Buffers), ctypes.POINTER(ctypes.c_void_p), ctypes.c_int64]),
    "diloco_state_get_counters": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int32)]),
    "diloco_state_set_counters": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int32]),
    "diloco_set_outer_hparams": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_float, ctypes.c_float]),
    "diloco_set_impl": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32]),
    "diloco_set_wait_limit": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32]),
    "diloco_check_device_status": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "diloco_compute_utilization": (ctypes.c_int, [ctypes.POINTER(CUInput), ctypes.POINTER(CUOutput)]),
    "diloco_bandwidth_for_utilization": (ctypes.c_double, [ctypes.POINTER(CUInput), ctypes.c_double]),
    "diloco_launch_count": (ctypes.c_int64, []),
    "diloco_last_cuda_error": (ctypes.c_int32, []),
    "diloco_status_string": (ctypes.c_char_p, [ctypes.c_int]),
}


def load_library() -> ctypes.CDLL:
    """Load libdiloco.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2502_12996_b200.build` "
                               "(there is no CPU fallback)")
        lib = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().diloco_status_string(int(status)).decode()


def last_cuda_error() -> int:
    return int(load_library().diloco_last_cuda_error())


def launch_count() -> int:
    return int(load_library().diloco_launch_count())


def wire_payload_bytes(P: int, exp_bits: int, man_bits: int) -> int:
    n = int(load_library().diloco_wire_payload_bytes(P, exp_bits, man_bits))
    if n < 0:
        raise DilocoError(n, "diloco_wire_payload_bytes")
    return n


def _cu_input(P, bits_per_param, M, H, step_time_s, bandwidth_bit_s, overlap_outer_steps, overlap_inner_steps, ring):
    return CUInput(int(P), float(bits_per_param), int(M), int(H), float(step_time_s), float(bandwidth_bit_s),
                   int(overlap_outer_steps), int(overlap_inner_steps), int(bool(ring)))


def compute_utilization(*, P, bits_per_param, M, H, step_time_s, bandwidth_bit_s, overlap_outer_steps=1,
                        overlap_inner_steps=0, ring=False) -> dict:
    """diloco_compute_utilization: the output struct as a dict."""
    inp = _cu_input(P, bits_per_param, M, H, step_time_s, bandwidth_bit_s, overlap_outer_steps, overlap_inner_steps, ring)
    out = CUOutput()
    _check(load_library().diloco_compute_utilization(ctypes.byref(inp), ctypes.byref(out)), "diloco_compute_utilization")
    return {n: getattr(out, n) for n, _ in CUOutput._fields_}


def bandwidth_for_utilization(target, *, P, bits_per_param, M, H, step_time_s, overlap_outer_steps=1,
                              overlap_inner_steps=0, ring=False) -> float:
    """diloco_bandwidth_for_utilization, bits per second."""
    inp = _cu_input(P, bits_per_param, M, H, step_time_s, 1.0, overlap_outer_steps, overlap_inner_steps, ring)
    w = float(load_library().diloco_bandwidth_for_utilization(ctypes.byref(inp), float(target)))
    if w < 0:
        raise DilocoError(int(w), "diloco_bandwidth_for_utilization")
    return w


def _check(status: int, where: str) -> None:
    if status != OK:
        raise DilocoError(status, where)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream or None
    return int(stream.cuda_stream)


def make_buffers(theta=None, master=None, start=None, delta_prev_local=None, delta_prev_avg=None, outer_mom=None,
                 adam_m=None, adam_v=None, device_status=None, comm_scratch=None) -> Buffers:
    return Buffers(_ptr(theta), _ptr(master), _ptr(start), _ptr(delta_prev_local), _ptr(delta_prev_avg),
                   _ptr(outer_mom), _ptr(adam_m), _ptr(adam_v), _ptr(device_status), _ptr(comm_scratch))


class State:
    """Owns a diloco_state_t handle and keeps the borrowed tensors alive."""

    def __init__(self, *, M, P, stride, theta, start, outer_mom, master=None, delta_prev_local=None,
                 delta_prev_avg=None, adam_m=None, adam_v=None, device_status=None, comm_scratch=None, H=0,
                 outer_lr=0.7,
                 outer_momentum=0.9, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, theta_kind=THETA_F32,
                 grad_kind=GRAD_F32, have_prev=None, impl=IMPL_AUTO, overlap_steps=1, shared_outer_state=False):
        self._handle = ctypes.c_void_p()
        self.tensors = dict(theta=theta, master=master, start=start, delta_prev_local=delta_prev_local,
                            delta_prev_avg=delta_prev_avg, outer_mom=outer_mom, adam_m=adam_m, adam_v=adam_v,
                            device_status=device_status, comm_scratch=comm_scratch)
        have_prev = overlap_steps if have_prev is None else int(have_prev)      # default: every generation seeded
        self.config = Config(M, H, P, stride, outer_lr, outer_momentum, beta1, beta2, eps, weight_decay,
                             theta_kind, grad_kind, have_prev, impl, overlap_steps, int(bool(shared_outer_state)))
        self.buffers = make_buffers(**self.tensors)
        _check(load_library().diloco_state_init(ctypes.byref(self.config), ctypes.byref(self.buffers),
                                                ctypes.byref(self._handle)), "diloco_state_init")

    @classmethod
    def from_dict(cls, st: dict, **kw) -> "State":
        keys = ("theta", "master", "start", "delta_prev_local", "delta_prev_avg", "outer_mom", "adam_m", "adam_v")
        args = {k: st.get(k) for k in keys}
        return cls(M=st["M"], P=st["P"], stride=st["stride"], theta_kind=st["theta_kind"], **args, **kw)

    def close(self) -> None:
        if self._handle:
            load_library().diloco_state_free(self._handle)
            self._handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- the entry points, same names as the C ABI
    def inner_adamw(self, grads, lr, stream=None, grad_stride=None) -> None:
        gs = grads.stride(0) if grad_stride is None else grad_stride
        _check(load_library().diloco_inner_adamw(self._handle, _ptr(grads), gs, lr, _stream_ptr(stream)),
               "diloco_inner_adamw")

    def outer_standard(self, stream=None) -> None:
        _check(load_library().diloco_outer_standard(self._handle, _stream_ptr(stream)), "diloco_outer_standard")

    def outer_delayed(self, stream=None) -> None:
        _check(load_library().diloco_outer_delayed(self._handle, _stream_ptr(stream)), "diloco_outer_delayed")

    def outer_eager(self, stream=None) -> None:
        _check(load_library().diloco_outer_eager(self._handle, _stream_ptr(stream)), "diloco_outer_eager")

    def outer(self, variant: int, stream=None) -> None:
        (self.outer_standard, self.outer_delayed, self.outer_eager)[variant](stream)

    def outer_quantized(self, variant, comm_format, exp_bits=0, man_bits=0, stream=None) -> None:
        _check(load_library().diloco_outer_quantized(self._handle, variant, comm_format, exp_bits, man_bits,
                                                     _stream_ptr(stream)), "diloco_outer_quantized")

    def outer_quantized_static(self, variant, comm_format, exp_bits=0, man_bits=0, stream=None) -> None:
        """diloco_outer_quantized with the scratch inside the library (no comm_scratch needed)."""
        _check(load_library().diloco_outer_quantized_static(self._handle, variant, comm_format, exp_bits, man_bits,
                                                            _stream_ptr(stream)), "diloco_outer_quantized_static")

    def worker_outer_send(self, delta_send, stream=None) -> None:
        _check(load_library().diloco_worker_outer_send(self._handle, _ptr(delta_send), _stream_ptr(stream)),
               "diloco_worker_outer_send")

    def worker_outer_apply(self, variant, world_replicas, delta_sum_recv, delta_send, stream=None) -> None:
        _check(load_library().diloco_worker_outer_apply(self._handle, variant, world_replicas, _ptr(delta_sum_recv),
                                                        _ptr(delta_send), _stream_ptr(stream)),
               "diloco_worker_outer_apply")

    def worker_quantized_send(self, exp_bits, man_bits, payload_send, amax_send, stream=None) -> None:
        _check(load_library().diloco_worker_quantized_send(self._handle, exp_bits, man_bits, _ptr(payload_send),
                                                           _ptr(amax_send), _stream_ptr(stream)),
               "diloco_worker_quantized_send")

    def worker_quantized_apply(self, variant, world_replicas, exp_bits, man_bits, payloads_recv, amaxes_recv,
                               payload_send, amax_send, stream=None) -> None:
        stride = 0 if payloads_recv is None else payloads_recv.stride(0) * payloads_recv.element_size()
        _check(load_library().diloco_worker_quantized_apply(
            self._handle, variant, world_replicas, exp_bits, man_bits, _ptr(payloads_recv), stride, _ptr(amaxes_recv),
            _ptr(payload_send), _ptr(amax_send), _stream_ptr(stream)), "diloco_worker_quantized_apply")

    def outer_fragment(self, variant, bootstrap, offset, length, stream=None) -> None:
        _check(load_library().diloco_outer_fragment(self._handle, variant, int(bool(bootstrap)), offset, length,
                                                    _stream_ptr(stream)), "diloco_outer_fragment")

    def fragments_set(self, offsets, lens) -> None:
        n = len(offsets)
        a, b = (ctypes.c_int64 * max(n, 1))(*offsets), (ctypes.c_int64 * max(n, 1))(*lens)
        _check(load_library().diloco_fragments_set(self._handle, n, a, b), "diloco_fragments_set")

    def outer_fragment_step(self, variant, fragment_id, stream=None) -> None:
        _check(load_library().diloco_outer_fragment_step(self._handle, variant, fragment_id, _stream_ptr(stream)),
               "diloco_outer_fragment_step")

    def outer_fragment_step_quantized(self, variant, fragment_id, comm_format, exp_bits=0, man_bits=0, stream=None) -> None:
        _check(load_library().diloco_outer_fragment_step_quantized(self._handle, variant, fragment_id, comm_format, exp_bits,
                                                                   man_bits, _stream_ptr(stream)),
               "diloco_outer_fragment_step_quantized")

    def fragment_get_counters(self, fragment_id):
        a, b = ctypes.c_int64(), ctypes.c_int32()
        _check(load_library().diloco_fragment_get_counters(self._handle, fragment_id, ctypes.byref(a), ctypes.byref(b)),
               "diloco_fragment_get_counters")
        return a.value, b.value

    def fragment_set_counters(self, fragment_id, outer_step, have_prev) -> None:
        _check(load_library().diloco_fragment_set_counters(self._handle, fragment_id, outer_step, int(have_prev)),
               "diloco_fragment_set_counters")

    def outer_step_host(self, variant, host: Buffers, streams, chunk) -> None:
        arr = (ctypes.c_void_p * 3)(*[int(s.cuda_stream) for s in streams])
        _check(load_library().diloco_outer_step_host(self._handle, variant, ctypes.byref(host), arr, chunk),
               "diloco_outer_step_host")

    def get_counters(self):
        a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int32()
        _check(load_library().diloco_state_get_counters(self._handle, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
               "diloco_state_get_counters")
        return a.value, b.value, c.value

    def set_counters(self, inner_step, outer_step, have_prev) -> None:
        _check(load_library().diloco_state_set_counters(self._handle, inner_step, outer_step, int(have_prev)),
               "diloco_state_set_counters")

    def set_outer_hparams(self, outer_lr, outer_momentum) -> None:
        _check(load_library().diloco_set_outer_hparams(self._handle, outer_lr, outer_momentum), "diloco_set_outer_hparams")

    def set_impl(self, impl) -> None:
        _check(load_library().diloco_set_impl(self._handle, impl), "diloco_set_impl")

    def set_wait_limit(self, limit_ns, test_extra_expect_bytes=0) -> None:
        _check(load_library().diloco_set_wait_limit(self._handle, limit_ns, test_extra_expect_bytes), "diloco_set_wait_limit")

    def check_device_status(self, stream=None) -> None:
        _check(load_library().diloco_check_device_status(self._handle, _stream_ptr(stream)), "diloco_check_device_status")
