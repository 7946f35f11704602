"""Thin ctypes binding of libdarkattn.so (argument marshalling only; all compute is in the library).

Function names mirror the C ABI declared in ``include/darkattn.h``. Tensors are torch CUDA tensors
used purely as device-memory handles; streams are torch CUDA streams. There is no fallback: if the
shared library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdarkattn.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE = range(7)
F32, BF16 = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2

EXPORTS = [
    "darkattn_plan", "darkattn_workspace_bytes", "darkattn_saved_bytes", "darkattn_plan_path",
    "darkattn_forward", "darkattn_backward", "darkattn_last_device_status",
    "darkattn_destroy", "darkattn_status_string", "darkattn_last_cuda_error", "darkattn_measure_alu_peak",
    "darkattn_static_scratch_needed", "darkattn_forward_static",
    "darkattn_backward_dw", "darkattn_decode_step", "darkattn_selftest_wait_limit",
]
# instruments of the benchmark, in a library of their own (include/darkattn_bench.h)
BENCH_EXPORTS = ["darkattn_plan_launches", "darkattn_kernel_timing", "darkattn_kernel_times", "darkattn_measure_mma_cycles"]
STATIC_SCRATCH_BYTES = 16 << 20


class Desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("d", ctypes.c_int32),
                ("r", ctypes.c_int32), ("m", ctypes.c_int32), ("dv", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("causal", ctypes.c_int32), ("chunk", ctypes.c_int32), ("scale", ctypes.c_float),
                ("w_per_head", ctypes.c_int32), ("path", ctypes.c_int32), ("H_kv", ctypes.c_int32)]


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_04127_b200.build` "
                      "(or __graft_entry__.build()); there is no fallback path")

lib = ctypes.CDLL(LIB_PATH)
_vp = ctypes.c_void_p
lib.darkattn_plan.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(_vp)]
lib.darkattn_plan.restype = ctypes.c_int
lib.darkattn_workspace_bytes.argtypes = [_vp]
lib.darkattn_workspace_bytes.restype = ctypes.c_size_t
lib.darkattn_saved_bytes.argtypes = [_vp]
lib.darkattn_saved_bytes.restype = ctypes.c_size_t
lib.darkattn_plan_path.argtypes = [_vp]
lib.darkattn_plan_path.restype = ctypes.c_int32
lib.darkattn_forward.argtypes = [_vp] * 10
lib.darkattn_forward.restype = ctypes.c_int
lib.darkattn_backward.argtypes = [_vp] * 15
lib.darkattn_backward.restype = ctypes.c_int
lib.darkattn_backward_dw.argtypes = [_vp] * 5
lib.darkattn_backward_dw.restype = ctypes.c_int
lib.darkattn_decode_step.argtypes = [_vp] * 10
lib.darkattn_decode_step.restype = ctypes.c_int
lib.darkattn_last_device_status.argtypes = [_vp, _vp, _vp]
lib.darkattn_last_device_status.restype = ctypes.c_int
lib.darkattn_destroy.argtypes = [_vp]
lib.darkattn_destroy.restype = None
lib.darkattn_status_string.argtypes = [ctypes.c_int]
lib.darkattn_status_string.restype = ctypes.c_char_p
lib.darkattn_last_cuda_error.argtypes = []
lib.darkattn_last_cuda_error.restype = ctypes.c_char_p
lib.darkattn_measure_alu_peak.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_double), _vp]
lib.darkattn_measure_alu_peak.restype = ctypes.c_int
lib.darkattn_selftest_wait_limit.argtypes = [ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double), _vp]
lib.darkattn_selftest_wait_limit.restype = ctypes.c_int
lib.darkattn_static_scratch_needed.argtypes = [_vp]
lib.darkattn_static_scratch_needed.restype = ctypes.c_size_t
lib.darkattn_forward_static.argtypes = [_vp] * 8
lib.darkattn_forward_static.restype = ctypes.c_int


BENCH_LIB_PATH = os.path.join(_HERE, "libdarkattn_bench.so")
_benchlib = None


def benchlib():
    """The instruments' library (loaded on first use; the product calls above never need it)."""
    global _benchlib
    if _benchlib is None:
        if not os.path.exists(BENCH_LIB_PATH):
            raise ImportError(f"{BENCH_LIB_PATH} is missing: build it with `python -m paper_2603_04127_b200.build`")
        b = ctypes.CDLL(BENCH_LIB_PATH)
        b.darkattn_plan_launches.argtypes = [_vp, ctypes.c_int32]
        b.darkattn_plan_launches.restype = ctypes.c_int32
        b.darkattn_measure_mma_cycles.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_double),
                                                  ctypes.POINTER(ctypes.c_double), _vp]
        b.darkattn_measure_mma_cycles.restype = ctypes.c_int
        b.darkattn_kernel_timing.argtypes = [_vp, ctypes.c_int32]
        b.darkattn_kernel_timing.restype = ctypes.c_int
        b.darkattn_kernel_times.argtypes = [_vp, ctypes.c_int32, ctypes.c_char_p, ctypes.POINTER(ctypes.c_float),
                                            ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
        b.darkattn_kernel_times.restype = ctypes.c_int
        _benchlib = b
    return _benchlib


class DarkAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.darkattn_status_string(status).decode()
        if status == ERR_CUDA:
            msg += ": " + lib.darkattn_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (status {status})")


def _check(status: int, where: str):
    if status != OK:
        raise DarkAttnError(status, where)


@dataclass
class Plan:
    """Owner of a darkattn_plan_t handle."""
    handle: int
    desc: Desc

    @property
    def workspace_bytes(self) -> int:
        return int(lib.darkattn_workspace_bytes(self.handle))

    @property
    def saved_bytes(self) -> int:
        return int(lib.darkattn_saved_bytes(self.handle))

    @property
    def path(self) -> int:
        return int(lib.darkattn_plan_path(self.handle))

    def launches(self, backward: bool = False) -> int:
        return int(benchlib().darkattn_plan_launches(self.handle, 1 if backward else 0))

    def alloc_workspace(self, device="cuda") -> torch.Tensor:
        return torch.empty(max(self.workspace_bytes, 256), dtype=torch.uint8, device=device)

    def destroy(self):
        if self.handle:
            lib.darkattn_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def darkattn_plan(B, H, N, d, m, *, r=0, dv=0, dtype=BF16, causal=False, chunk=0, scale=0.0, w_per_head=False,
                  path=PATH_AUTO, H_kv=0) -> Plan:
    desc = Desc(B, H, N, d, r, m, dv, dtype, int(bool(causal)), chunk, float(scale), int(bool(w_per_head)), path, H_kv)
    h = _vp()
    _check(lib.darkattn_plan(ctypes.byref(desc), ctypes.byref(h)), "darkattn_plan")
    return Plan(h.value, desc)


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def darkattn_forward(plan: Plan, Q, K, V, M, W, O, workspace, saved=None, stream=None):
    _check(lib.darkattn_forward(plan.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(M), _ptr(W), _ptr(O), _ptr(saved),
                                _ptr(workspace), _stream(stream)), "darkattn_forward")
    return O


def darkattn_backward(plan: Plan, Q, K, V, M, W, O, dO, dQ, dK, dV, dM, workspace, saved=None, stream=None):
    assert dM.dtype == torch.float32
    _check(lib.darkattn_backward(plan.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(M), _ptr(W), _ptr(O), _ptr(dO),
                                 _ptr(saved), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dM), _ptr(workspace),
                                 _stream(stream)), "darkattn_backward")
    return dQ, dK, dV, dM


def darkattn_backward_dw(plan: Plan, M, dW, workspace, stream=None):
    """Gradient of the projection rows W, from what the preceding darkattn_backward left in ``workspace``."""
    assert dW.dtype == torch.float32
    _check(lib.darkattn_backward_dw(plan.handle, _ptr(M), _ptr(dW), _ptr(workspace), _stream(stream)),
           "darkattn_backward_dw")
    return dW


def darkattn_decode_step(plan: Plan, q, k, v, M, W, S, z, o, stream=None):
    """One recurrent step: S, z (float32, caller-owned running state) are updated in place, o receives the output."""
    assert S.dtype == torch.float32 and z.dtype == torch.float32
    _check(lib.darkattn_decode_step(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(M), _ptr(W), _ptr(S), _ptr(z), _ptr(o),
                                    _stream(stream)), "darkattn_decode_step")
    return o


def darkattn_last_device_status(plan: Plan, workspace, stream=None) -> int:
    return int(lib.darkattn_last_device_status(plan.handle, _ptr(workspace), _stream(stream)))


def darkattn_measure_alu_peak(which: int, iters: int = 20, stream=None) -> float:
    out = ctypes.c_double(0.0)
    _check(lib.darkattn_measure_alu_peak(which, iters, ctypes.byref(out), _stream(stream)),
           "darkattn_measure_alu_peak")
    return out.value


def darkattn_measure_mma_cycles(variant: int, busy_epilogue: bool = False, stream=None):
    """(cycles per MMA, fixed cycles per batch) of one tcgen05.mma form; see the header for the variants."""
    per, fixed = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(benchlib().darkattn_measure_mma_cycles(variant, int(bool(busy_epilogue)), ctypes.byref(per), ctypes.byref(fixed),
                                           _stream(stream)), "darkattn_measure_mma_cycles")
    return per.value, fixed.value


def darkattn_selftest_wait_limit(stream=None):
    """(device status word, kernel seconds) of a wait on a barrier nobody arrives on."""
    st, sec = ctypes.c_int32(0), ctypes.c_double(0.0)
    _check(lib.darkattn_selftest_wait_limit(ctypes.byref(st), ctypes.byref(sec), _stream(stream)), "darkattn_selftest_wait_limit")
    return st.value, sec.value


def darkattn_kernel_timing(plan: Plan, enable: bool):
    _check(benchlib().darkattn_kernel_timing(plan.handle, int(bool(enable))), "darkattn_kernel_timing")


def darkattn_kernel_times(plan: Plan, max_entries: int = 32) -> dict:
    """{kernel name: (total milliseconds, launches)} since timing was enabled."""
    names = ctypes.create_string_buffer(64 * max_entries)
    ms = (ctypes.c_float * max_entries)()
    cnt = (ctypes.c_int32 * max_entries)()
    n = ctypes.c_int32(0)
    _check(benchlib().darkattn_kernel_times(plan.handle, max_entries, names, ms, cnt, ctypes.byref(n)), "darkattn_kernel_times")
    out = {}
    for i in range(n.value):
        out[names.raw[64 * i:64 * (i + 1)].split(b"\0", 1)[0].decode()] = (float(ms[i]), int(cnt[i]))
    return out


def darkattn_static_scratch_needed(plan: Plan) -> int:
    return int(lib.darkattn_static_scratch_needed(plan.handle))


def darkattn_forward_static(plan: Plan, Q, K, V, M, W, O, stream=None):
    """Forward pass on the library's built-in scratch array: for callers that cannot allocate device
    memory. Calls on one device must not overlap; problems that need more than STATIC_SCRATCH_BYTES
    raise with status ERR_WORKSPACE."""
    _check(lib.darkattn_forward_static(plan.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(M), _ptr(W), _ptr(O),
                                       _stream(stream)), "darkattn_forward_static")
    return O
