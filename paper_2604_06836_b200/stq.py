"""Thin ctypes binding over libstq (the C-ABI declared in ``include/stq.h``).

Argument marshalling only: torch tensors supply device memory and streams, every step of the path
runs in the library's CUDA kernels.  There is no fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstq.so")

GRAD_F32, GRAD_BF16, GRAD_F16 = 0, 1, 2
LP_NONE, LP_BF16, LP_F16 = 0, 1, 2
WITH_STATS = 1
TILE = 4096              # STQ_TILE_ELEMS: elements per tile of the step kernels
VLOG_POLY, VLOG_PL, VLOG_SR, VLOG_TS = 0, 1, 2, 3      # codes of the second moment (stq_tensor.v_log)
VLOG_BY_NAME = {"poly": VLOG_POLY, "pl": VLOG_PL, "sr": VLOG_SR, "ts": VLOG_TS}
WIDTHS = (2, 3, 4, 8, 16, 32)
E_STATE, E_TIMEOUT, E_TOO_LARGE = -10, -11, -12     # the STQ_E_* codes callers test for


class StqError(RuntimeError):
    def __init__(self, code: int, what: str, detail: str = ""):
        super().__init__(f"{what}: error {code} ({_strerror(code)}){' - ' + detail if detail else ''}")
        self.code = code


class CTensor(C.Structure):
    """struct stq_tensor"""
    _fields_ = [
        ("param", C.c_void_p), ("grad", C.c_void_p),
        ("m_codes_in", C.c_void_p), ("m_scales_in", C.c_void_p),
        ("v_codes_in", C.c_void_p), ("v_scales_in", C.c_void_p),
        ("m_codes_out", C.c_void_p), ("m_scales_out", C.c_void_p),
        ("v_codes_out", C.c_void_p), ("v_scales_out", C.c_void_p),
        ("numel", C.c_uint64), ("block", C.c_uint32),
        ("bits_m", C.c_uint8), ("bits_v", C.c_uint8), ("bits_m_out", C.c_uint8), ("bits_v_out", C.c_uint8),
        ("weight_decay", C.c_float), ("lp_dtype", C.c_uint32),
        ("param_lp", C.c_void_p),
        ("v_log", C.c_uint32), ("sr_id", C.c_uint32),
    ]


class CHParams(C.Structure):
    """struct stq_hparams"""
    _fields_ = [("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("step", C.c_int64), ("decoupled_wd", C.c_int32), ("grad_dtype", C.c_int32),
                ("inv_grad_scale", C.c_void_p), ("found_inf", C.c_void_p),
                ("step_dev", C.c_void_p), ("lr_dev", C.c_void_p), ("sr_seed", C.c_uint64)]


class CPolicyCfg(C.Structure):
    """struct stq_policy_cfg"""
    _fields_ = [("alpha", C.c_double), ("tau", C.c_double), ("eps_stat", C.c_double),
                ("interval", C.c_int64), ("cv_of_signed", C.c_int32), ("reserved", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Loads libstq.so; raises if it has not been built (``python -m paper_2604_06836_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_06836_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, PT = C.c_void_p, C.POINTER(CTensor)
        L.stq_create.argtypes = [C.POINTER(vp), C.c_int]
        L.stq_destroy.argtypes = [vp]
        L.stq_codes_bytes.argtypes = [C.c_uint64, C.c_int]
        L.stq_codes_bytes.restype = C.c_size_t
        L.stq_scales_bytes.argtypes = [C.c_uint64, C.c_uint32]
        L.stq_scales_bytes.restype = C.c_size_t
        L.stq_v_scales_bytes.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32]
        L.stq_v_scales_bytes.restype = C.c_size_t
        L.stq_init_state.argtypes = [vp, PT, C.c_int, vp]
        L.stq_step.argtypes = [vp, PT, C.c_int, C.POINTER(CHParams), C.c_uint, vp]
        L.stq_grad_stats.argtypes = [vp, PT, C.c_int, C.c_int, vp]
        L.stq_layer_stats.argtypes = [vp, vp, C.c_int, vp]
        L.stq_repack.argtypes = [vp, PT, C.c_int, vp]
        L.stq_step_host.argtypes = [vp, PT, C.c_int, C.POINTER(CHParams), C.c_uint,
                                    C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.stq_device_status.argtypes = [vp, vp]
        L.stq_selftest_wait_timeout.argtypes = [vp, vp]
        L.stq_grad_stats_static.argtypes = [C.c_int, vp, C.c_uint64, C.c_int, vp, vp]
        L.stq_launch_count.argtypes = [vp]
        L.stq_launch_count.restype = C.c_uint64
        L.stq_grid_size.argtypes = [vp]
        L.stq_sm_count.argtypes = [vp]
        L.stq_policy_create.argtypes = [C.POINTER(vp), C.POINTER(CPolicyCfg)]
        L.stq_policy_destroy.argtypes = [vp]
        L.stq_policy_is_decision_step.argtypes = [vp, C.c_int64]
        L.stq_decide.argtypes = [vp, vp, C.c_int, C.c_int64, vp, vp]
        L.stq_policy_get_state.argtypes = [vp, vp]
        L.stq_policy_set_state.argtypes = [vp, vp]
        L.stq_strerror.argtypes = [C.c_int]
        L.stq_strerror.restype = C.c_char_p
        L.stq_last_cuda_error.argtypes = [vp]
        L.stq_last_cuda_error.restype = C.c_char_p
        _lib = L
    return _lib


def _strerror(code: int) -> str:
    try:
        return lib().stq_strerror(code).decode()
    except Exception:   # pragma: no cover
        return "?"


def codes_bytes(numel: int, bits: int) -> int:
    return int(lib().stq_codes_bytes(numel, bits))


def scales_bytes(numel: int, block: int) -> int:
    return int(lib().stq_scales_bytes(numel, block))


# ------------------------------------------------------------------------------------------------
# per-tensor buffers (torch owns the memory)
# ------------------------------------------------------------------------------------------------
@dataclass
class QState:
    """Stored optimizer state of one tensor: packed codes + block scales for m and v."""
    m_codes: torch.Tensor   # uint8[codes_bytes]
    m_scales: torch.Tensor  # float32[nblocks] (empty at width 32)
    bits_m: int
    v_codes: torch.Tensor
    v_scales: torch.Tensor
    bits_v: int
    v_log: int = 0          # VLOG_POLY | VLOG_PL: how v is coded at widths 8 and 16


def alloc_codes(numel: int, bits: int, device) -> torch.Tensor:
    return torch.zeros(codes_bytes(numel, bits), dtype=torch.uint8, device=device)


def alloc_scales(numel: int, bits: int, block: int, device, v_log: int | None = None) -> torch.Tensor:
    """Scale buffer of a state; v_log (for a second moment) selects the size of its code: the two-scale code
    keeps two floats per block."""
    n = (scales_bytes(numel, block) if v_log is None else int(lib().stq_v_scales_bytes(numel, block, v_log))) // 4
    return torch.zeros(n, dtype=torch.float32, device=device)


def alloc_state(numel: int, block: int, bits_m: int, bits_v: int, device, v_log: int = 0) -> QState:
    return QState(alloc_codes(numel, bits_m, device), alloc_scales(numel, bits_m, block, device), bits_m,
                  alloc_codes(numel, bits_v, device), alloc_scales(numel, bits_v, block, device, v_log), bits_v, v_log)


def _ptr(t: torch.Tensor | None) -> int | None:
    return None if t is None or t.numel() == 0 else t.data_ptr()


def grad_dtype_of(t: torch.Tensor) -> int:
    return {torch.float32: GRAD_F32, torch.bfloat16: GRAD_BF16, torch.float16: GRAD_F16}[t.dtype]


def make_row(numel: int, block: int, st_in: QState | None, st_out: QState, param: torch.Tensor | None = None,
             grad: torch.Tensor | None = None, weight_decay: float = 0.0,
             param_lp: torch.Tensor | None = None, sr_id: int = 0) -> CTensor:
    """One table row.  st_out may be st_in (in-place) when the widths are unchanged.  param_lp: an
    optional bf16/fp16 tensor that receives the rounded copy of the updated parameters.  sr_id: the
    tensor's number in the random stream of the stochastic-rounding code (ignored by the other codes)."""
    r = CTensor()
    r.param = _ptr(param)
    r.grad = _ptr(grad)
    if st_in is not None:
        r.m_codes_in, r.m_scales_in = _ptr(st_in.m_codes), _ptr(st_in.m_scales)
        r.v_codes_in, r.v_scales_in = _ptr(st_in.v_codes), _ptr(st_in.v_scales)
        r.bits_m, r.bits_v = st_in.bits_m, st_in.bits_v
    else:
        r.bits_m, r.bits_v = st_out.bits_m, st_out.bits_v
    r.m_codes_out, r.m_scales_out = _ptr(st_out.m_codes), _ptr(st_out.m_scales)
    r.v_codes_out, r.v_scales_out = _ptr(st_out.v_codes), _ptr(st_out.v_scales)
    r.bits_m_out, r.bits_v_out = st_out.bits_m, st_out.bits_v
    if st_in is not None and st_in.v_log != st_out.v_log:
        raise ValueError("a state is read and written with the same variant of the v quantizer")
    r.v_log, r.sr_id = st_out.v_log, (sr_id if st_out.v_log == VLOG_SR else 0)
    r.numel, r.block, r.weight_decay = numel, block, weight_decay
    if param_lp is not None:
        r.lp_dtype = LP_BF16 if param_lp.dtype == torch.bfloat16 else LP_F16
        r.param_lp = param_lp.data_ptr()
    else:
        r.lp_dtype, r.param_lp = LP_NONE, None
    return r


def table(rows: Sequence[CTensor]):
    return (CTensor * len(rows))(*rows)


def _stream_ptr(stream) -> int | None:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


STATIC_STATS_MAX_NUMEL = 64 * 1024 * 1024


def check_static_stats_args(grad: torch.Tensor, out: torch.Tensor) -> None:
    """The C entry point sees only pointers and a count: what it cannot check is checked here, before
    anything is launched.  A gradient of another type would be read as numel fp32 values (twice the
    length of an fp16 buffer), a strided one as if it were dense."""
    if grad.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError(f"grad_stats_static takes float32 or bfloat16 gradients, not {grad.dtype}")
    if not grad.is_contiguous():
        raise ValueError("grad_stats_static needs a contiguous gradient")
    if out.dtype != torch.float64 or out.numel() < 4 or not out.is_contiguous():
        raise ValueError("out is a contiguous float64 tensor of at least 4 elements")
    if grad.device.type != "cuda" or out.device != grad.device:
        raise ValueError("grad and out live on the same CUDA device")


def grad_stats_static(grad: torch.Tensor, out: torch.Tensor, stream=None) -> int:
    """Gradient sums of one tensor through the entry point that allocates nothing.

    For callers that cannot let a library allocate device memory (all free memory already belongs
    to the framework's caching allocator, or a fixed budget is in force): the scratch space is a
    static array inside libstq.  ``out`` is a caller-owned float64[4] tensor on the same device; the
    call is asynchronous on the stream.  Returns the C status code (0 = ok) instead of raising, so
    that callers can test for STQ_E_TOO_LARGE (-12) and fall back to splitting the tensor."""
    check_static_stats_args(grad, out)
    dt = GRAD_BF16 if grad.dtype == torch.bfloat16 else GRAD_F32
    return int(lib().stq_grad_stats_static(grad.device.index if grad.device.index is not None else
                                           torch.cuda.current_device(), grad.data_ptr(), grad.numel(), dt,
                                           out.data_ptr(), _stream_ptr(stream)))


class Handle:
    """Owns one stq_handle (device table, tile map, statistics workspace)."""

    def __init__(self, device: int | None = None):
        if device is None:
            device = torch.cuda.current_device()
        self.device = int(device)
        self._h = C.c_void_p()
        rc = lib().stq_create(C.byref(self._h), self.device)
        if rc != 0:
            raise StqError(rc, "stq_create")

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            lib().stq_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):   # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, what: str):
        if rc != 0:
            raise StqError(rc, what, lib().stq_last_cuda_error(self._h).decode())

    def init_state(self, tbl, stream=None):
        self._check(lib().stq_init_state(self._h, tbl, len(tbl), _stream_ptr(stream)), "stq_init_state")

    def step(self, tbl, *, lr, beta1, beta2, eps, t, grad_dtype=GRAD_F32, decoupled_wd=True, flags=0, stream=None,
             inv_grad_scale: torch.Tensor | None = None, found_inf: torch.Tensor | None = None,
             step_dev: torch.Tensor | None = None, lr_dev: torch.Tensor | None = None, sr_seed: int = 0):
        """inv_grad_scale / found_inf: optional one-element float32 device tensors (loss-scaled training).
        sr_seed: seed of the random words of tensors coded with stochastic rounding.
        step_dev (one int64) / lr_dev (one float32): optional device tensors that replace t and lr, for steps
        replayed from a CUDA graph."""
        if step_dev is not None and step_dev.dtype != torch.int64:
            raise ValueError("step_dev holds one int64")
        if lr_dev is not None and lr_dev.dtype != torch.float32:
            raise ValueError("lr_dev holds one float32")
        hp = CHParams(lr, beta1, beta2, eps, t, 1 if decoupled_wd else 0, grad_dtype,
                      _ptr(inv_grad_scale), _ptr(found_inf), _ptr(step_dev), _ptr(lr_dev), sr_seed)
        self._check(lib().stq_step(self._h, tbl, len(tbl), C.byref(hp), flags, _stream_ptr(stream)), "stq_step")

    def grad_stats(self, tbl, grad_dtype=GRAD_F32, stream=None):
        self._check(lib().stq_grad_stats(self._h, tbl, len(tbl), grad_dtype, _stream_ptr(stream)), "stq_grad_stats")

    def layer_stats(self, L: int, stream=None) -> np.ndarray:
        out = np.zeros((L, 4), dtype=np.float64)
        self._check(lib().stq_layer_stats(self._h, out.ctypes.data_as(C.c_void_p), L, _stream_ptr(stream)),
                    "stq_layer_stats")
        return out

    def repack(self, tbl, stream=None):
        self._check(lib().stq_repack(self._h, tbl, len(tbl), _stream_ptr(stream)), "stq_repack")

    def step_host(self, tbl, *, lr, beta1, beta2, eps, t, grad_dtype=GRAD_F32, decoupled_wd=True, flags=0,
                  inv_grad_scale=None, found_inf=None, sr_seed: int = 0):
        if inv_grad_scale is not None or found_inf is not None:
            raise ValueError("step_host takes host buffers only: unscale the gradients on the device path")
        hp = CHParams(lr, beta1, beta2, eps, t, 1 if decoupled_wd else 0, grad_dtype, None, None, None, None, sr_seed)
        h2d, d2h = C.c_uint64(0), C.c_uint64(0)
        self._check(lib().stq_step_host(self._h, tbl, len(tbl), C.byref(hp), flags, C.byref(h2d), C.byref(d2h)),
                    "stq_step_host")
        return int(h2d.value), int(d2h.value)

    def device_status(self, stream=None):
        """Synchronises the stream; raises if a kernel gave up on a bounded wait."""
        self._check(lib().stq_device_status(self._h, _stream_ptr(stream)), "stq_device_status")

    def selftest_wait_timeout(self, stream=None):
        """Runs the bounded-wait self-test; afterwards device_status() raises with code -11."""
        self._check(lib().stq_selftest_wait_timeout(self._h, _stream_ptr(stream)), "stq_selftest_wait_timeout")

    @property
    def launch_count(self) -> int:
        return int(lib().stq_launch_count(self._h))

    @property
    def grid_size(self) -> int:
        return int(lib().stq_grid_size(self._h))

    @property
    def sm_count(self) -> int:
        return int(lib().stq_sm_count(self._h))


class Policy:
    """Host-side transition decision (stq_policy)."""

    def __init__(self, alpha=0.1, tau=100.0, eps_stat=1e-8, interval=10, cv_of_signed=False):
        cfg = CPolicyCfg(alpha, tau, eps_stat, interval, 1 if cv_of_signed else 0, 0)
        self._p = C.c_void_p()
        rc = lib().stq_policy_create(C.byref(self._p), C.byref(cfg))
        if rc != 0:
            raise StqError(rc, "stq_policy_create")

    def close(self):
        if getattr(self, "_p", None) and self._p.value:
            lib().stq_policy_destroy(self._p)
            self._p = C.c_void_p()

    def __del__(self):   # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def is_decision_step(self, t: int) -> bool:
        return bool(lib().stq_policy_is_decision_step(self._p, t))

    def decide(self, stats: np.ndarray, t: int):
        stats = np.ascontiguousarray(stats, dtype=np.float64)
        L = stats.shape[0]
        bits = np.zeros(L, dtype=np.uint8)
        score = np.zeros(L, dtype=np.float64)
        rc = lib().stq_decide(self._p, stats.ctypes.data_as(C.c_void_p), L, t,
                              bits.ctypes.data_as(C.c_void_p), score.ctypes.data_as(C.c_void_p))
        if rc != 0:
            raise StqError(rc, "stq_decide")
        return bits, score

    @property
    def state(self) -> np.ndarray:
        out = np.zeros(3, dtype=np.float64)
        lib().stq_policy_get_state(self._p, out.ctypes.data_as(C.c_void_p))
        return out

    @state.setter
    def state(self, v):
        v = np.ascontiguousarray(v, dtype=np.float64)
        lib().stq_policy_set_state(self._p, v.ctypes.data_as(C.c_void_p))
