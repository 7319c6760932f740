"""ctypes access to the CPU oracle (``stq_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  The product package never imports
this module and shares nothing with it.  Arguments are numpy arrays; nothing here touches CUDA.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stq_oracle.cpp")
_LIB = os.path.join(_HERE, "libstq_oracle.so")

# -ffp-contract=off: every fp32 operation in the source is one rounded operation.
CXXFLAGS = ["-O2", "-std=c++17", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math"]


def build(force: bool = False) -> str:
    """Compile the oracle with g++ if the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", *CXXFLAGS, "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class HParams(C.Structure):
    _fields_ = [("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("weight_decay", C.c_double), ("step", C.c_int64), ("decoupled_wd", C.c_int),
                ("grad_dtype", C.c_int), ("inv_grad_scale", C.c_float), ("found_inf", C.c_int),
                ("v_mode", C.c_int), ("sr_seed", C.c_uint64), ("tensor_index", C.c_uint32),
                ("elem_offset", C.c_uint64)]


class Policy(C.Structure):
    _fields_ = [("n_ema", C.c_double), ("r_ema", C.c_double), ("v_ema", C.c_double),
                ("alpha", C.c_double), ("tau", C.c_double), ("eps_stat", C.c_double),
                ("cv_of_signed", C.c_int)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        # STQ_ORACLE_LIB: the pin suite can be pointed at another build of the oracle source (the mutation
        # check in tests/ runs it against deliberately broken copies to see that the pins notice)
        L = C.CDLL(os.environ.get("STQ_ORACLE_LIB") or build())
        L.orc_codes_bytes.restype = C.c_uint64
        L.orc_codes_bytes.argtypes = [C.c_uint64, C.c_int]
        L.orc_num_blocks.restype = C.c_uint64
        L.orc_num_blocks.argtypes = [C.c_uint64, C.c_uint32]
        L.orc_num_scales.restype = C.c_uint64
        L.orc_num_scales.argtypes = [C.c_uint64, C.c_uint32, C.c_int]
        L.orc_mix32.restype = C.c_uint32
        L.orc_mix32.argtypes = [C.c_uint32]
        L.orc_sr_key.restype = C.c_uint32
        L.orc_sr_key.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32]
        L.orc_sr_word.restype = C.c_uint32
        L.orc_sr_word.argtypes = [C.c_uint32, C.c_uint64]
        L.orc_sr_code.restype = C.c_uint32
        L.orc_sr_code.argtypes = [C.c_float, C.c_float, C.c_int, C.c_uint32]
        L.orc_sr_level.restype = C.c_float
        L.orc_sr_level.argtypes = [C.c_uint32, C.c_int]
        L.orc_sr_enumerate.restype = None
        L.orc_sr_enumerate.argtypes = [C.c_float, C.c_float, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_quantize_keyed.argtypes = [C.c_void_p, C.c_uint64, C.c_int, C.c_uint32, C.c_int, C.c_uint32,
                                         C.c_void_p, C.c_void_p]
        L.orc_lg_P.restype = C.c_float
        L.orc_lg_P.argtypes = [C.c_float]
        L.orc_lg_E.restype = C.c_int
        L.orc_lg_E.argtypes = [C.c_float]
        L.orc_ex2.restype = C.c_float
        L.orc_ex2.argtypes = [C.c_float]
        vp = C.c_void_p
        L.orc_pack.argtypes = [vp, C.c_uint64, C.c_int, vp]
        L.orc_unpack.argtypes = [vp, C.c_uint64, C.c_int, vp]
        L.orc_quantize.argtypes = [vp, C.c_uint64, C.c_int, C.c_uint32, C.c_int, vp, vp]
        L.orc_dequantize.argtypes = [vp, vp, C.c_uint64, C.c_int, C.c_uint32, C.c_int, vp]
        L.orc_init_state.argtypes = [C.c_uint64, C.c_uint32, C.c_int, C.c_int, vp, vp, vp, vp]
        L.orc_grad_stats.argtypes = [vp, C.c_int, C.c_uint64, vp]
        L.orc_grad_stats.restype = None
        L.orc_step.argtypes = [vp, vp, C.c_uint64, C.c_uint32,
                               vp, vp, C.c_int, vp, vp, C.c_int,
                               vp, vp, C.c_int, vp, vp, C.c_int,
                               C.POINTER(HParams), vp]
        L.orc_repack.argtypes = [vp, vp, C.c_int, vp, vp, C.c_int, C.c_uint64, C.c_uint32, C.c_int]
        L.orc_round_lp.argtypes = [vp, C.c_uint64, C.c_int, vp]
        L.orc_round_lp.restype = None
        L.orc_widen_f16.argtypes = [vp, C.c_uint64, vp]
        L.orc_widen_f16.restype = None
        L.orc_is_decision_step.argtypes = [C.c_int64, C.c_int64]
        L.orc_decide.argtypes = [C.POINTER(Policy), vp, C.c_int, C.c_int64, vp, vp]
        L.orc_decide.restype = None
        _lib = L
    return _lib


LINEAR, LOG, LOG_PL = 0, 1, 2      # LOG_PL: the log quantizer with the piecewise-linear logarithm
LOG_SR, LOG_TS = 3, 4              # LOG_SR: stochastic rounding (normalised piecewise-linear log); LOG_TS: two scales
WIDTHS = (2, 3, 4, 8, 16, 32)


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a: np.ndarray, dtype) -> np.ndarray:
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a


def codes_bytes(n: int, bits: int) -> int:
    return int(lib().orc_codes_bytes(n, bits))


def num_blocks(n: int, block: int) -> int:
    return int(lib().orc_num_blocks(n, block))


def lg_P(x: float) -> float:
    return float(lib().orc_lg_P(float(np.float32(x))))


def lg_E(x: float) -> int:
    return int(lib().orc_lg_E(float(np.float32(x))))


def ex2(e: float) -> float:
    return float(lib().orc_ex2(float(np.float32(e))))


def pack(code: np.ndarray, bits: int) -> np.ndarray:
    code = np.ascontiguousarray(code, dtype=np.uint32)
    out = np.zeros(codes_bytes(code.size, bits), dtype=np.uint8)
    lib().orc_pack(_p(code), code.size, bits, _p(out))
    return out


def unpack(buf: np.ndarray, n: int, bits: int) -> np.ndarray:
    _chk(buf, np.uint8)
    out = np.zeros(n, dtype=np.uint32)
    lib().orc_unpack(_p(buf), n, bits, _p(out))
    return out


def num_scales(n: int, block: int, mode: int) -> int:
    """Stored fp32 scales of a state: one per block, two in the two-scale variant."""
    return int(lib().orc_num_scales(n, block, mode))


def alloc_state(n: int, bits: int, block: int, mode: int = LOG):
    """Zero-filled (codes, scales) buffers of the stored sizes."""
    return (np.zeros(codes_bytes(n, bits), dtype=np.uint8),
            np.zeros(num_scales(n, block, mode) if bits != 32 else 0, dtype=np.float32))


def quantize(x: np.ndarray, bits: int, block: int, mode: int, key: int | None = None):
    """key: the 32-bit key of the stochastic-rounding variant (None: it rounds to nearest)."""
    x = _chk(np.ascontiguousarray(x), np.float32)
    codes, scales = alloc_state(x.size, bits, block, mode)
    if key is None:
        rc = lib().orc_quantize(_p(x), x.size, bits, block, mode, _p(codes), _p(scales))
    else:
        rc = lib().orc_quantize_keyed(_p(x), x.size, bits, block, mode, key, _p(codes), _p(scales))
    assert rc == 0
    return codes, scales


def mix32(h: int) -> int:
    return int(lib().orc_mix32(h & 0xFFFFFFFF))


def sr_key(seed: int, step: int, tensor: int) -> int:
    return int(lib().orc_sr_key(seed, step, tensor))


def sr_word(key: int, element: int) -> int:
    return int(lib().orc_sr_word(key, element))


def sr_code(x: float, s: float, bits: int, word: int) -> int:
    return int(lib().orc_sr_code(float(np.float32(x)), float(np.float32(s)), bits, word))


def sr_level(code: int, bits: int) -> float:
    return float(lib().orc_sr_level(code, bits))


def sr_enumerate(x: float, s: float, bits: int):
    """Over all 2^32 random words: ((lower code, count), (upper code, count)) of element x in a block of maximum s."""
    codes = np.zeros(2, dtype=np.uint32)
    counts = np.zeros(2, dtype=np.uint64)
    lib().orc_sr_enumerate(float(np.float32(x)), float(np.float32(s)), bits, _p(codes), _p(counts))
    return (int(codes[0]), int(counts[0])), (int(codes[1]), int(counts[1]))


def dequantize(codes: np.ndarray, scales: np.ndarray, n: int, bits: int, block: int, mode: int):
    _chk(codes, np.uint8)
    _chk(scales, np.float32)
    out = np.zeros(n, dtype=np.float32)
    rc = lib().orc_dequantize(_p(codes), _p(scales), n, bits, block, mode, _p(out))
    assert rc == 0
    return out


def init_state(n: int, block: int, bits_m: int, bits_v: int):
    mc, ms = alloc_state(n, bits_m, block)
    vc, vs = alloc_state(n, bits_v, block)
    rc = lib().orc_init_state(n, block, bits_m, bits_v, _p(mc), _p(ms), _p(vc), _p(vs))
    assert rc == 0
    return mc, ms, vc, vs


def _grad_dtype(grad: np.ndarray, fp16: bool) -> int:
    if grad.dtype == np.uint16:
        return 2 if fp16 else 1
    _chk(grad, np.float32)
    return 0


def grad_stats(grad: np.ndarray, fp16: bool = False) -> np.ndarray:
    """grad: float32, or uint16 holding bf16 (default) or fp16 (fp16=True) bit patterns."""
    dt = _grad_dtype(grad, fp16)
    out = np.zeros(4, dtype=np.float64)
    lib().orc_grad_stats(_p(grad), dt, grad.size, _p(out))
    return out


@dataclass
class State:
    """Stored optimizer state of one tensor (or block range)."""
    m_codes: np.ndarray
    m_scales: np.ndarray
    bits_m: int
    v_codes: np.ndarray
    v_scales: np.ndarray
    bits_v: int


def new_state(n: int, block: int, bits_m: int, bits_v: int, v_mode: int = LOG) -> State:
    mc, ms, vc, vs = init_state(n, block, bits_m, bits_v)
    if v_mode == LOG_TS and bits_v != 32:
        vs = np.zeros(num_scales(n, block, LOG_TS), dtype=np.float32)     # zero state: both scales 0
    return State(mc, ms, bits_m, vc, vs, bits_v)


def step(theta: np.ndarray, grad: np.ndarray, st: State, block: int, *, lr, beta1, beta2, eps,
         weight_decay, t: int, bits_m_out: int | None = None, bits_v_out: int | None = None,
         decoupled_wd: bool = True, want_stats: bool = False, fp16_grad: bool = False,
         inv_grad_scale: float = 1.0, found_inf: bool = False, v_mode: int = LOG, sr_seed: int = 0,
         tensor_index: int = 0):
    """One Algorithm-1 step on one tensor.  theta is updated in place; returns (new State, stats).
    A uint16 grad holds bf16 bit patterns, or fp16 ones with fp16_grad=True.  v_mode: LOG, LOG_PL, LOG_SR or
    LOG_TS, the quantizer of the second moment (the stored state must have been written with the same one);
    sr_seed and tensor_index key the random words of LOG_SR."""
    _chk(theta, np.float32)
    n = theta.size
    dt = _grad_dtype(grad, fp16_grad)
    assert grad.size == n
    bm = st.bits_m if bits_m_out is None else bits_m_out
    bv = st.bits_v if bits_v_out is None else bits_v_out
    mc, ms = alloc_state(n, bm, block)
    vc, vs = alloc_state(n, bv, block, v_mode)
    hp = HParams(lr, beta1, beta2, eps, weight_decay, t, 1 if decoupled_wd else 0, dt, inv_grad_scale,
                 1 if found_inf else 0, v_mode, sr_seed, tensor_index, 0)
    stats = np.zeros(4, dtype=np.float64) if want_stats else None
    rc = lib().orc_step(_p(theta), _p(grad), n, block,
                        _p(st.m_codes), _p(st.m_scales), st.bits_m,
                        _p(st.v_codes), _p(st.v_scales), st.bits_v,
                        _p(mc), _p(ms), bm, _p(vc), _p(vs), bv, C.byref(hp), _p(stats))
    assert rc == 0
    if found_inf:      # the skipped step touched nothing: the stored state stands, no statistics
        return st, (np.zeros(4) if want_stats else None)
    return State(mc, ms, bm, vc, vs, bv), stats


def step_range(theta: np.ndarray, grad: np.ndarray, e0: int, e1: int, block: int, st_in: State, st_out: State, *,
               lr, beta1, beta2, eps, weight_decay, t: int, decoupled_wd: bool = True, fp16_grad: bool = False,
               inv_grad_scale: float = 1.0, v_mode: int = LOG, stats: np.ndarray | None = None, sr_seed: int = 0,
               tensor_index: int = 0) -> None:
    """The same Algorithm-1 step on the elements [e0, e1) of one tensor, e0 a multiple of the block size (blocks
    are independent given their inputs, so a tensor may be stepped range by range, in any order or in
    parallel).  theta, grad and the buffers of st_in / st_out belong to the whole tensor; theta and st_out are
    written in place for the range only.  stats: float64[4] for this range's sums, or None."""
    assert e0 % block == 0 and 0 <= e0 < e1 <= theta.size
    n = e1 - e0
    dt = _grad_dtype(grad, fp16_grad)

    def cut(st: State):
        def codes(c, b):
            return c[e0 * 4:] if b == 32 else c[e0 * b // 8:]          # a block is a whole number of bytes
        spb = 2 if v_mode == LOG_TS else 1
        return (codes(st.m_codes, st.bits_m), st.m_scales[e0 // block:] if st.bits_m != 32 else st.m_scales,
                codes(st.v_codes, st.bits_v), st.v_scales[spb * (e0 // block):] if st.bits_v != 32 else st.v_scales)

    mci, msi, vci, vsi = cut(st_in)
    mco, mso, vco, vso = cut(st_out)
    hp = HParams(lr, beta1, beta2, eps, weight_decay, t, 1 if decoupled_wd else 0, dt, inv_grad_scale, 0, v_mode,
                 sr_seed, tensor_index, e0)
    rc = lib().orc_step(_p(theta[e0:]), _p(grad[e0:]), n, block, _p(mci), _p(msi), st_in.bits_m, _p(vci), _p(vsi),
                        st_in.bits_v, _p(mco), _p(mso), st_out.bits_m, _p(vco), _p(vso), st_out.bits_v,
                        C.byref(hp), _p(stats))
    assert rc == 0


def round_lp(x: np.ndarray, lp: str) -> np.ndarray:
    """Nearest-even rounding of fp32 values to "bf16" or "fp16"; returns the uint16 bit patterns."""
    x = _chk(np.ascontiguousarray(x), np.float32)
    out = np.zeros(x.size, dtype=np.uint16)
    lib().orc_round_lp(_p(x), x.size, 1 if lp == "bf16" else 2, _p(out))
    return out


def widen_f16(bits: np.ndarray) -> np.ndarray:
    _chk(bits, np.uint16)
    out = np.zeros(bits.size, dtype=np.float32)
    lib().orc_widen_f16(_p(bits), bits.size, _p(out))
    return out


def repack(codes: np.ndarray, scales: np.ndarray, bits_in: int, bits_out: int, n: int, block: int,
           mode: int):
    co, so = alloc_state(n, bits_out, block, mode)
    rc = lib().orc_repack(_p(codes), _p(scales), bits_in, _p(co), _p(so), bits_out, n, block, mode)
    assert rc == 0
    return co, so


def is_decision_step(t: int, U: int) -> bool:
    return bool(lib().orc_is_decision_step(t, U))


def new_policy(alpha: float, tau: float, eps_stat: float = 1e-8, cv_of_signed: bool = False) -> Policy:
    return Policy(0.0, 0.0, 0.0, alpha, tau, eps_stat, 1 if cv_of_signed else 0)


def decide(pol: Policy, stats: np.ndarray, t: int):
    """stats: [L,4] float64.  Returns (bits[L] uint8, score[L] float64); pol is updated."""
    stats = _chk(np.ascontiguousarray(stats), np.float64)
    L = stats.shape[0]
    bits = np.zeros(L, dtype=np.uint8)
    score = np.zeros(L, dtype=np.float64)
    lib().orc_decide(C.byref(pol), _p(stats), L, t, _p(bits), _p(score))
    return bits, score
