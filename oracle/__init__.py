"""CPU oracle for the truncated-quantization compressor -- TEST INFRASTRUCTURE.

A thin NumPy/ctypes face on ``tq_oracle.c`` (plain single-threaded C written from the
paper).  It is independent of the CUDA library: it imports nothing from the product
package and the product never imports it.  Only ``tests/``, the smoke check and the
benchmark's CPU-baseline leg may use it.

Every function here marshals arguments and calls one C routine; the arithmetic lives in
``tq_oracle.c``, whose header lists the passages of the paper each routine follows and
the readings taken where the paper is silent.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tq_oracle.c")
_LIB = os.path.join(_HERE, "libtq_oracle.so")

MAX_LEVELS = 16
UNIFORM, NONUNIFORM, BISCALED = 0, 1, 2
ALPHA_CLOSED, ALPHA_FIXED_POINT, ALPHA_USER, ALPHA_MAXABS = 0, 1, 2, 3
FLAG_ALPHA_CAPPED, FLAG_ALPHA_AT_GMIN, FLAG_GAMMA_FROM_MLE = 1, 2, 4
OK, ERR_ARG, ERR_DOMAIN, ERR_LEVELS = 0, -1, -2, -5


class Stats(C.Structure):
    _fields_ = [("d", C.c_uint64), ("n_tail", C.c_uint64), ("n_nonfinite", C.c_uint64),
                ("sum_abs", C.c_double), ("sum_sq", C.c_double), ("sum_log_tail", C.c_double),
                ("max_abs", C.c_float), ("g_min", C.c_float)]


class Params(C.Structure):
    _fields_ = [("bits", C.c_uint32), ("num_levels", C.c_uint32), ("mode", C.c_uint32),
                ("flags", C.c_uint32), ("alpha", C.c_float), ("inv_step", C.c_float),
                ("gamma", C.c_float), ("g_min", C.c_float), ("rho", C.c_float),
                ("iterations", C.c_int32),
                ("levels", C.c_float * MAX_LEVELS), ("inv_width", C.c_float * MAX_LEVELS)]

    def levels_np(self) -> np.ndarray:
        return np.array(self.levels[: self.num_levels], dtype=np.float32)

    def inv_width_np(self) -> np.ndarray:
        return np.array(self.inv_width[: self.num_levels - 1], dtype=np.float32)


class Model(C.Structure):
    _fields_ = [("g_min", C.c_double), ("rho", C.c_double), ("gamma", C.c_double)]


def build(force: bool = False) -> str:
    """Compile ``tq_oracle.c`` into ``libtq_oracle.so`` beside it (no-op when up to date)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
           "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        # TQ_ORACLE_LIB: load another build of the oracle (the mutation test plants mistakes this way)
        L = C.CDLL(os.environ.get("TQ_ORACLE_LIB") or build())
        u32, u64, f32, f64, i32 = C.c_uint32, C.c_uint64, C.c_float, C.c_double, C.c_int
        P = C.POINTER
        L.orc_philox4x32_10.argtypes = [P(u32), P(u32), P(u32)]
        L.orc_philox4x32_10.restype = None
        L.orc_rand16.argtypes = [u64, u32, u64]; L.orc_rand16.restype = u32
        L.orc_bf16_to_f32.argtypes = [C.c_void_p, u64, C.c_void_p]; L.orc_bf16_to_f32.restype = None
        L.orc_stats.argtypes = [C.c_void_p, u64, f32, f64, P(Stats)]; L.orc_stats.restype = i32
        L.orc_pow2_floor.argtypes = [f32]; L.orc_pow2_floor.restype = f32
        for name in ("orc_model_pdf", "orc_model_QU", "orc_model_H", "orc_model_Hinv",
                     "orc_model_QN", "orc_truncation_bias"):
            fn = getattr(L, name); fn.argtypes = [P(Model), f64]; fn.restype = f64
        for name in ("orc_etq_uniform", "orc_etq_nonuniform", "orc_etq_theorem", "orc_etq_biscaled", "orc_model_QB"):
            fn = getattr(L, name); fn.argtypes = [P(Model), f64, f64]; fn.restype = f64
        L.orc_biscaled_kstar.argtypes = [P(Model), f64]; L.orc_biscaled_kstar.restype = f64
        L.orc_biscaled_density.argtypes = [P(Model), f64, f64, P(f64), P(f64), P(f64)]; L.orc_biscaled_density.restype = None
        L.orc_alpha_prime.argtypes = [P(Model), f64]; L.orc_alpha_prime.restype = f64
        L.orc_alpha_fixed_point.argtypes = [P(Model), f64, i32, f64, P(i32), P(i32)]
        L.orc_alpha_fixed_point.restype = f64
        L.orc_build_table.argtypes = [P(Model), u32, i32, f32, P(Params)]; L.orc_build_table.restype = i32
        L.orc_table_from_levels.argtypes = [C.c_void_p, u32, i32, P(Params)]
        L.orc_table_from_levels.restype = i32
        L.orc_params.argtypes = [P(Stats), u32, i32, f64, i32, f64, P(Params)]; L.orc_params.restype = i32
        L.orc_code_from_bits.argtypes = [P(Params), f32, u32]; L.orc_code_from_bits.restype = u32
        L.orc_code_at.argtypes = [P(Params), f32, u64, u32, u64]; L.orc_code_at.restype = u32
        L.orc_decision.argtypes = [P(Params), f32, P(f32), P(u32), P(f32), P(u32)]
        L.orc_decision.restype = None
        L.orc_quantize.argtypes = [C.c_void_p, u64, P(Params), u64, u32, C.c_void_p]
        L.orc_quantize.restype = None
        L.orc_quantize_window.argtypes = [C.c_void_p, u64, u64, P(Params), u64, u32, C.c_void_p]
        L.orc_quantize_window.restype = None
        L.orc_packed_words.argtypes = [u64, u32]; L.orc_packed_words.restype = u64
        L.orc_pack.argtypes = [C.c_void_p, u64, u32, C.c_void_p, u64]; L.orc_pack.restype = None
        L.orc_unpack.argtypes = [C.c_void_p, u64, u32, C.c_void_p]; L.orc_unpack.restype = None
        L.orc_compress.argtypes = [C.c_void_p, u64, P(Params), u64, u32, C.c_void_p, u64, C.c_void_p]
        L.orc_compress.restype = i32
        L.orc_decompress_aggregate.argtypes = [C.c_void_p, u64, u32, u64, P(Params), C.c_void_p, C.c_void_p]
        L.orc_decompress_aggregate.restype = i32
        L.orc_decompress_aggregate_apply.argtypes = [C.c_void_p, u64, u32, u64, P(Params), C.c_void_p, C.c_void_p,
                                                     C.c_void_p, f32, f32, f32, C.c_void_p]
        L.orc_decompress_aggregate_apply.restype = i32
        L.orc_sizeof_params.restype = u32; L.orc_sizeof_stats.restype = u32
        assert L.orc_sizeof_params() == C.sizeof(Params), "Params layout drifted from tq_oracle.c"
        assert L.orc_sizeof_stats() == C.sizeof(Stats), "Stats layout drifted from tq_oracle.c"
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: oracle status {code}")
        self.code = code


def _check(code: int, where: str) -> None:
    if code != OK:
        raise OracleError(code, where)


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


# ---------------------------------------------------------------- random bits
def philox4x32_10(counter: Sequence[int], key: Sequence[int]) -> np.ndarray:
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in counter])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return np.array(list(o), dtype=np.uint32)


def rand16(seed: int, worker: int, j: int) -> int:
    return int(lib().orc_rand16(seed, worker, j))


# ---------------------------------------------------------------- statistics / parameters
def bf16_to_f32(raw_u16: np.ndarray) -> np.ndarray:
    raw = np.ascontiguousarray(raw_u16, dtype=np.uint16)
    out = np.empty(raw.shape, dtype=np.float32)
    lib().orc_bf16_to_f32(raw.ctypes.data, raw.size, out.ctypes.data)
    return out


def stats(g: np.ndarray, g_min: float = 0.0, kappa: float = 1.0) -> Stats:
    g = _f32(g)
    st = Stats()
    _check(lib().orc_stats(g.ctypes.data, g.size, g_min, kappa, C.byref(st)), "orc_stats")
    return st


def pow2_floor(x: float) -> float:
    return float(lib().orc_pow2_floor(C.c_float(x)))


def stats_pow2(g: np.ndarray, kappa: float = 1.0) -> Stats:
    """Statistics under the power-of-two threshold rule: g_min = pow2_floor((float)(kappa * mean|g|))."""
    first = stats(g, 0.0, kappa)
    g_min = pow2_floor(first.g_min)
    if not g_min > 0.0:
        first.g_min = 0.0
        first.n_tail = 0
        first.sum_log_tail = 0.0
        return first
    return stats(g, g_min, kappa)


def params(st: Stats, num_levels: int, mode: int, gamma: float = math.nan,
           alpha_rule: int = ALPHA_FIXED_POINT, alpha_user: float = 0.0) -> Params:
    p = Params()
    _check(lib().orc_params(C.byref(st), num_levels, mode, gamma, alpha_rule, alpha_user, C.byref(p)),
           "orc_params")
    return p


def build_table(model: Model, num_levels: int, mode: int, alpha: float) -> Params:
    p = Params()
    bits = {2: 1, 4: 2, 8: 3, 16: 4}[num_levels]
    p.bits, p.num_levels, p.mode = bits, num_levels, mode
    _check(lib().orc_build_table(C.byref(model), num_levels, mode, alpha, C.byref(p)), "orc_build_table")
    return p


def table_params(levels: Sequence[float], mode: int = NONUNIFORM) -> Params:
    """Params for a caller-supplied antisymmetric codebook (no density model)."""
    lv = _f32(levels)
    p = Params()
    _check(lib().orc_table_from_levels(lv.ctypes.data, lv.size, mode, C.byref(p)), "orc_table_from_levels")
    return p


def model_fn(name: str, model: Model, x: float, s: Optional[float] = None) -> float:
    fn = getattr(lib(), "orc_" + name)
    return float(fn(C.byref(model), x) if s is None else fn(C.byref(model), x, s))


def biscaled_kstar(model: Model, alpha: float) -> float:
    return float(lib().orc_biscaled_kstar(C.byref(model), alpha))


def biscaled_density(model: Model, alpha: float, s: float):
    """(k*, lambda_in, lambda_out) of the boxed BiScaled density."""
    k, a, b = C.c_double(), C.c_double(), C.c_double()
    lib().orc_biscaled_density(C.byref(model), alpha, s, C.byref(k), C.byref(a), C.byref(b))
    return k.value, a.value, b.value


def alpha_prime(model: Model, s: float) -> float:
    return float(lib().orc_alpha_prime(C.byref(model), s))


def alpha_fixed_point(model: Model, s: float, mode: int, cap: float = 0.0):
    it, capped = C.c_int(0), C.c_int(0)
    a = lib().orc_alpha_fixed_point(C.byref(model), s, mode, cap, C.byref(it), C.byref(capped))
    return float(a), it.value, bool(capped.value)


# ---------------------------------------------------------------- compressor
def decision(p: Params, g: float):
    """(t, k, p_r, T) for one value: truncated value, interval, round-up probability, threshold."""
    t, k, pr, T = C.c_float(), C.c_uint32(), C.c_float(), C.c_uint32()
    lib().orc_decision(C.byref(p), g, C.byref(t), C.byref(k), C.byref(pr), C.byref(T))
    return t.value, k.value, pr.value, T.value


def code_from_bits(p: Params, g: float, r16: int) -> int:
    return int(lib().orc_code_from_bits(C.byref(p), g, r16))


def code_at(p: Params, g: float, seed: int, worker: int, j: int) -> int:
    return int(lib().orc_code_at(C.byref(p), g, seed, worker, j))


def quantize(g: np.ndarray, p: Params, seed: int, worker: int) -> np.ndarray:
    g = _f32(g)
    codes = np.empty(g.size, dtype=np.uint8)
    lib().orc_quantize(g.ctypes.data, g.size, C.byref(p), seed, worker, codes.ctypes.data)
    return codes


def quantize_window(g: np.ndarray, j0: int, p: Params, seed: int, worker: int) -> np.ndarray:
    """Codes of elements j0 .. j0+len(g)-1 of a longer vector (``g`` holds just that window)."""
    g = _f32(g)
    codes = np.empty(g.size, dtype=np.uint8)
    lib().orc_quantize_window(g.ctypes.data, g.size, j0, C.byref(p), seed, worker, codes.ctypes.data)
    return codes


def packed_words(d: int, bits: int) -> int:
    return int(lib().orc_packed_words(d, bits))


def pack(codes: np.ndarray, bits: int, words: Optional[int] = None) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    words = packed_words(codes.size, bits) if words is None else words
    out = np.empty(words, dtype=np.uint32)
    lib().orc_pack(codes.ctypes.data, codes.size, bits, out.ctypes.data, words)
    return out


def unpack(packed: np.ndarray, d: int, bits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    codes = np.empty(d, dtype=np.uint8)
    lib().orc_unpack(packed.ctypes.data, d, bits, codes.ctypes.data)
    return codes


def compress(g: np.ndarray, p: Params, seed: int, worker: int, words: Optional[int] = None) -> np.ndarray:
    g = _f32(g)
    words = packed_words(g.size, p.bits) if words is None else words
    out = np.empty(words, dtype=np.uint32)
    scratch = np.empty(max(g.size, 1), dtype=np.uint8)
    _check(lib().orc_compress(g.ctypes.data, g.size, C.byref(p), seed, worker, out.ctypes.data, words,
                              scratch.ctypes.data), "orc_compress")
    return out


def decompress_aggregate(packed: np.ndarray, d: int, params_list: Sequence[Params],
                         weights: Optional[Sequence[float]] = None) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    n = len(params_list)
    assert packed.ndim == 2 and packed.shape[0] == n
    arr = (Params * n)(*params_list)
    out = np.empty(d, dtype=np.float32)
    w = None if weights is None else _f32(weights)
    _check(lib().orc_decompress_aggregate(packed.ctypes.data, packed.shape[1], n, d, arr,
                                          None if w is None else w.ctypes.data, out.ctypes.data),
           "orc_decompress_aggregate")
    return out


def decompress_aggregate_apply(packed: np.ndarray, d: int, params_list: Sequence[Params], theta: np.ndarray,
                               momentum_buf: Optional[np.ndarray], lr: float, mu: float, wd: float,
                               weights: Optional[Sequence[float]] = None):
    """Aggregate and apply the model update in place on ``theta`` (and ``momentum_buf`` if given)."""
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    n = len(params_list)
    arr = (Params * n)(*params_list)
    assert theta.dtype == np.float32 and theta.flags.c_contiguous and theta.size == d
    if momentum_buf is not None:
        assert momentum_buf.dtype == np.float32 and momentum_buf.flags.c_contiguous and momentum_buf.size == d
    scratch = np.empty(d, dtype=np.float32)
    w = None if weights is None else _f32(weights)
    _check(lib().orc_decompress_aggregate_apply(packed.ctypes.data, packed.shape[1], n, d, arr,
                                                None if w is None else w.ctypes.data, theta.ctypes.data,
                                                None if momentum_buf is None else momentum_buf.ctypes.data,
                                                lr, mu, wd, scratch.ctypes.data), "orc_decompress_aggregate_apply")
    return theta
