"""ctypes binding of libtq.so: same names and argument order as include/tq.h.

Only argument marshalling happens here.  Tensors are torch tensors used as typed device
buffers; the stream is torch's current CUDA stream unless one is given.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional, Sequence, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtq.so")

MAX_LEVELS, MAX_WORKERS = 16, 64
OK, ERR_INVALID_ARG, ERR_DOMAIN, ERR_ALIGNMENT, ERR_BUFFER_TOO_SMALL, ERR_DEGENERATE_LEVELS, ERR_CUDA = \
    0, -1, -2, -3, -4, -5, -6
ERR_STATIC_LIMIT = -7
STATIC_MAX_WORKERS = 16
F32, BF16 = 0, 1
UNIFORM, NONUNIFORM, BISCALED = 0, 1, 2
ALPHA_CLOSED, ALPHA_FIXED_POINT, ALPHA_USER, ALPHA_MAXABS = 0, 1, 2, 3
FLAG_ALPHA_CAPPED, FLAG_ALPHA_AT_GMIN, FLAG_GAMMA_FROM_MLE, FLAG_INVALID = 1, 2, 4, 8

EXPORTS = ("tq_packed_words", "tq_stats_workspace_bytes", "tq_stats", "tq_stats_hinted", "tq_stats_static", "tq_params", "tq_params_batch", "tq_params_from_levels", "tq_params_device",
           "tq_compress_device_params", "tq_decompress_aggregate_device_params",
           "tq_compress", "tq_decompress_aggregate", "tq_decompress_aggregate_rows", "tq_decompress_aggregate_apply",
           "tq_segments_packed_words", "tq_stats_segments", "tq_stats_hinted_segments", "tq_compress_segments", "tq_decompress_aggregate_segments", "tq_strerror", "tq_last_cuda_error", "tq_kernel_launches", "tq_wait_expired_count")


class Stats(C.Structure):
    """tq_stats_t (64 bytes)."""
    _fields_ = [("d", C.c_uint64), ("n_tail", C.c_uint64), ("n_nonfinite", C.c_uint64),
                ("sum_abs", C.c_double), ("sum_sq", C.c_double), ("sum_log_tail", C.c_double),
                ("max_abs", C.c_float), ("g_min", C.c_float), ("reserved", C.c_uint64)]


class Params(C.Structure):
    """tq_params_t (176 bytes)."""
    _fields_ = [("bits", C.c_uint32), ("num_levels", C.c_uint32), ("mode", C.c_uint32), ("flags", C.c_uint32),
                ("alpha", C.c_float), ("inv_step", C.c_float), ("gamma", C.c_float), ("g_min", C.c_float),
                ("rho", C.c_float), ("iterations", C.c_int32), ("reserved", C.c_float * 2),
                ("levels", C.c_float * MAX_LEVELS), ("inv_width", C.c_float * MAX_LEVELS)]


assert C.sizeof(Stats) == 64 and C.sizeof(Params) == 176


class TqError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        super().__init__(f"{where}: {detail or status} (status {status})")
        self.status = status


_lib: Optional[C.CDLL] = None


class Segment(C.Structure):
    """tq_segment_t: a layer group, [offset, offset + length) of every worker's row (elements)."""
    _fields_ = [("offset", C.c_uint64), ("length", C.c_uint64)]


def lib() -> C.CDLL:
    """Load libtq.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2402_01798_b200.build` "
                "(there is no CPU or PyTorch fallback for the compressor)")
        L = C.CDLL(LIB_PATH)
        vp, u32, u64, f32, f64, sz = C.c_void_p, C.c_uint32, C.c_uint64, C.c_float, C.c_double, C.c_size_t
        L.tq_packed_words.argtypes = [u64, u32]; L.tq_packed_words.restype = sz
        L.tq_stats_workspace_bytes.argtypes = [u32]; L.tq_stats_workspace_bytes.restype = sz
        L.tq_stats.argtypes = [vp, C.c_int, u64, u64, u32, f32, f32, vp, vp, sz, vp]; L.tq_stats.restype = C.c_int
        L.tq_stats_hinted.argtypes = [vp, C.c_int, u64, u64, u32, f32, vp, vp, vp, sz, vp]; L.tq_stats_hinted.restype = C.c_int
        L.tq_stats_static.argtypes = [vp, C.c_int, u64, u64, u32, f32, f32, vp, vp]; L.tq_stats_static.restype = C.c_int
        L.tq_params.argtypes = [C.POINTER(Stats), u32, C.c_int, f64, C.c_int, f64, C.POINTER(Params)]
        L.tq_params.restype = C.c_int
        L.tq_params_batch.argtypes = [vp, u32, u32, C.c_int, f64, C.c_int, f64, vp]
        L.tq_params_batch.restype = C.c_int
        L.tq_params_from_levels.argtypes = [C.POINTER(f32), u32, C.c_int, C.POINTER(Params)]
        L.tq_params_from_levels.restype = C.c_int
        L.tq_compress.argtypes = [vp, C.c_int, u64, u64, u32, C.POINTER(Params), u64, u32, vp, sz, vp]
        L.tq_compress.restype = C.c_int
        L.tq_decompress_aggregate.argtypes = [vp, sz, u32, u64, C.POINTER(Params), C.POINTER(f32), vp, vp]
        L.tq_decompress_aggregate.restype = C.c_int
        L.tq_decompress_aggregate_rows.argtypes = [C.POINTER(C.c_void_p), u32, u64, C.POINTER(Params), C.POINTER(f32), vp, vp]
        L.tq_decompress_aggregate_rows.restype = C.c_int
        L.tq_params_device.argtypes = [vp, u32, u32, C.c_int, f64, C.c_int, f64, vp, vp]
        L.tq_params_device.restype = C.c_int
        L.tq_compress_device_params.argtypes = [vp, C.c_int, u64, u64, u32, vp, u32, C.c_int, u64, u32, vp, sz, vp]
        L.tq_compress_device_params.restype = C.c_int
        L.tq_decompress_aggregate_device_params.argtypes = [vp, sz, u32, u64, vp, u32, C.POINTER(f32), vp, vp]
        L.tq_decompress_aggregate_device_params.restype = C.c_int
        L.tq_decompress_aggregate_apply.argtypes = [vp, sz, u32, u64, C.POINTER(Params), C.POINTER(f32), vp, vp, f32, f32, f32, vp]
        L.tq_decompress_aggregate_apply.restype = C.c_int
        L.tq_segments_packed_words.argtypes = [C.POINTER(Segment), u32, u32]; L.tq_segments_packed_words.restype = sz
        L.tq_stats_segments.argtypes = [vp, C.c_int, u64, u32, C.POINTER(Segment), u32, f32, f32, vp, vp, sz, vp]
        L.tq_stats_segments.restype = C.c_int
        L.tq_stats_hinted_segments.argtypes = [vp, C.c_int, u64, u32, C.POINTER(Segment), u32, f32, vp, vp, vp, sz, vp]
        L.tq_stats_hinted_segments.restype = C.c_int
        L.tq_compress_segments.argtypes = [vp, C.c_int, u64, u32, C.POINTER(Segment), u32, vp, u32, C.c_int, u64, u32, vp, sz, vp]
        L.tq_compress_segments.restype = C.c_int
        L.tq_decompress_aggregate_segments.argtypes = [vp, sz, u32, C.POINTER(Segment), u32, vp, u32, C.POINTER(f32), vp, vp]
        L.tq_decompress_aggregate_segments.restype = C.c_int
        L.tq_strerror.argtypes = [C.c_int]; L.tq_strerror.restype = C.c_char_p
        L.tq_last_cuda_error.restype = C.c_int
        L.tq_kernel_launches.restype = u64
        L.tq_wait_expired_count.argtypes = [C.POINTER(u32)]; L.tq_wait_expired_count.restype = C.c_int
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != OK:
        L = lib()
        detail = L.tq_strerror(status).decode()
        if status == ERR_CUDA:
            detail += f" (cudaError {L.tq_last_cuda_error()})"
        raise TqError(status, where, detail)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("gradient must be float32 or bfloat16")


def _grad_layout(grad: torch.Tensor, d: Optional[int]):
    """(n_workers, d, stride) of a [N, stride] or [d] gradient tensor on the GPU."""
    if not grad.is_cuda:
        raise ValueError("gradient must be a CUDA tensor")
    if grad.dim() == 1:
        grad = grad.unsqueeze(0)
    if grad.dim() != 2 or grad.stride(1) != 1:
        raise ValueError("gradient must be [N, stride] with unit inner stride")
    n, width = grad.shape
    return n, (width if d is None else d), (grad.stride(0) if n > 1 else width)


def params_array(params: Sequence[Params]):
    """A contiguous tq_params_t[N] for tq_compress / tq_decompress_aggregate (build once, pass many times)."""
    return (Params * len(params))(*params)


def _params_array(params):
    return params if isinstance(params, C.Array) else params_array(params)


# ------------------------------------------------------------------------------------------------
def tq_packed_words(d: int, bits: int) -> int:
    return int(lib().tq_packed_words(d, bits))


def tq_stats_workspace_bytes(n_workers: int) -> int:
    return int(lib().tq_stats_workspace_bytes(n_workers))


def tq_stats(grad: torch.Tensor, d: Optional[int] = None, g_min: float = 0.0, kappa: float = 1.0,
             stats_dev: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None):
    """Enqueue the statistics reduction; returns the device tensor holding n_workers 64-byte records."""
    n, d, stride = _grad_layout(grad, d)
    if stats_dev is None:
        stats_dev = torch.empty(n * 64, dtype=torch.uint8, device=grad.device)
    if workspace is None:
        workspace = torch.empty(tq_stats_workspace_bytes(n), dtype=torch.uint8, device=grad.device)
    _check(lib().tq_stats(grad.data_ptr(), _dtype_code(grad), d, stride, n, g_min, kappa, stats_dev.data_ptr(),
                          workspace.data_ptr(), workspace.numel(), _stream(stream)), "tq_stats")
    return stats_dev


def tq_stats_hinted(grad: torch.Tensor, hint: torch.Tensor, d: Optional[int] = None, kappa: float = 1.0,
                    stats_dev: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None):
    """One-pass statistics with g_min = kappa * mean|g| rounded down to a power of two.

    ``hint`` is a device tensor of n_workers * 8 bytes (tq_gmin_hint_t records) that the caller keeps from
    round to round; zero it before the first one (``new_gmin_hint``).  Returns the records' device tensor.
    """
    n, d, stride = _grad_layout(grad, d)
    if stats_dev is None:
        stats_dev = torch.empty(n * 64, dtype=torch.uint8, device=grad.device)
    if workspace is None:
        workspace = torch.empty(tq_stats_workspace_bytes(n), dtype=torch.uint8, device=grad.device)
    _check(lib().tq_stats_hinted(grad.data_ptr(), _dtype_code(grad), d, stride, n, kappa, hint.data_ptr(),
                                 stats_dev.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream(stream)),
           "tq_stats_hinted")
    return stats_dev


def new_gmin_hint(n_workers: int, device="cuda") -> torch.Tensor:
    """A zeroed hint buffer for tq_stats_hinted (n_workers records of {float level; uint32 hit})."""
    return torch.zeros(n_workers * 8, dtype=torch.uint8, device=device)


def gmin_hint_to_host(hint: torch.Tensor):
    """[(level, hit)] per worker (synchronises)."""
    raw = hint.cpu().numpy()
    return list(zip(raw.view("<f4")[0::2].tolist(), raw.view("<u4")[1::2].tolist()))


def tq_stats_static(grad: torch.Tensor, stats_dev: torch.Tensor, d: Optional[int] = None, g_min: float = 0.0,
                    kappa: float = 1.0, stream=None) -> torch.Tensor:
    """tq_stats for callers that cannot allocate: the scratch is the library's own fixed array.

    The caller passes the gradient and the output records (``stats_dev``, n_workers * 64 bytes); this
    wrapper allocates nothing either.  At most STATIC_MAX_WORKERS rows; calls that overlap on the GPU race.
    """
    n, d, stride = _grad_layout(grad, d)
    _check(lib().tq_stats_static(grad.data_ptr(), _dtype_code(grad), d, stride, n, g_min, kappa,
                                 stats_dev.data_ptr(), _stream(stream)), "tq_stats_static")
    return stats_dev


def stats_to_host(stats_dev: torch.Tensor):
    """Copy the records back (synchronises the current stream) and view them as Stats structures."""
    raw = stats_dev.cpu().numpy().tobytes()
    n = len(raw) // 64
    return [Stats.from_buffer_copy(raw[i * 64:(i + 1) * 64]) for i in range(n)]


def tq_params(stats: Stats, num_levels: int, mode: int, gamma: float = math.nan,
              alpha_rule: int = ALPHA_FIXED_POINT, alpha_user: float = 0.0) -> Params:
    p = Params()
    _check(lib().tq_params(C.byref(stats), num_levels, mode, gamma, alpha_rule, alpha_user, C.byref(p)), "tq_params")
    return p


def tq_params_batch(stats_raw, n_workers: int, num_levels: int, mode: int, gamma: float = math.nan,
                    alpha_rule: int = ALPHA_FIXED_POINT, alpha_user: float = 0.0):
    """tq_params for n workers at once.  ``stats_raw``: the n 64-byte records as bytes, a ctypes array of
    Stats, or a pinned CPU uint8 tensor (used in place).  Returns a ctypes tq_params_t[n] array."""
    out = (Params * n_workers)()
    if isinstance(stats_raw, torch.Tensor):
        src = C.c_void_p(stats_raw.data_ptr())
    elif isinstance(stats_raw, (bytes, bytearray)):
        src = C.cast(C.create_string_buffer(bytes(stats_raw), len(stats_raw)), C.c_void_p)
    else:
        src = C.cast(stats_raw, C.c_void_p)
    _check(lib().tq_params_batch(src, n_workers, num_levels, mode, gamma, alpha_rule, alpha_user,
                                 C.cast(out, C.c_void_p)), "tq_params_batch")
    return out


def tq_params_from_levels(levels: Sequence[float], mode: int = NONUNIFORM) -> Params:
    arr = (C.c_float * len(levels))(*[float(x) for x in levels])
    p = Params()
    _check(lib().tq_params_from_levels(arr, len(levels), mode, C.byref(p)), "tq_params_from_levels")
    return p


def tq_compress(grad: torch.Tensor, params: Sequence[Params], seed: int, first_worker: int = 0,
                d: Optional[int] = None, packed: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Enqueue truncate + stochastic round + pack for all rows of ``grad``; returns [N, words] int32."""
    n, d, stride = _grad_layout(grad, d)
    if len(params) != n:
        raise ValueError("one Params per worker")
    if packed is None:
        packed = torch.empty((n, tq_packed_words(d, params[0].bits)), dtype=torch.int32, device=grad.device)
    words_stride = packed.stride(0) if packed.dim() == 2 and n > 1 else packed.shape[-1]
    _check(lib().tq_compress(grad.data_ptr(), _dtype_code(grad), d, stride, n, _params_array(params),
                             seed & 0xFFFFFFFFFFFFFFFF, first_worker, packed.data_ptr(), words_stride,
                             _stream(stream)), "tq_compress")
    return packed


def tq_decompress_aggregate(packed: torch.Tensor, d: int, params: Sequence[Params],
                            weights: Optional[Sequence[float]] = None, out: Optional[torch.Tensor] = None,
                            stream=None) -> torch.Tensor:
    """Enqueue unpack + dequantize + average of the N packed rows; returns the [d] fp32 update."""
    if not packed.is_cuda or packed.dim() != 2:
        raise ValueError("packed must be a [N, words] CUDA tensor")
    n = packed.shape[0]
    if len(params) != n:
        raise ValueError("one Params per worker")
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=packed.device)
    w = None if weights is None else (C.c_float * n)(*[float(x) for x in weights])
    words_stride = packed.stride(0) if n > 1 else packed.shape[1]
    _check(lib().tq_decompress_aggregate(packed.data_ptr(), words_stride, n, d, _params_array(params), w,
                                         out.data_ptr(), _stream(stream)), "tq_decompress_aggregate")
    return out


def tq_decompress_aggregate_rows(rows: Sequence, d: int, params: Sequence[Params],
                                 weights: Optional[Sequence[float]] = None, out: Optional[torch.Tensor] = None,
                                 stream=None) -> torch.Tensor:
    """tq_decompress_aggregate with one packed row per worker, each given as a 1-D int32 CUDA tensor or as a
    raw device address (an int, e.g. a peer's buffer mapped into this process).  The caller keeps the rows
    alive until the stream has passed the call."""
    n = len(rows)
    if len(params) != n:
        raise ValueError("one Params per worker")
    ptrs = (C.c_void_p * n)(*[int(r) if isinstance(r, int) else r.data_ptr() for r in rows])
    if out is None:
        dev = next((r.device for r in rows if not isinstance(r, int)), "cuda")
        out = torch.empty(d, dtype=torch.float32, device=dev)
    w = None if weights is None else (C.c_float * n)(*[float(x) for x in weights])
    _check(lib().tq_decompress_aggregate_rows(ptrs, n, d, _params_array(params), w, out.data_ptr(), _stream(stream)),
           "tq_decompress_aggregate_rows")
    return out


def tq_params_device(stats_dev: torch.Tensor, n_workers: int, num_levels: int, mode: int, gamma: float = math.nan,
                     alpha_rule: int = ALPHA_FIXED_POINT, alpha_user: float = 0.0,
                     params_dev: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Enqueue the parameter design on the device; returns the device tensor of n_workers 176-byte records."""
    if params_dev is None:
        params_dev = torch.empty(n_workers * C.sizeof(Params), dtype=torch.uint8, device=stats_dev.device)
    _check(lib().tq_params_device(stats_dev.data_ptr(), n_workers, num_levels, mode, gamma, alpha_rule, alpha_user,
                                  params_dev.data_ptr(), _stream(stream)), "tq_params_device")
    return params_dev


def params_to_host(params_dev: torch.Tensor):
    """Copy device parameter records back (synchronises) and view them as Params structures."""
    raw = params_dev.cpu().numpy().tobytes()
    sz = C.sizeof(Params)
    return [Params.from_buffer_copy(raw[i * sz:(i + 1) * sz]) for i in range(len(raw) // sz)]


def tq_compress_device_params(grad: torch.Tensor, params_dev: torch.Tensor, num_levels: int, mode: int, seed: int,
                              first_worker: int = 0, d: Optional[int] = None, packed: Optional[torch.Tensor] = None,
                              stream=None) -> torch.Tensor:
    n, d, stride = _grad_layout(grad, d)
    bits = {2: 1, 4: 2, 8: 3, 16: 4}[num_levels]
    if packed is None:
        packed = torch.empty((n, tq_packed_words(d, bits)), dtype=torch.int32, device=grad.device)
    words_stride = packed.stride(0) if packed.dim() == 2 and n > 1 else packed.shape[-1]
    _check(lib().tq_compress_device_params(grad.data_ptr(), _dtype_code(grad), d, stride, n, params_dev.data_ptr(),
                                           num_levels, mode, seed & 0xFFFFFFFFFFFFFFFF, first_worker, packed.data_ptr(),
                                           words_stride, _stream(stream)), "tq_compress_device_params")
    return packed


def tq_decompress_aggregate_device_params(packed: torch.Tensor, d: int, params_dev: torch.Tensor, num_levels: int,
                                          weights: Optional[Sequence[float]] = None,
                                          out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    n = packed.shape[0]
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=packed.device)
    w = None if weights is None else (C.c_float * n)(*[float(x) for x in weights])
    words_stride = packed.stride(0) if n > 1 else packed.shape[1]
    _check(lib().tq_decompress_aggregate_device_params(packed.data_ptr(), words_stride, n, d, params_dev.data_ptr(),
                                                       num_levels, w, out.data_ptr(), _stream(stream)),
           "tq_decompress_aggregate_device_params")
    return out


def segments_array(segments: Sequence[Tuple[int, int]]):
    """A tq_segment_t[n] from (offset, length) pairs."""
    return (Segment * len(segments))(*[Segment(int(o), int(n)) for o, n in segments])


def tq_segments_packed_words(segments, bits: int) -> int:
    seg = segments if isinstance(segments, C.Array) else segments_array(segments)
    return int(lib().tq_segments_packed_words(seg, len(seg), bits))


def tq_stats_segments(grad: torch.Tensor, segments, g_min: float = 0.0, kappa: float = 1.0,
                      stats_dev: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    """One record per (worker, segment), index worker * n_segments + segment; returns the device records."""
    n, _, stride = _grad_layout(grad, None)
    seg = segments if isinstance(segments, C.Array) else segments_array(segments)
    jobs = n * len(seg)
    if stats_dev is None:
        stats_dev = torch.empty(jobs * C.sizeof(Stats), dtype=torch.uint8, device=grad.device)
    if workspace is None:
        workspace = torch.empty(tq_stats_workspace_bytes(jobs), dtype=torch.uint8, device=grad.device)
    _check(lib().tq_stats_segments(grad.data_ptr(), _dtype_code(grad), stride, n, seg, len(seg), g_min, kappa,
                                   stats_dev.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream(stream)),
           "tq_stats_segments")
    return stats_dev


def tq_stats_hinted_segments(grad: torch.Tensor, segments, hint: torch.Tensor, kappa: float = 1.0,
                             stats_dev: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                             stream=None) -> torch.Tensor:
    """tq_stats_hinted for every (worker, segment) pair; `hint` = new_gmin_hint(n_workers * n_segments), kept across rounds."""
    n, _, stride = _grad_layout(grad, None)
    seg = segments if isinstance(segments, C.Array) else segments_array(segments)
    jobs = n * len(seg)
    if stats_dev is None:
        stats_dev = torch.empty(jobs * C.sizeof(Stats), dtype=torch.uint8, device=grad.device)
    if workspace is None:
        workspace = torch.empty(tq_stats_workspace_bytes(jobs), dtype=torch.uint8, device=grad.device)
    _check(lib().tq_stats_hinted_segments(grad.data_ptr(), _dtype_code(grad), stride, n, seg, len(seg), kappa, hint.data_ptr(),
                                          stats_dev.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream(stream)),
           "tq_stats_hinted_segments")
    return stats_dev


def tq_compress_segments(grad: torch.Tensor, segments, params_dev: torch.Tensor, num_levels: int, mode: int, seed: int,
                         first_worker: int = 0, packed: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    n, _, stride = _grad_layout(grad, None)
    seg = segments if isinstance(segments, C.Array) else segments_array(segments)
    bits = {2: 1, 4: 2, 8: 3, 16: 4}[num_levels]
    if packed is None:
        packed = torch.empty((n, tq_segments_packed_words(seg, bits)), dtype=torch.int32, device=grad.device)
    words_stride = packed.stride(0) if packed.dim() == 2 and n > 1 else packed.shape[-1]
    _check(lib().tq_compress_segments(grad.data_ptr(), _dtype_code(grad), stride, n, seg, len(seg), params_dev.data_ptr(),
                                      num_levels, mode, seed & 0xFFFFFFFFFFFFFFFF, first_worker, packed.data_ptr(),
                                      words_stride, _stream(stream)), "tq_compress_segments")
    return packed


def tq_decompress_aggregate_segments(packed: torch.Tensor, segments, params_dev: torch.Tensor, num_levels: int,
                                     out: torch.Tensor, weights: Optional[Sequence[float]] = None, stream=None) -> torch.Tensor:
    """Aggregates every segment into out[offset : offset + length]; elements of `out` outside the segments are left alone."""
    n = packed.shape[0]
    seg = segments if isinstance(segments, C.Array) else segments_array(segments)
    w = None if weights is None else (C.c_float * n)(*[float(x) for x in weights])
    words_stride = packed.stride(0) if n > 1 else packed.shape[1]
    _check(lib().tq_decompress_aggregate_segments(packed.data_ptr(), words_stride, n, seg, len(seg), params_dev.data_ptr(),
                                                  num_levels, w, out.data_ptr(), _stream(stream)),
           "tq_decompress_aggregate_segments")
    return out


def tq_decompress_aggregate_apply(packed: torch.Tensor, d: int, params, theta: torch.Tensor,
                                  momentum_buf: Optional[torch.Tensor], lr: float, momentum: float = 0.0,
                                  weight_decay: float = 0.0, weights: Optional[Sequence[float]] = None, stream=None):
    """Aggregate the N packed rows and apply the SGD step in place on ``theta`` (and ``momentum_buf``)."""
    n = packed.shape[0]
    w = None if weights is None else (C.c_float * n)(*[float(x) for x in weights])
    words_stride = packed.stride(0) if n > 1 else packed.shape[1]
    _check(lib().tq_decompress_aggregate_apply(packed.data_ptr(), words_stride, n, d, _params_array(params), w,
                                               theta.data_ptr(), None if momentum_buf is None else momentum_buf.data_ptr(),
                                               lr, momentum, weight_decay, _stream(stream)), "tq_decompress_aggregate_apply")
    return theta


def tq_kernel_launches() -> int:
    return int(lib().tq_kernel_launches())


def tq_wait_expired_count() -> int:
    """Give-ups of bounded barrier waits inside the library's kernels on the current device (0 when healthy)."""
    n = C.c_uint32(0)
    _check(lib().tq_wait_expired_count(C.byref(n)), "tq_wait_expired_count")
    return int(n.value)
