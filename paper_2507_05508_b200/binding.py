"""ctypes binding of libmlmc.so: argument marshalling only.

Every function has the name and the argument order of its C entry point in include/mlmc.h; torch
tensors are passed as raw device pointers and the current torch CUDA stream as the stream.  There is
no CPU path: if the CUDA library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmlmc.so")

MLMC_F32, MLMC_BF16 = 0, 1
MLMC_TOPK, MLMC_BITWISE, MLMC_RTN = 0, 1, 2
MLMC_OK = 0
MLMC_ERR_ARG, MLMC_ERR_SCHEDULE, MLMC_ERR_PROB, MLMC_ERR_CAPACITY = -1, -2, -3, -4
MLMC_ERR_NONFINITE, MLMC_ERR_TIMEOUT, MLMC_ERR_CUDA, MLMC_ERR_NOMEM, MLMC_ERR_INTERNAL = -5, -6, -7, -8, -9
MLMC_MAX_LEVELS = 32

EXPORTS = ["mlmc_create", "mlmc_destroy", "mlmc_get_status", "mlmc_launch_count", "mlmc_read_u", "mlmc_read_listed_tiles",
           "mlmc_read_bracket_stats",
           "mlmc_kernel_count", "mlmc_kernel_name", "mlmc_timing_enable", "mlmc_timing_read",
           "mlmc_level_probs", "mlmc_compress_topk", "mlmc_compress_bitwise", "mlmc_aggregate",
           "mlmc_aggregate_topk_noalloc", "mlmc_compress_stopk", "mlmc_compress_floatbits", "mlmc_aggregate_floatbits",
           "mlmc_compress_rtn", "mlmc_aggregate_rtn"]


class MlmcError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where} returned status {code}")
        self.code = code


class mlmc_topk_msgs(C.Structure):
    _fields_ = [("idx", C.c_void_p), ("val", C.c_void_p), ("count", C.c_void_p), ("level", C.c_void_p),
                ("p_sel", C.c_void_p), ("capacity", C.c_int64)]


class mlmc_bit_msgs(C.Structure):
    _fields_ = [("planes", C.c_void_p), ("gmax", C.c_void_p), ("level", C.c_void_p), ("p_sel", C.c_void_p),
                ("w_max", C.c_int32)]


class mlmc_float_msgs(C.Structure):
    _fields_ = [("expo", C.c_void_p), ("planes", C.c_void_p), ("level", C.c_void_p), ("p_sel", C.c_void_p),
                ("w_max", C.c_int32)]


class mlmc_rtn_msgs(C.Structure):
    _fields_ = [("val", C.c_void_p), ("c", C.c_void_p), ("level", C.c_void_p), ("p_sel", C.c_void_p),
                ("ldv", C.c_int64)]


_lib = None


def lib() -> C.CDLL:
    """The CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2507_05508_b200.build` "
                                    "(or __graft_entry__.build()) first; there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64 = C.c_void_p, C.c_int, C.c_int64, C.c_uint64
        L.mlmc_create.argtypes = [C.POINTER(vp), i32, i64, i32, i32]
        L.mlmc_destroy.argtypes = [vp]
        L.mlmc_get_status.argtypes = [vp, vp]
        L.mlmc_launch_count.argtypes = [vp]
        L.mlmc_launch_count.restype = i64
        L.mlmc_read_u.argtypes = [vp, u64, u64, i32, vp, vp]
        L.mlmc_read_listed_tiles.argtypes = [vp, i32, vp, vp, vp]
        L.mlmc_read_bracket_stats.argtypes = [vp, vp, vp]
        L.mlmc_level_probs.argtypes = [vp, vp, i32, i64, i32, i64, i32, vp, i32, vp, vp, vp, vp]
        L.mlmc_compress_topk.argtypes = [vp, vp, i32, i64, i32, i64, vp, i32, vp, u64, u64, vp, vp]
        L.mlmc_compress_bitwise.argtypes = [vp, vp, i32, i64, i32, i64, vp, i32, vp, u64, u64, vp, vp]
        L.mlmc_aggregate.argtypes = [vp, i32, vp, vp, i32, i32, i64, vp, vp]
        L.mlmc_aggregate_topk_noalloc.argtypes = [vp, i32, i64, vp, vp]
        L.mlmc_compress_stopk.argtypes = [vp, vp, i32, i64, i32, i64, i64, vp, u64, u64, vp, vp]
        L.mlmc_compress_floatbits.argtypes = [vp, vp, i32, i64, i32, i64, vp, i32, vp, u64, u64, vp, vp]
        L.mlmc_aggregate_floatbits.argtypes = [vp, vp, vp, i32, i32, i64, vp, vp]
        L.mlmc_compress_rtn.argtypes = [vp, vp, i32, i64, i32, i64, vp, i32, vp, u64, u64, vp, vp]
        L.mlmc_aggregate_rtn.argtypes = [vp, vp, i32, i64, vp, vp]
        L.mlmc_kernel_count.argtypes = []
        L.mlmc_kernel_name.argtypes = [i32]
        L.mlmc_timing_enable.argtypes = [vp, i32]
        L.mlmc_timing_read.argtypes = [vp, vp, vp, vp]
        for name in EXPORTS:
            if name not in ("mlmc_launch_count", "mlmc_kernel_name"):
                getattr(L, name).restype = i32
        L.mlmc_kernel_name.restype = C.c_char_p
        _lib = L
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(g: torch.Tensor) -> int:
    if g.dtype == torch.float32:
        return MLMC_F32
    if g.dtype == torch.bfloat16:
        return MLMC_BF16
    raise TypeError("gradients must be float32 or bfloat16")


def _check(rc: int, where: str) -> None:
    if rc != MLMC_OK:
        raise MlmcError(rc, where)


def _host_array(ctype, values: Optional[Sequence]):
    if values is None:
        return None
    return (ctype * len(values))(*values)


def mlmc_create(device: int, d_max: int, M_max: int, L_max: int) -> C.c_void_p:
    ctx = C.c_void_p()
    _check(lib().mlmc_create(C.byref(ctx), device, d_max, M_max, L_max), "mlmc_create")
    return ctx


def mlmc_destroy(ctx) -> None:
    _check(lib().mlmc_destroy(ctx), "mlmc_destroy")


def mlmc_get_status(ctx) -> int:
    return int(lib().mlmc_get_status(ctx, _stream()))


def mlmc_launch_count(ctx) -> int:
    return int(lib().mlmc_launch_count(ctx))


def mlmc_kernel_count() -> int:
    return int(lib().mlmc_kernel_count())


def mlmc_kernel_name(i: int) -> str:
    return lib().mlmc_kernel_name(i).decode()


def mlmc_timing_enable(ctx, on: bool) -> None:
    _check(lib().mlmc_timing_enable(ctx, 1 if on else 0), "mlmc_timing_enable")


def mlmc_timing_read(ctx):
    """{kernel name: (total ms, launches)} recorded since the previous read (synchronises the stream)."""
    n = mlmc_kernel_count()
    ms, cnt = (C.c_double * n)(), (C.c_int64 * n)()
    _check(lib().mlmc_timing_read(ctx, ms, cnt, _stream()), "mlmc_timing_read")
    return {mlmc_kernel_name(i): (ms[i], cnt[i]) for i in range(n) if cnt[i]}


def mlmc_read_u(ctx, seed: int, step: int, M: int):
    buf = (C.c_double * M)()
    _check(lib().mlmc_read_u(ctx, seed, step, M, buf, _stream()), "mlmc_read_u")
    return list(buf)


def mlmc_read_listed_tiles(ctx, M: int):
    """(tiles read per worker by the last Top-k emission, tiles per row)."""
    buf = (C.c_uint32 * M)()
    tiles = C.c_int64(0)
    _check(lib().mlmc_read_listed_tiles(ctx, M, buf, C.byref(tiles), _stream()), "mlmc_read_listed_tiles")
    return list(buf), int(tiles.value)


def mlmc_read_bracket_stats(ctx):
    """(workers whose brackets held, workers with a missed bracket, workers without a stored bin), cumulative."""
    buf = (C.c_uint64 * 3)()
    _check(lib().mlmc_read_bracket_stats(ctx, buf, _stream()), "mlmc_read_bracket_stats")
    return tuple(int(x) for x in buf)


def _g_args(g: torch.Tensor):
    assert g.is_cuda and g.dim() == 2 and g.stride(1) == 1
    return g.data_ptr(), _dtype_code(g), g.shape[1], g.shape[0], g.stride(0)


def mlmc_level_probs(ctx, g: torch.Tensor, kind: int, sched: Sequence[int], p: Optional[Sequence[float]],
                     p_out: torch.Tensor, delta_out: Optional[torch.Tensor]) -> None:
    ptr, dt, d, M, ld = _g_args(g)
    sch = _host_array(C.c_int64, list(sched))
    ph = _host_array(C.c_double, None if p is None else list(p))
    L = len(sched) + (1 if kind == MLMC_RTN else 0)      # the RTN schedule lists the widths below the identity level
    _check(lib().mlmc_level_probs(ctx, ptr, dt, d, M, ld, kind, sch, L, ph, p_out.data_ptr(),
                                  None if delta_out is None else delta_out.data_ptr(), _stream()), "mlmc_level_probs")


def mlmc_compress_topk(ctx, g: torch.Tensor, k: Sequence[int], p: Optional[Sequence[float]], seed: int, step: int,
                       out: "TopkBuffers") -> None:
    ptr, dt, d, M, ld = _g_args(g)
    kh = _host_array(C.c_int64, list(k))
    ph = _host_array(C.c_double, None if p is None else list(p))
    _check(lib().mlmc_compress_topk(ctx, ptr, dt, d, M, ld, kh, len(k), ph, seed, step, C.byref(out.struct),
                                    _stream()), "mlmc_compress_topk")


def mlmc_compress_bitwise(ctx, g: torch.Tensor, b: Sequence[int], p: Optional[Sequence[float]], seed: int, step: int,
                          out: "BitBuffers") -> None:
    ptr, dt, d, M, ld = _g_args(g)
    bh = _host_array(C.c_int32, list(b))
    ph = _host_array(C.c_double, None if p is None else list(p))
    _check(lib().mlmc_compress_bitwise(ctx, ptr, dt, d, M, ld, bh, len(b), ph, seed, step, C.byref(out.struct),
                                       _stream()), "mlmc_compress_bitwise")


def mlmc_aggregate(ctx, kind: int, msgs, b: Optional[Sequence[int]], M: int, d: int, out: torch.Tensor) -> None:
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.numel() >= d
    bh = _host_array(C.c_int32, None if b is None else list(b))
    _check(lib().mlmc_aggregate(ctx, kind, C.byref(msgs.struct), bh, 0 if b is None else len(b), M, d,
                                out.data_ptr(), _stream()), "mlmc_aggregate")


def mlmc_aggregate_topk_noalloc(msgs: "TopkBuffers", M: int, d: int, out: torch.Tensor) -> None:
    """Top-k server average that needs no context and allocates nothing (fixed built-in scratch; see mlmc.h)."""
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.numel() >= d
    _check(lib().mlmc_aggregate_topk_noalloc(C.byref(msgs.struct), M, d, out.data_ptr(), _stream()),
           "mlmc_aggregate_topk_noalloc")


def mlmc_compress_stopk(ctx, g: torch.Tensor, s: int, p: Optional[Sequence[float]], seed: int, step: int,
                        out: "TopkBuffers") -> None:
    ptr, dt, d, M, ld = _g_args(g)
    ph = None if p is None else (C.c_double * len(p)).from_buffer_copy(memoryview(_as_f64(p)))
    _check(lib().mlmc_compress_stopk(ctx, ptr, dt, d, M, ld, s, ph, seed, step, C.byref(out.struct), _stream()),
           "mlmc_compress_stopk")


def _as_f64(p):
    import numpy as np
    return np.ascontiguousarray(p, dtype=np.float64)


def mlmc_compress_floatbits(ctx, g: torch.Tensor, mb: Sequence[int], p: Optional[Sequence[float]], seed: int, step: int,
                            out: "FloatBuffers") -> None:
    ptr, dt, d, M, ld = _g_args(g)
    mh = _host_array(C.c_int32, list(mb))
    ph = _host_array(C.c_double, None if p is None else list(p))
    _check(lib().mlmc_compress_floatbits(ctx, ptr, dt, d, M, ld, mh, len(mb), ph, seed, step, C.byref(out.struct),
                                         _stream()), "mlmc_compress_floatbits")


def mlmc_aggregate_floatbits(ctx, msgs: "FloatBuffers", mb: Sequence[int], M: int, d: int, out: torch.Tensor) -> None:
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.numel() >= d
    mh = _host_array(C.c_int32, list(mb))
    _check(lib().mlmc_aggregate_floatbits(ctx, C.byref(msgs.struct), mh, len(mb), M, d, out.data_ptr(), _stream()),
           "mlmc_aggregate_floatbits")


def mlmc_compress_rtn(ctx, g: torch.Tensor, r: Sequence[int], p: Optional[Sequence[float]], seed: int, step: int,
                      out: "RtnBuffers") -> None:
    """r: the L - 1 round-to-nearest widths; level L - 1 is the identity."""
    ptr, dt, d, M, ld = _g_args(g)
    rh = _host_array(C.c_int32, list(r)) if len(r) else None
    ph = _host_array(C.c_double, None if p is None else list(p))
    _check(lib().mlmc_compress_rtn(ctx, ptr, dt, d, M, ld, rh, len(r) + 1, ph, seed, step, C.byref(out.struct),
                                   _stream()), "mlmc_compress_rtn")


def mlmc_aggregate_rtn(ctx, msgs: "RtnBuffers", M: int, d: int, out: torch.Tensor) -> None:
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.numel() >= d
    _check(lib().mlmc_aggregate_rtn(ctx, C.byref(msgs.struct), M, d, out.data_ptr(), _stream()), "mlmc_aggregate_rtn")


class FloatBuffers:
    """Caller-owned device buffers of a floating-point message batch."""

    def __init__(self, M: int, d: int, w_max: int, device: str = "cuda"):
        self.M, self.d, self.w_max = M, d, w_max
        self.words = (d + 31) // 32
        self.expo = torch.zeros((M, self.words * 32), dtype=torch.uint8, device=device)
        self.planes = torch.zeros((M, 1 + w_max, self.words), dtype=torch.int32, device=device)  # uint32 payload
        self.level = torch.full((M,), -1, dtype=torch.int32, device=device)
        self.p_sel = torch.zeros(M, dtype=torch.float64, device=device)
        self.struct = mlmc_float_msgs(self.expo.data_ptr(), self.planes.data_ptr(), self.level.data_ptr(),
                                      self.p_sel.data_ptr(), w_max)


class RtnBuffers:
    """Caller-owned device buffers of a dense MLMC-RTN message batch (rows padded to 16 bytes)."""

    def __init__(self, M: int, d: int, device: str = "cuda"):
        self.M, self.d = M, d
        self.ldv = (d + 3) // 4 * 4
        self.val = torch.zeros((M, self.ldv), dtype=torch.float32, device=device)
        self.c = torch.zeros(M, dtype=torch.float32, device=device)
        self.level = torch.full((M,), -1, dtype=torch.int32, device=device)
        self.p_sel = torch.zeros(M, dtype=torch.float64, device=device)
        self.struct = mlmc_rtn_msgs(self.val.data_ptr(), self.c.data_ptr(), self.level.data_ptr(),
                                    self.p_sel.data_ptr(), self.ldv)


class TopkBuffers:
    """Caller-owned device buffers of a Top-k message batch (torch only provides the memory)."""

    def __init__(self, M: int, capacity: int, device: str = "cuda"):
        self.M, self.capacity = M, capacity
        self.idx = torch.empty((M, max(capacity, 1)), dtype=torch.int32, device=device)   # uint32 payload
        self.val = torch.empty((M, max(capacity, 1)), dtype=torch.float32, device=device)
        self.count = torch.zeros(M, dtype=torch.int64, device=device)
        self.level = torch.full((M,), -1, dtype=torch.int32, device=device)
        self.p_sel = torch.zeros(M, dtype=torch.float64, device=device)
        self.struct = mlmc_topk_msgs(self.idx.data_ptr(), self.val.data_ptr(), self.count.data_ptr(),
                                     self.level.data_ptr(), self.p_sel.data_ptr(), capacity)


class BitBuffers:
    """Caller-owned device buffers of a bit-plane message batch."""

    def __init__(self, M: int, d: int, w_max: int, device: str = "cuda"):
        self.M, self.d, self.w_max = M, d, w_max
        self.words = (d + 31) // 32
        self.planes = torch.zeros((M, 1 + w_max, self.words), dtype=torch.int32, device=device)  # uint32 payload
        self.gmax = torch.zeros(M, dtype=torch.float32, device=device)
        self.level = torch.full((M,), -1, dtype=torch.int32, device=device)
        self.p_sel = torch.zeros(M, dtype=torch.float64, device=device)
        self.struct = mlmc_bit_msgs(self.planes.data_ptr(), self.gmax.data_ptr(), self.level.data_ptr(),
                                    self.p_sel.data_ptr(), w_max)
