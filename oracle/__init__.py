"""CPU oracle for the MLMC compression hot path: TEST INFRASTRUCTURE ONLY.

ctypes wrapper around ``mlmc_oracle.cpp`` (single-threaded C++17, built by :func:`build`).
Nothing in the product package imports this module; the tests, the smoke check and the
benchmark's CPU-baseline leg do.  Each wrapper only marshals numpy arrays; the arithmetic is
in the C++ file, which cites the passages of the paper it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mlmc_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

F32, BF16 = 0, 1
OK, ERR_ARG, ERR_SCHEDULE, ERR_PROB, ERR_CAPACITY, ERR_NONFINITE = 0, -1, -2, -3, -4, -5


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction) and return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.mlmc_oracle_uniform.restype = C.c_double
        _lib.mlmc_oracle_uniform.argtypes = [C.c_uint64] * 3
        _lib.mlmc_oracle_hash.restype = C.c_uint64
        _lib.mlmc_oracle_hash.argtypes = [C.c_uint64] * 3
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _as_input(g):
    """Accept float32 arrays, or uint16 arrays holding bf16 bit patterns."""
    g = np.ascontiguousarray(g)
    if g.dtype == np.float32:
        return g, F32
    if g.dtype == np.uint16:
        return g, BF16
    raise TypeError("oracle input must be float32 or uint16 (bf16 bits)")


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle status {code}")
        self.code = code


def _check(rc):
    if rc != OK:
        raise OracleError(rc)


def hash64(seed: int, step: int, worker: int) -> int:
    return int(lib().mlmc_oracle_hash(seed, step, worker))


def uniform(seed: int, step: int, worker: int) -> float:
    return float(lib().mlmc_oracle_uniform(seed, step, worker))


def draw(p, u: float):
    p = np.ascontiguousarray(p, dtype=np.float64)
    level, margin = C.c_int(), C.c_double()
    _check(lib().mlmc_oracle_draw(_ptr(p), C.c_int(len(p)), C.c_double(u), C.byref(level), C.byref(margin)))
    return level.value, margin.value


def rank(g):
    g, dt = _as_input(g)
    perm = np.empty(g.size, dtype=np.uint32)
    _check(lib().mlmc_oracle_rank(_ptr(g), C.c_int(dt), C.c_int64(g.size), _ptr(perm)))
    return perm


@dataclass
class TopkMsg:
    level: int
    p_sel: float
    u: float
    margin: float
    p: np.ndarray
    delta: np.ndarray
    idx: np.ndarray
    val: np.ndarray


def topk(g, k, p=None, seed=0, step=0, worker=0, force_level=-1) -> TopkMsg:
    g, dt = _as_input(g)
    d = g.size
    k = np.ascontiguousarray(k, dtype=np.int64)
    L = len(k)
    p_in = None if p is None else np.ascontiguousarray(p, dtype=np.float64)
    p_out, delta = np.empty(L), np.empty(L)
    level, count = C.c_int32(), C.c_int64()
    p_sel, u, margin = C.c_double(), C.c_double(), C.c_double()
    cap = int(np.max(np.diff(np.concatenate([[0], k])))) if L else 0
    idx = np.empty(max(cap, 1), dtype=np.uint32)
    val = np.empty(max(cap, 1), dtype=np.float32)
    _check(lib().mlmc_oracle_topk(
        _ptr(g), C.c_int(dt), C.c_int64(d), _ptr(k), C.c_int(L), _ptr(p_in),
        C.c_uint64(seed), C.c_uint64(step), C.c_uint64(worker), C.c_int(force_level),
        _ptr(p_out), _ptr(delta), C.byref(level), C.byref(p_sel), C.byref(u), C.byref(margin),
        C.byref(count), _ptr(idx), _ptr(val), C.c_int64(idx.size)))
    n = count.value
    return TopkMsg(level.value, p_sel.value, u.value, margin.value, p_out, delta, idx[:n].copy(), val[:n].copy())


def fixed_point_codes(g, B: int):
    g, dt = _as_input(g)
    q = np.empty(g.size, dtype=np.uint32)
    gmax = C.c_float()
    _check(lib().mlmc_oracle_fixed_point_codes(_ptr(g), C.c_int(dt), C.c_int64(g.size), C.c_int(B),
                                               C.byref(gmax), _ptr(q)))
    return gmax.value, q


@dataclass
class BitMsg:
    level: int
    p_sel: float
    u: float
    margin: float
    p: np.ndarray
    delta: np.ndarray
    S: np.ndarray
    gmax: float
    planes: np.ndarray  # [1 + w_level][ceil(d/32)] uint32


def bitwise(g, b, p=None, seed=0, step=0, worker=0, force_level=-1) -> BitMsg:
    g, dt = _as_input(g)
    d = g.size
    b = np.ascontiguousarray(b, dtype=np.int32)
    L = len(b)
    p_in = None if p is None else np.ascontiguousarray(p, dtype=np.float64)
    widths = np.diff(np.concatenate([[0], b]))
    w_max = int(widths.max())
    words = (d + 31) // 32
    planes = np.zeros((1 + w_max, words), dtype=np.uint32)
    p_out, delta, S = np.empty(L), np.empty(L), np.empty(L, dtype=np.uint64)
    level, gmax = C.c_int32(), C.c_float()
    p_sel, u, margin = C.c_double(), C.c_double(), C.c_double()
    _check(lib().mlmc_oracle_bitwise(
        _ptr(g), C.c_int(dt), C.c_int64(d), _ptr(b), C.c_int(L), _ptr(p_in),
        C.c_uint64(seed), C.c_uint64(step), C.c_uint64(worker), C.c_int(force_level),
        _ptr(p_out), _ptr(delta), _ptr(S), C.byref(level), C.byref(p_sel), C.byref(u), C.byref(margin),
        C.byref(gmax), _ptr(planes), C.c_int32(w_max)))
    w = int(widths[level.value])
    return BitMsg(level.value, p_sel.value, u.value, margin.value, p_out, delta, S, gmax.value,
                  planes[:1 + w].copy())


def bitwise_decode(planes, d, b, level, gmax, p_sel):
    planes = np.ascontiguousarray(planes, dtype=np.uint32)
    b = np.ascontiguousarray(b, dtype=np.int32)
    est = np.empty(d, dtype=np.float64)
    _check(lib().mlmc_oracle_bitwise_decode(_ptr(planes), C.c_int64(d), _ptr(b), C.c_int(len(b)),
                                            C.c_int(level), C.c_float(gmax), C.c_double(p_sel), _ptr(est)))
    return est


def aggregate_topk(msgs, d):
    """msgs: list of (idx uint32[n], val float32[n]).  Returns (mean fp64[d], scale fp64[d])."""
    M = len(msgs)
    idxs = [np.ascontiguousarray(i, dtype=np.uint32) for i, _ in msgs]
    vals = [np.ascontiguousarray(v, dtype=np.float32) for _, v in msgs]
    count = np.array([i.size for i in idxs], dtype=np.int64)
    ip = (C.c_void_p * M)(*[i.ctypes.data for i in idxs])
    vp = (C.c_void_p * M)(*[v.ctypes.data for v in vals])
    out, scale = np.empty(d), np.empty(d)
    _check(lib().mlmc_oracle_aggregate_topk(C.c_int(M), _ptr(count), ip, vp, C.c_int64(d), _ptr(out), _ptr(scale)))
    return out, scale


def aggregate_bitwise(msgs, b, d):
    """msgs: list of BitMsg-like objects with planes, gmax, level, p_sel."""
    M = len(msgs)
    b = np.ascontiguousarray(b, dtype=np.int32)
    planes = [np.ascontiguousarray(m.planes, dtype=np.uint32) for m in msgs]
    pp = (C.c_void_p * M)(*[p.ctypes.data for p in planes])
    gmax = np.array([m.gmax for m in msgs], dtype=np.float32)
    level = np.array([m.level for m in msgs], dtype=np.int32)
    p_sel = np.array([m.p_sel for m in msgs], dtype=np.float64)
    out, scale = np.empty(d), np.empty(d)
    _check(lib().mlmc_oracle_aggregate_bitwise(C.c_int(M), pp, _ptr(gmax), _ptr(level), _ptr(p_sel), _ptr(b),
                                               C.c_int(len(b)), C.c_int64(d), _ptr(out), _ptr(scale)))
    return out, scale


# ----------------------------------------------------------------------------------------------
# floating-point bit-wise MLMC (App. B), s-Top-k (App. D), MLMC-RTN (App. G)
# ----------------------------------------------------------------------------------------------
def float_compress(g, keep: int):
    """Dense C(g) that keeps sign, exponent and the first `keep` mantissa digits (fp64 copy)."""
    g, dt = _as_input(g)
    out = np.empty(g.size)
    _check(lib().mlmc_oracle_float_compress(_ptr(g), C.c_int(dt), C.c_int64(g.size), C.c_int(keep), _ptr(out)))
    return out


@dataclass
class FloatMsg:
    level: int
    p_sel: float
    u: float
    margin: float
    p: np.ndarray
    expo: np.ndarray     # uint8[d]
    planes: np.ndarray   # [1 + w_level][ceil(d/32)] uint32
    est: np.ndarray      # fp64[d]: g^0 + (C^l - C^{l-1}) / p_l


def floatbits(g, mb, p=None, seed=0, step=0, worker=0, force_level=-1) -> FloatMsg:
    g, dt = _as_input(g)
    d = g.size
    mb = np.ascontiguousarray(mb, dtype=np.int32)
    L = len(mb)
    p_in = None if p is None else np.ascontiguousarray(p, dtype=np.float64)
    widths = np.diff(np.concatenate([[0], mb]))
    w_max = int(widths.max())
    words = (d + 31) // 32
    planes = np.zeros((1 + w_max, words), dtype=np.uint32)
    expo = np.empty(d, dtype=np.uint8)
    est = np.empty(d)
    p_out = np.empty(L)
    level = C.c_int32()
    p_sel, u, margin = C.c_double(), C.c_double(), C.c_double()
    _check(lib().mlmc_oracle_floatbits(
        _ptr(g), C.c_int(dt), C.c_int64(d), _ptr(mb), C.c_int(L), _ptr(p_in),
        C.c_uint64(seed), C.c_uint64(step), C.c_uint64(worker), C.c_int(force_level),
        _ptr(p_out), C.byref(level), C.byref(p_sel), C.byref(u), C.byref(margin),
        _ptr(expo), _ptr(planes), C.c_int32(w_max), _ptr(est)))
    w = int(widths[level.value])
    return FloatMsg(level.value, p_sel.value, u.value, margin.value, p_out, expo, planes[:1 + w].copy(), est)


def floatbits_decode(expo, planes, d, mb, level, p_sel, bf16=False):
    expo = np.ascontiguousarray(expo, dtype=np.uint8)
    planes = np.ascontiguousarray(planes, dtype=np.uint32)
    mb = np.ascontiguousarray(mb, dtype=np.int32)
    est = np.empty(d)
    _check(lib().mlmc_oracle_floatbits_decode(_ptr(expo), _ptr(planes), C.c_int64(d), C.c_int(BF16 if bf16 else F32),
                                              _ptr(mb), C.c_int(len(mb)), C.c_int(level), C.c_double(p_sel), _ptr(est)))
    return est


def aggregate_dense(rows, d):
    """rows: list of fp64[d] (or fp32) dense estimates.  Returns (mean fp64[d], scale fp64[d])."""
    rows = [np.ascontiguousarray(r, dtype=np.float64) for r in rows]
    M = len(rows)
    rp = (C.c_void_p * M)(*[r.ctypes.data for r in rows])
    out, scale = np.empty(d), np.empty(d)
    _check(lib().mlmc_oracle_aggregate_dense(C.c_int(M), rp, C.c_int64(d), _ptr(out), _ptr(scale)))
    return out, scale


def stopk(g, s: int, p=None, seed=0, step=0, worker=0, force_level=-1) -> TopkMsg:
    g, dt = _as_input(g)
    d = g.size
    L = (d + s - 1) // s
    p_in = None if p is None else np.ascontiguousarray(p, dtype=np.float64)
    p_out, delta = np.empty(L), np.empty(L)
    level, count = C.c_int32(), C.c_int64()
    p_sel, u, margin = C.c_double(), C.c_double(), C.c_double()
    idx = np.empty(s, dtype=np.uint32)
    val = np.empty(s, dtype=np.float32)
    _check(lib().mlmc_oracle_stopk(
        _ptr(g), C.c_int(dt), C.c_int64(d), C.c_int64(s), _ptr(p_in),
        C.c_uint64(seed), C.c_uint64(step), C.c_uint64(worker), C.c_int(force_level),
        _ptr(p_out), _ptr(delta), C.byref(level), C.byref(p_sel), C.byref(u), C.byref(margin),
        C.byref(count), _ptr(idx), _ptr(val), C.c_int64(s)))
    n = count.value
    return TopkMsg(level.value, p_sel.value, u.value, margin.value, p_out, delta, idx[:n].copy(), val[:n].copy())


def rtn_compress(g, r, level: int):
    """Dense C^level(g) for the RTN widths r (len L-1; level L-1 is the identity), fp64."""
    g, dt = _as_input(g)
    r = np.ascontiguousarray(r, dtype=np.int32)
    out = np.empty(g.size)
    _check(lib().mlmc_oracle_rtn_compress(_ptr(g), C.c_int(dt), C.c_int64(g.size), _ptr(r), C.c_int(len(r) + 1),
                                          C.c_int(level), _ptr(out)))
    return out


@dataclass
class RtnMsg:
    level: int
    p_sel: float
    u: float
    margin: float
    p: np.ndarray
    delta: np.ndarray
    c: float
    val: np.ndarray      # float32[d]: (C^l - C^{l-1}) / p_l


def rtn(g, r, p=None, seed=0, step=0, worker=0, force_level=-1) -> RtnMsg:
    g, dt = _as_input(g)
    d = g.size
    r = np.ascontiguousarray(r, dtype=np.int32)
    L = len(r) + 1
    p_in = None if p is None else np.ascontiguousarray(p, dtype=np.float64)
    p_out, delta = np.empty(L), np.empty(L)
    val = np.empty(d, dtype=np.float32)
    level, c = C.c_int32(), C.c_float()
    p_sel, u, margin = C.c_double(), C.c_double(), C.c_double()
    _check(lib().mlmc_oracle_rtn(
        _ptr(g), C.c_int(dt), C.c_int64(d), _ptr(r), C.c_int(L), _ptr(p_in),
        C.c_uint64(seed), C.c_uint64(step), C.c_uint64(worker), C.c_int(force_level),
        _ptr(p_out), _ptr(delta), C.byref(level), C.byref(p_sel), C.byref(u), C.byref(margin), C.byref(c), _ptr(val)))
    return RtnMsg(level.value, p_sel.value, u.value, margin.value, p_out, delta, c.value, val)
