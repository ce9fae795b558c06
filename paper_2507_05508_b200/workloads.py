"""Seeded synthetic gradient workloads and level schedules.

This module holds input generation only: configs, level schedules and random gradients.  None of
the method's arithmetic (ranking, level draws, quantisation, averaging) lives here, so both the
CUDA path and the CPU oracle can be fed from it.

The five workloads stand in for the gradients of the paper's experiments (Sec. 5: a ~1.1e8
parameter transformer and a ~1.1e7 parameter ResNet, M in {4, 32}), whose datasets and weights
are not available: only the sizes, the layer-segment structure and heavy-tailed value
distributions are kept.

Recipe: scales are a function of the config seed alone (same for every worker and step);
noise is drawn from a torch.Generator on the target device seeded by (config seed, step), so a
buffer is reproducible on a given device type.  The generated buffer is the input for both
sides of every parity test.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str                 # "topk" | "bitwise" | "floatbits" | "rtn" | "stopk"
    d: int
    M: int
    dtype: str                # "f32" | "bf16"
    adaptive: bool
    seed: int
    steps: int
    dist: str                 # "normal" | "student_t3"
    scale_kind: str           # "coord_loguniform" | "const" | "segments"
    scale_lo: float = 1.0
    scale_hi: float = 1.0
    segments: int = 0
    outlier_frac: float = 0.0
    outlier_mult: float = 1.0
    k_base: int = 0           # topk: k_l = k_base * 2^l            (when k_den == 0)
    k_den: int = 0            # topk: k_l = min(d, floor(d * 2^l / k_den))
    bits: tuple = ()          # bitwise: b_l;  floatbits: mantissa digits mb_l;  rtn: widths r_l (identity level implied)
    seg_len: int = 0          # stopk: segment length s


C1 = Workload("c1", "topk", 65_536, 4, "f32", False, 0, 10, "normal", "coord_loguniform", 1e-3, 1.0, k_base=64)
C2 = Workload("c2", "bitwise", 1_048_576, 8, "f32", False, 1, 20, "student_t3", "const", 1e-2, 1e-2,
              bits=(1, 2, 4, 8, 16, 23))
C3 = Workload("c3", "topk", 11_689_512, 16, "f32", False, 2, 20, "normal", "segments", 1e-4, 1e-1, segments=62,
              k_den=1000)
C4 = Workload("c4", "topk", 25_557_032, 32, "bf16", True, 3, 20, "student_t3", "segments", 1e-4, 1e-1,
              segments=161, k_den=2000)
C5A = Workload("c5a", "topk", 124_439_808, 8, "f32", True, 4, 10, "normal", "segments", 1e-5, 1e-1, segments=148,
               outlier_frac=1e-3, outlier_mult=100.0, k_den=10000)
C5B = replace(C5A, name="c5b", kind="bitwise", k_den=0, bits=(1, 2, 4, 8, 16, 23))

# The further compressors of the paper on the same synthetic gradients (not among the five benchmark configurations: measured beside them).
C5F = replace(C5A, name="c5f", kind="floatbits", adaptive=False, k_den=0, bits=(1, 2, 4, 8, 16, 23))   # App. B, fixed p
C5R = replace(C5A, name="c5r", kind="rtn", k_den=0, bits=(2, 4, 8, 16))                                # App. G, adaptive
C3S = replace(C3, name="c3s", kind="stopk", k_den=0, seg_len=11_690)                                   # App. D, L = 1000, fixed p

C3A = replace(C3, name="c3a", kind="stopk", adaptive=True, k_den=0, seg_len=116_896)                  # App. D, L = 100, adaptive p

ALL = {w.name: w for w in (C1, C2, C3, C4, C5A, C5B, C5F, C5R, C3S, C3A)}


def shrink(w: Workload, d: int, M: Optional[int] = None) -> Workload:
    """Same structure at a smaller gradient length (for cases the oracle finishes in seconds)."""
    segs = min(w.segments, max(1, d // 8)) if w.segments else 0
    return replace(w, name=f"{w.name}_d{d}", d=d, M=M or w.M, segments=segs)


def topk_schedule(w: Workload) -> List[int]:
    """Nondecreasing k_0..k_{L-1} with k_{L-1} = d, in exact integer arithmetic."""
    ks: List[int] = []
    l = 0
    while True:
        k = (w.d * (1 << l)) // w.k_den if w.k_den else w.k_base * (1 << l)
        if k >= w.d:
            ks.append(w.d)
            return ks
        ks.append(max(k, 0))
        l += 1


def geometric_probs(L: int) -> np.ndarray:
    """p_l proportional to 2^-l, normalised in fp64."""
    p = np.ldexp(1.0, -np.arange(L))
    return p / p.sum()


def max_band(ks: List[int]) -> int:
    return int(np.max(np.diff(np.concatenate([[0], np.asarray(ks, dtype=np.int64)]))))


def _segment_lengths(d: int, n: int, gen: torch.Generator) -> np.ndarray:
    """Largest-remainder rounding of d * w_s / sum(w), w_s log-uniform in [1, 1e4], each length >= 1."""
    wts = np.power(10.0, 4.0 * torch.rand(n, generator=gen, dtype=torch.float64).numpy())
    raw = d * wts / wts.sum()
    base = np.maximum(np.floor(raw).astype(np.int64), 1)
    rem = d - int(base.sum())
    order = np.argsort(-(raw - np.floor(raw)), kind="stable")
    i = 0
    while rem != 0:
        j = order[i % n]
        if rem > 0:
            base[j] += 1
            rem -= 1
        elif base[j] > 1:
            base[j] -= 1
            rem += 1
        i += 1
    return base


def scales(w: Workload, device: str = "cpu") -> torch.Tensor:
    """Per-coordinate fp32 scale vector [d]; depends on the config seed only."""
    gen = torch.Generator().manual_seed(1_000_003 * w.seed + 17)
    if w.scale_kind == "const":
        s = torch.full((w.d,), w.scale_lo, dtype=torch.float32)
    elif w.scale_kind == "coord_loguniform":
        lo, hi = np.log10(w.scale_lo), np.log10(w.scale_hi)
        s = torch.pow(10.0, lo + (hi - lo) * torch.rand(w.d, generator=gen, dtype=torch.float64)).float()
    elif w.scale_kind == "segments":
        lens = _segment_lengths(w.d, w.segments, gen)
        lo, hi = np.log10(w.scale_lo), np.log10(w.scale_hi)
        seg = torch.pow(10.0, lo + (hi - lo) * torch.rand(w.segments, generator=gen, dtype=torch.float64)).float()
        s = torch.repeat_interleave(seg, torch.from_numpy(lens))
    else:
        raise ValueError(w.scale_kind)
    s = s.to(device)
    if w.outlier_frac > 0:
        n_out = max(1, int(round(w.outlier_frac * w.d)))
        pos = torch.randint(0, w.d, (n_out,), generator=gen)
        s[pos.to(device)] *= w.outlier_mult
    return s


def gradients(w: Workload, step: int, device: str = "cpu", scale: Optional[torch.Tensor] = None) -> torch.Tensor:
    """[M, d] gradient batch for one step: fp32, or bf16 (round-to-nearest-even of the fp32 sample)."""
    if scale is None:
        scale = scales(w, device)
    gen = torch.Generator(device=device).manual_seed((w.seed * 7_919 + step) * 2_654_435_761 % (2**63 - 1))
    out = torch.empty((w.M, w.d), dtype=torch.bfloat16 if w.dtype == "bf16" else torch.float32, device=device)
    for m in range(w.M):  # row by row keeps the temporaries at a few vectors
        z = torch.randn(w.d, generator=gen, device=device, dtype=torch.float32)
        if w.dist == "student_t3":
            chi = torch.zeros_like(z)
            for _ in range(3):
                y = torch.randn(w.d, generator=gen, device=device, dtype=torch.float32)
                chi.addcmul_(y, y)
            z = z / torch.sqrt(chi / 3.0)
        out[m] = (z * scale).to(out.dtype)
    return out


def as_numpy_bits(g: torch.Tensor) -> np.ndarray:
    """Host view the oracle accepts: float32 array, or uint16 array of bf16 bit patterns."""
    g = g.detach().cpu().contiguous()
    if g.dtype == torch.bfloat16:
        return g.view(torch.int16).numpy().view(np.uint16)
    return g.numpy()
