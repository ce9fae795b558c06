"""CPU-side checks: the C-ABI library loads and exports what include/*.h declare; workload generators."""
import ctypes
import os
import re

import numpy as np

from paper_2507_05508_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    inc = os.path.join(ROOT, "include")
    text = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mlmc_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2507_05508_b200 import build, binding
    lib = ctypes.CDLL(build.build())
    names = _declared_functions()
    assert set(binding.EXPORTS) == set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_argument_checks_without_a_gpu():
    # host-side validation happens before any CUDA call: null context / bad sizes come back as MLMC_ERR_ARG
    from paper_2507_05508_b200 import binding as B
    lib = B.lib()
    assert lib.mlmc_destroy(None) == B.MLMC_ERR_ARG
    assert lib.mlmc_get_status(None, None) == B.MLMC_ERR_ARG
    ctx = ctypes.c_void_p()
    assert lib.mlmc_create(ctypes.byref(ctx), 0, 0, 1, 1) == B.MLMC_ERR_ARG
    assert lib.mlmc_create(ctypes.byref(ctx), 0, 1 << 32, 1, 1) == B.MLMC_ERR_ARG
    assert lib.mlmc_create(ctypes.byref(ctx), 0, 100, 1, 33) == B.MLMC_ERR_ARG
    assert lib.mlmc_compress_topk(None, None, 0, 1, 1, 1, None, 1, None, 0, 0, None, None) == B.MLMC_ERR_ARG
    assert lib.mlmc_aggregate(None, 0, None, None, 0, 1, 1, None, None) == B.MLMC_ERR_ARG


def test_schedules_match_the_configs():
    assert wl.topk_schedule(wl.C1) == [64 * 2**l for l in range(10)] + [65536]
    k3 = wl.topk_schedule(wl.C3)
    assert len(k3) == 11 and k3[0] == 11689 and k3[1] == 23379 and k3[9] == 5_985_030 and k3[-1] == wl.C3.d
    k4 = wl.topk_schedule(wl.C4)
    assert len(k4) == 12 and k4[0] == 12778 and k4[10] == 13_085_200 and wl.max_band(k4) == 12_471_832
    k5 = wl.topk_schedule(wl.C5A)
    assert len(k5) == 15 and k5[0] == 12443 and k5[13] == 101_941_090 and wl.max_band(k5) == 50_970_545
    p = wl.geometric_probs(11)
    assert abs(p.sum() - 1) < 1e-15 and np.allclose(p[:-1] / p[1:], 2.0)


def test_generators_are_seeded_and_structured():
    w = wl.shrink(wl.C3, 50_000, 3)
    a, b = wl.gradients(w, 2), wl.gradients(w, 2)
    assert a.shape == (3, 50_000) and (a == b).all() and not (a == wl.gradients(w, 3)).all()
    s = wl.scales(w)
    assert len(np.unique(s.numpy())) == w.segments and s.min() >= 1e-4 and s.max() <= 1e-1
    w5 = wl.shrink(wl.C5A, 100_000, 2)
    s5 = wl.scales(w5).numpy()
    assert (s5 > 0.1).sum() >= 50           # the x100 outlier coordinates
    w4 = wl.shrink(wl.C4, 10_000, 2)
    g4 = wl.gradients(w4, 0)
    assert g4.dtype.is_floating_point and g4.element_size() == 2 and wl.as_numpy_bits(g4).dtype == np.uint16
