"""The allocation-free Top-k average against the regular one (collected last on purpose).

Some callers cannot create an mlmc_ctx because that calls cudaMalloc: a serving process whose
framework has already taken the whole GPU for its pool, or code running where the allocator must not
be entered.  mlmc_aggregate_topk_noalloc serves them from a scratch table built into the library.
It launches the same kernels as mlmc_aggregate, so the two results must agree bit for bit; the check
runs on two calls in a row with different messages, since every call reuses the same table.  The result
is also held against the CPU oracle's fp64 average of the same messages (Alg. 2, "Server aggregates").
"""
import numpy as np
import pytest
import torch

from paper_2507_05508_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_noalloc_aggregate_matches_context_aggregate_twice(ora):
    from paper_2507_05508_b200 import binding as B
    B.lib()
    torch.cuda.set_device(0)
    ctx = B.mlmc_create(0, 1_000_004, 6, 32)
    try:
        first = wl.shrink(wl.C3, 1_000_004, 6)      # ragged length, several hundred output tiles
        second = wl.shrink(wl.C5A, 300_004, 3)      # smaller second call: stale entries of the first must not leak
        for call, (w, probs) in enumerate(((first, "fixed"), (second, None))):
            k = wl.topk_schedule(w)
            p = list(wl.geometric_probs(len(k))) if probs == "fixed" else None
            g = wl.gradients(w, call, "cuda")
            msgs = B.TopkBuffers(w.M, wl.max_band(k))
            B.mlmc_compress_topk(ctx, g, k, p, 7, call, msgs)
            ref = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
            got = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
            B.mlmc_aggregate(ctx, B.MLMC_TOPK, msgs, None, w.M, w.d, ref)
            B.mlmc_aggregate_topk_noalloc(msgs, w.M, w.d, got)
            assert B.mlmc_get_status(ctx) == 0
            torch.cuda.synchronize()
            assert not torch.isnan(got).any()
            assert torch.equal(got, ref)             # same kernels, same order of additions: tolerance 0 <= 1e-6
            n = msgs.count.tolist()
            host = [(msgs.idx[m, :n[m]].cpu().numpy().view(np.uint32), msgs.val[m, :n[m]].cpu().numpy())
                    for m in range(w.M)]
            mean, scale = ora.aggregate_topk(host, w.d)
            assert np.all(np.abs(got.cpu().numpy().astype(np.float64) - mean) <= 1e-6 * scale + 1e-45)
        # beyond the built-in table (M * (tiles + 1) > 2^20): refused with an argument error, nothing is launched
        import ctypes
        rc = B.lib().mlmc_aggregate_topk_noalloc(ctypes.byref(msgs.struct), 1, (1 << 32) - 1, got.data_ptr(), None)
        assert rc == B.MLMC_ERR_ARG
    finally:
        B.mlmc_destroy(ctx)
