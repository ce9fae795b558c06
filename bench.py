#!/usr/bin/env python
"""Benchmark of the MLMC compress+aggregate hot path.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl reference]

One step = mlmc_compress_* on all M workers + mlmc_aggregate into the dense mean, on one batch of
synthetic gradients already resident in HBM.  The default workload c5 is the 124M-parameter config with
both of its variants per step (adaptive MLMC-Top-k, then adaptive bit-wise MLMC, each a full
compress + aggregate over the same gradient batch).  `value` is gradient GB/s = gradient bytes swept by
the variants (M*d*sizeof(T) each) / step time, summed over ranks (ranks are independent replicas: the
path has no inter-GPU exchange).  On one GPU the default run also times c4, c5a, c5b and c3 for a few steps each
and reports them under `also` in the same line.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "MLMC compress+aggregate gradient GB/s per step (1 B200); fraction of HBM peak"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic_ratios.txt")


def ncu_traffic_ratios():
    """DRAM traffic per launch of a sweep kernel relative to its algorithmic bytes, from the ncu captures summarised
    under profiles/ (one line per kernel: `kernel:dtype ratio`).  A kernel that has no line, or whose line was
    removed because the kernel changed after the capture, reports traffic null."""
    out = {}
    try:
        for ln in open(TRAFFIC_FILE):
            ln = ln.split("#")[0].split()
            if len(ln) == 2:
                out[ln[0]] = float(ln[1])
    except OSError:
        pass
    return out


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c5", choices=["c1", "c2", "c3", "c4", "c5", "c5a", "c5b", "c5f", "c5r", "c3s", "c3a"])
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="skip the shorter runs of c4, c5a, c5b and c3 reported under `also`")
    ap.add_argument("--also-steps", type=int, default=10)
    ap.add_argument("--shrink-d", type=int, default=0, help="profiling aid: same workload structure at a smaller d")
    ap.add_argument("--shrink-M", type=int, default=0)
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def elem_size(w):
    return 2 if w.dtype == "bf16" else 4


def sub_workloads(name: str):
    """The variants one step runs: c5 is both the Top-k and the bit-wise variant of the 124M config."""
    from paper_2507_05508_b200 import workloads as wl
    return [wl.C5A, wl.C5B] if name == "c5" else [wl.ALL[name]]


def describe(subs) -> str:
    w = subs[0]
    kinds = " + ".join(f"{'adaptive' if x.adaptive else 'fixed-p'} MLMC-{x.kind}" for x in subs)
    return f"{'c5' if len(subs) == 2 else w.name}: {kinds}, d={w.d}, M={w.M}, {w.dtype}"


# --------------------------------------------------------------------------------------------------
# multi-rank plumbing (ranks are independent replicas; the only collective is the max over times)
# --------------------------------------------------------------------------------------------------
def dist_setup(n_gpus: int):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
        return dist.get_rank(), world, int(os.environ.get("LOCAL_RANK", "0"))
    return 0, 1, 0


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(local_ms: float, world: int, device: str) -> float:
    """Slowest rank's time: the step count is fixed per rank, so whole-job throughput divides by this."""
    if world == 1:
        return local_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(device_index)], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def _stamp(text: str):
        try:
            return datetime.datetime.strptime(text.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except Exception:
            return None

    def stop(self, t0: float = None, t1: float = None):
        """Median SM clock, reasons and power over the samples taken between the wall-clock times t0 and t1 (the
        timed region; the sampler is started before the warm-up so that it is already running); all samples when
        none carries a usable time stamp inside the window."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        rows = [r.strip().split(",") for r in self.tmp.read().splitlines() if r.strip()]
        self.tmp.close()
        os.unlink(self.tmp.name)
        if t0 is not None and t1 is not None:
            inside = [r for r in rows if (lambda ts: ts is not None and t0 <= ts <= t1)(self._stamp(r[0]))]
            if inside:
                rows = inside
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
                power.append(float(r[3]))
                for name, v in zip(names, r[4:8]):
                    if v.strip().lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w_max=max(power))
        return out


# --------------------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------------------
class Runner:
    """Owns the buffers of one workload (one or two variants over the same batch) and runs steps through the C ABI.
    Every variant has its own context, message buffers and dense output; the variants of a step do not depend on one
    another, so a step runs them side by side, each on a CUDA stream of its own (a context serves one stream at a
    time), forked from and joined to the stream that times the step."""

    def __init__(self, subs, device_index: int, n_batches: int = 2, rank: int = 0):
        import torch
        from paper_2507_05508_b200 import binding as B
        from paper_2507_05508_b200 import workloads as wl
        self.torch, self.B, self.wl, self.subs = torch, B, wl, subs
        w = self.w = subs[0]
        self.dev = f"cuda:{device_index}"
        torch.cuda.set_device(device_index)
        self.ctxs = [B.mlmc_create(device_index, w.d, w.M, 32) for _ in subs]
        # the last variant runs on the timing stream, the ones before it on high-priority streams (the Top-k pipeline,
        # listed first, is a chain of many short kernels that should not queue behind the other variant's sweeps)
        self.side = [torch.cuda.Stream(device=self.dev, priority=-1) for _ in subs[:-1]] + [None]
        sc = wl.scales(w, self.dev)
        self.batches = [wl.gradients(w, 1000 * rank + i, self.dev, sc) for i in range(n_batches)]
        del sc
        self.denses = [torch.empty(w.d, dtype=torch.float32, device=self.dev) for _ in subs]
        self.plan = []
        for x in subs:
            if x.kind == "topk":
                sched = wl.topk_schedule(x)
                msgs = B.TopkBuffers(x.M, wl.max_band(sched), self.dev)
            elif x.kind == "stopk":
                sched = list(range(-(-x.d // x.seg_len)))           # one entry per level (segment)
                msgs = B.TopkBuffers(x.M, x.seg_len, self.dev)
            elif x.kind == "rtn":
                sched = list(x.bits) + [0]                          # the widths and the identity level
                msgs = B.RtnBuffers(x.M, x.d, self.dev)
            elif x.kind == "floatbits":
                sched = list(x.bits)
                widths = [sched[0]] + [sched[i] - sched[i - 1] for i in range(1, len(sched))]
                msgs = B.FloatBuffers(x.M, x.d, max(widths), self.dev)
            else:
                sched = list(x.bits)
                widths = [sched[0]] + [sched[i] - sched[i - 1] for i in range(1, len(sched))]
                msgs = B.BitBuffers(x.M, x.d, max(widths), self.dev)
            p = None if (x.adaptive or x.kind == "floatbits") else list(wl.geometric_probs(len(sched)))
            self.plan.append((x, sched, p, msgs))
        self.L = [len(pl[1]) for pl in self.plan]
        torch.cuda.synchronize()

    def _variant(self, j: int, i: int, g):
        B = self.B
        ctx, dense = self.ctxs[j], self.denses[j]
        x, sched, p, msgs = self.plan[j]
        if x.kind == "topk":
            B.mlmc_compress_topk(ctx, g, sched, p, x.seed, i, msgs)
            B.mlmc_aggregate(ctx, B.MLMC_TOPK, msgs, None, x.M, x.d, dense)
        elif x.kind == "stopk":
            B.mlmc_compress_stopk(ctx, g, x.seg_len, p, x.seed, i, msgs)
            B.mlmc_aggregate(ctx, B.MLMC_TOPK, msgs, None, x.M, x.d, dense)
        elif x.kind == "rtn":
            B.mlmc_compress_rtn(ctx, g, sched[:-1], p, x.seed, i, msgs)
            B.mlmc_aggregate_rtn(ctx, msgs, x.M, x.d, dense)
        elif x.kind == "floatbits":
            B.mlmc_compress_floatbits(ctx, g, sched, p, x.seed, i, msgs)
            B.mlmc_aggregate_floatbits(ctx, msgs, sched, x.M, x.d, dense)
        else:
            B.mlmc_compress_bitwise(ctx, g, sched, p, x.seed, i, msgs)
            B.mlmc_aggregate(ctx, B.MLMC_BITWISE, msgs, sched, x.M, x.d, dense)

    def step(self, i: int, g=None, side_by_side: bool = True):
        torch = self.torch
        g = self.batches[i % len(self.batches)] if g is None else g
        if len(self.plan) == 1 or not side_by_side:
            for j in range(len(self.plan)):
                self._variant(j, i, g)
            return
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        joins = []
        for j in range(len(self.plan) - 1):
            self.side[j].wait_event(fork)          # the batch is ready
            with torch.cuda.stream(self.side[j]):
                self._variant(j, i, g)
                done = torch.cuda.Event()
                done.record(self.side[j])
            joins.append(done)
        self._variant(len(self.plan) - 1, i, g)
        for done in joins:
            main.wait_event(done)                  # the step ends when every variant has

    def status(self) -> int:
        for ctx in self.ctxs:
            st = self.B.mlmc_get_status(ctx)
            if st != 0:
                return st
        return 0

    def launch_count(self) -> int:
        return sum(self.B.mlmc_launch_count(ctx) for ctx in self.ctxs)

    def timing_enable(self, on: bool):
        for ctx in self.ctxs:
            self.B.mlmc_timing_enable(ctx, on)

    def timing_read(self) -> dict:
        out = {}
        for ctx in self.ctxs:
            for name, (ms, n) in self.B.mlmc_timing_read(ctx).items():
                a = out.setdefault(name, [0.0, 0])
                a[0] += ms
                a[1] += n
        return {k: (v[0], v[1]) for k, v in out.items()}

    def topk_ctx(self):
        for ctx, (x, _, _, _) in zip(self.ctxs, self.plan):
            if x.kind in ("topk", "stopk"):
                return ctx
        return None

    def message_bytes(self):
        """Per variant kind: bytes of the messages of the last step (written once by compress, read once by aggregate)."""
        out = {}
        for x, sched, p, msgs in self.plan:
            if x.kind in ("topk", "stopk"):
                out["topk"] = float(msgs.count.sum().item()) * 8.0
            elif x.kind == "rtn":
                out["dense"] = float(sum(1 for l in msgs.level.tolist() if l >= 0)) * x.d * 4.0
            elif x.kind == "floatbits":
                widths = [sched[0]] + [sched[i] - sched[i - 1] for i in range(1, len(sched))]
                out["floatbits"] = float(sum((1 + widths[l]) * msgs.words * 4 + x.d for l in msgs.level.tolist() if l >= 0))
            else:
                widths = [sched[0]] + [sched[i] - sched[i - 1] for i in range(1, len(sched))]
                out["bitwise"] = float(sum((1 + widths[l]) * msgs.words * 4 for l in msgs.level.tolist() if l >= 0))
        return out

    def close(self):
        for ctx in self.ctxs:
            self.B.mlmc_destroy(ctx)


def sweeps_charged(w, emit_read_frac=None) -> float:
    """Gradient sweeps charged to the step: what the method needs (a true data dependence separates them: select ->
    emit for Top-k, max -> pack for fixed-p bit-wise, max -> field energies -> pack for adaptive bit-wise), or what
    the kernels moved where that is less.  Top-k moves one whole histogram sweep, for adaptive fp32 a second whole
    sweep, and two passes over the listed tiles (emit_read_frac of the row each); the fixed-p candidate sweep,
    which also skips tiles, is counted as nothing, so the figure is a lower bound of the bytes moved."""
    if w.kind in ("topk", "stopk"):
        if emit_read_frac is None:
            return 2.0
        moved = 1.0 + (1.0 if (w.adaptive and w.dtype != "bf16") else 0.0) + 2.0 * emit_read_frac
        return min(2.0, moved)
    if w.kind == "floatbits":
        return 1.0  # App. B's probabilities are fixed: the level is drawn before the data is read, one sweep packs it
    return 3.0 if w.adaptive else 2.0  # bit-wise and RTN: max -> level statistics -> message


# Algorithmic bytes of one launch of each kernel, as a function of (sweep bytes, message bytes of its variant, dense
# bytes, share of the row in the listed tiles).  band_count and emit read only the tiles that can hold band entries,
# so they are charged that share of the row; the candidate sweep of fixed p also skips tiles, by a share that is not
# read back, so its bytes are unknown (None) there.
def kernel_alg_bytes(name: str, sweep: float, msg: dict, dense: float, read_frac, adaptive: bool):
    mt, mb = msg.get("topk", 0.0), msg.get("bitwise", 0.0)
    mf, md = msg.get("floatbits", 0.0), msg.get("dense", 0.0)
    listed = None if read_frac is None else read_frac * sweep
    table = {
        # masked_pass2/3 and norm_sweep are the full-sweep fall-back of a worker whose candidates overflowed: they exit
        # at once otherwise, so no bytes are claimed for them
        "hist1": sweep, "sums_candidates": sweep if adaptive else None,
        "band_count": listed, "emit": None if listed is None else listed + mt,
        "aggregate_topk": mt + dense,
        "absmax": sweep, "bit_stats": sweep, "bit_pack": sweep + mb, "aggregate_bitwise": mb + dense,
        "float_pack": sweep + mf, "aggregate_floatbits": mf + dense,
        "rtn_stats": sweep, "rtn_emit": sweep + md, "aggregate_dense": md + dense,
    }
    return table.get(name)


def sort_step_bytes(name: str, sweep: float, elem: int):
    """Bytes per STEP of the radix-sort kernels of the adaptive s-Top-k path with many segments (their launches
    differ in size: the rows are sorted in groups): 32-bit keys, 4 passes for fp32 and 2 for bf16, the first pass
    reading the gradient itself; a count pass reads its input, a scatter pass reads it and writes the keys."""
    keys, passes = sweep * 4.0 / elem, (4 if elem == 4 else 2)
    reads = sweep + (passes - 1) * keys
    return {"sort_count": reads, "sort_scatter": reads + passes * keys, "segment_norms": keys}.get(name)


def l2_policy(sweep_bytes: float, n_batches: int) -> str:
    l2 = 126e6
    if sweep_bytes > l2:
        return f"inputs larger than L2: {sweep_bytes / 1e6:.0f} MB per sweep, {n_batches} batches alternated"
    return (f"inputs smaller than L2 ({sweep_bytes / 1e6:.1f} MB per sweep): a {2 * l2 / 1e6:.0f} MB buffer is written "
            "between timed steps (flush), outside the event pairs")


def measure(subs, local: int, rank: int, world: int, steps: int, warmup: int, peak: float, peak_kind: str,
            e2e_steps: int = 0):
    """Times `steps` steps of one workload on this rank's GPU and returns its figures.  Three loops: the headline
    loop (device-timed, nothing else enqueued), a second loop with one CUDA event pair around every kernel launch
    (per-kernel times, message volume and the share of the row the emission read, step by step), and optionally
    the end-to-end loop with host buffers."""
    import torch
    w = subs[0]
    r = Runner(subs, local, rank=rank)
    B = r.B
    sweep_bytes = float(w.M) * w.d * elem_size(w)
    dense_bytes = float(w.d) * 4.0
    small = sweep_bytes <= 126e6
    flush = torch.empty(int(252e6) // 4, dtype=torch.float32, device=r.dev) if small else None

    sampler = ClockSampler(local)  # running before the warm-up; only its samples inside the timed region are kept
    for i in range(max(warmup, 3)):
        r.step(i)
    torch.cuda.synchronize()
    assert r.status() == 0, "device status after warm-up"

    # ---- headline loop: exactly `steps` steps, device-timed, per-kernel timing off
    launches0 = r.launch_count()
    barrier(world)
    torch.cuda.synchronize()
    t_wall0 = time.time()
    if small:  # an L2-sized input: flush between steps, every step has its own event pair
        local_ms = 0.0
        for i in range(steps):
            flush.fill_(float(i))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            r.step(warmup + i)
            e1.record()
            torch.cuda.synchronize()
            local_ms += e0.elapsed_time(e1)
    else:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            r.step(warmup + i)
        e1.record()
        torch.cuda.synchronize()
        local_ms = e0.elapsed_time(e1)
    barrier(world)
    t_wall = time.time() - t_wall0
    clocks = sampler.stop(t_wall0, t_wall0 + t_wall)
    total_ms = max_over_ranks(local_ms, world, r.dev)
    launches = r.launch_count() - launches0
    status = r.status()
    ms_per_step = total_ms / steps
    value = world * len(subs) * sweep_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- second loop, same steps: per-kernel event pairs, message volume, listed tiles (read back after every step)
    r.timing_enable(True)
    per_kernel, msg_acc = {}, {}
    listed_acc, listed_n = 0.0, 0
    probe = min(steps, 16)
    for i in range(probe):
        if small:
            flush.fill_(float(i))
        r.step(warmup + i, side_by_side=False)  # one variant after the other: the event pairs time kernels that run alone
        for name, (ms, n) in r.timing_read().items():
            acc = per_kernel.setdefault(name, [0.0, 0])
            acc[0] += ms
            acc[1] += n
        for kind, v in r.message_bytes().items():
            msg_acc[kind] = msg_acc.get(kind, 0.0) + v
        if any(x.kind in ("topk", "stopk") for x in subs):
            listed, tiles = B.mlmc_read_listed_tiles(r.topk_ctx(), w.M)
            listed_acc += sum(listed) / float(max(1, tiles * w.M))
            listed_n += 1
    r.timing_enable(False)
    emit_read_frac = (listed_acc / listed_n) if listed_n else None
    msg_by_kind = {kind: v / probe for kind, v in msg_acc.items()}
    msg_bytes = sum(msg_by_kind.values())

    # ---- roofline of the dominant kernel and of the whole step
    ratios = ncu_traffic_ratios()
    adaptive_topk = any(x.kind in ("topk", "stopk") and x.adaptive for x in subs)
    kernels = {}
    t_all = sum(v[0] for v in per_kernel.values())
    for name, (ms, n) in sorted(per_kernel.items(), key=lambda kv: -kv[1][0]):
        kb = kernel_alg_bytes(name, sweep_bytes, msg_by_kind, dense_bytes, emit_read_frac, adaptive_topk)
        avg_ms = ms / n
        ach = None if not kb else kb / (avg_ms * 1e-3) / 1e9
        sb = sort_step_bytes(name, sweep_bytes, elem_size(w))
        if sb:
            ach = sb / (ms / probe * 1e-3) / 1e9
        kernels[name] = {"ms_per_step": round(ms / probe, 4), "launches_per_step": n / probe,
                         "share": round(ms / t_all, 4), "achieved_gbs": None if ach is None else round(ach, 1),
                         "frac": None if ach is None else round(ach / peak, 4)}
    dom_name = next(iter(kernels))
    dom_ms, dom_n = per_kernel[dom_name]
    dom_bytes = kernel_alg_bytes(dom_name, sweep_bytes, msg_by_kind, dense_bytes, emit_read_frac, adaptive_topk)
    dom_avg_s = dom_ms / dom_n * 1e-3
    achieved = None if not dom_bytes else dom_bytes / dom_avg_s / 1e9
    ratio = ratios.get(f"{dom_name}:{w.dtype}")
    roofline = {"bound": "hbm", "kernel": dom_name, "achieved": None if achieved is None else round(achieved, 1),
                "peak": peak, "unit": "GB/s", "frac": None if achieved is None else round(achieved / peak, 4),
                "peak_source": peak_kind,
                "traffic": None if (ratio is None or not dom_bytes) else ratio * dom_bytes,
                "alg_bytes_per_launch": dom_bytes, "avg_launch_ms": round(dom_avg_s * 1e3, 4)}
    b_alg = sum(sweeps_charged(x, emit_read_frac) * sweep_bytes + dense_bytes for x in subs) + 2 * msg_bytes
    step_frac = b_alg / (ms_per_step * 1e-3) / 1e9 / peak

    # ---- end to end: inputs start in pinned host memory, the dense mean ends in host memory
    e2e = None
    if e2e_steps > 0:
        host_in = torch.empty(r.batches[0].shape, dtype=r.batches[0].dtype, pin_memory=True)
        host_in.copy_(r.batches[0])
        host_out = [torch.empty(w.d, dtype=torch.float32, pin_memory=True) for _ in r.denses]  # every variant's mean
        # Three streams, as a training loop would run it: the copy of step i + 1's gradients into the other device
        # batch and the read-back of step i's means run beside the compute of the steps between them.  Every step
        # copies its whole input from pinned host memory and reads every variant's dense mean back; the timed region
        # starts before the first copy and ends after the last read-back.
        bufs = r.batches[:2] if len(r.batches) >= 2 else [r.batches[0], torch.empty_like(r.batches[0])]
        s_in, s_out = torch.cuda.Stream(device=r.dev), torch.cuda.Stream(device=r.dev)
        main = torch.cuda.current_stream()

        def e2e_run(n, first):
            computed, copied_out = {}, None
            for k in range(n):
                i = first + k
                buf = bufs[k % 2]
                if k >= 2:
                    s_in.wait_event(computed[k - 2])       # the step that read this batch has finished
                with torch.cuda.stream(s_in):
                    buf.copy_(host_in, non_blocking=True)
                    arrived = torch.cuda.Event()
                    arrived.record(s_in)
                main.wait_event(arrived)
                if copied_out is not None:
                    main.wait_event(copied_out)            # the means of the step before are on the host
                r.step(i, buf)
                computed[k] = torch.cuda.Event()
                computed[k].record(main)
                s_out.wait_event(computed[k])
                with torch.cuda.stream(s_out):
                    for dst, src in zip(host_out, r.denses):
                        dst.copy_(src, non_blocking=True)
                    copied_out = torch.cuda.Event()
                    copied_out.record(s_out)
            main.wait_event(copied_out)

        e2e_run(1, 0)
        torch.cuda.synchronize()
        barrier(world)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        s_in.wait_event(a)
        e2e_run(e2e_steps, 1)
        b.record()
        torch.cuda.synchronize()
        barrier(world)
        e2e_ms = max_over_ranks(a.elapsed_time(b), world, r.dev) / e2e_steps
        e2e = {"value": round(world * len(subs) * sweep_bytes / (e2e_ms * 1e-3) / 1e9, 2), "unit": UNIT,
               "h2d_bytes_per_step": int(sweep_bytes), "d2h_bytes_per_step": int(dense_bytes) * len(r.denses),
               "ms_per_step": round(e2e_ms, 3)}
        del host_in, host_out

    words = describe(subs) + f", L={r.L}"
    if len(subs) > 1:
        words += (f"; value counts the gradient bytes once per variant ({len(subs)} x M*d*4 per step); the variants of "
                  f"a step run side by side on {len(subs)} CUDA streams, a context each")
    res = {
        "value": round(value, 2), "ms_per_step": round(ms_per_step, 4), "steps": steps,
        "config": {"workload": words, "l2_policy": l2_policy(sweep_bytes, len(r.batches)),
                   "parallelism": "replicas only"},
        "elements_per_s": round(world * len(subs) * w.M * w.d / (ms_per_step * 1e-3), 1),
        "step_roofline": {"alg_bytes_per_step": b_alg,
                          "sweeps_charged": [round(sweeps_charged(x, emit_read_frac), 3) for x in subs],
                          "emit_tiles_read_frac": None if emit_read_frac is None else round(emit_read_frac, 4),
                          "message_bytes_per_step": msg_bytes, "frac_of_peak": round(step_frac, 4),
                          "frac_of_8TBs": round(b_alg / (ms_per_step * 1e-3) / 8e12, 4)},
        "roofline": roofline, "kernels": kernels, "gpu_launches": int(launches), "e2e": e2e, "clocks": clocks,
        "device_status": status, "wall_s_timed": round(t_wall, 3),
    }
    row0 = r.batches[0][0].clone() if (rank == 0 and world == 1) else None
    r.close()
    del r, flush
    torch.cuda.empty_cache()
    return res, row0


def run_cuda(args):
    import torch
    from paper_2507_05508_b200 import build as cuda_build
    from paper_2507_05508_b200 import workloads as wl
    cuda_build.build()
    rank, world, local = dist_setup(args.gpus)
    subs = sub_workloads(args.workload)
    if args.shrink_d or args.shrink_M:
        subs = [wl.shrink(x, args.shrink_d or x.d, args.shrink_M or x.M) for x in subs]
    w = subs[0]
    peak, peak_kind = measured_peak()
    res, row0 = measure(subs, local, rank, world, args.steps, args.warmup, peak, peak_kind, args.e2e_steps)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(subs, row0, budget_s=15.0)
    del row0

    # the other benchmark workloads, shorter runs of the same measurement (single GPU, default workload only)
    also = None
    if world == 1 and args.workload == "c5" and not args.no_also and not (args.shrink_d or args.shrink_M):
        also = {}
        for name in ("c4", "c5a", "c5b", "c3"):
            r2, _ = measure(sub_workloads(name), local, rank, world, args.also_steps, 3, peak, peak_kind, 0)
            also[name] = {k: r2[k] for k in ("ms_per_step", "value", "steps", "config", "step_roofline", "roofline",
                                            "gpu_launches", "device_status")}
            also[name]["kernels"] = {k: v for k, v in list(r2["kernels"].items())[:6]}
            also[name]["clocks"] = {k: r2["clocks"].get(k) for k in ("sm_mhz", "sm_max_mhz", "reasons")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" if w.dtype == "f32" else "bf16",
            "data": "synthetic", "config": res["config"], "elements_per_s": res["elements_per_s"],
            "step_roofline": res["step_roofline"], "roofline": res["roofline"], "kernels": res["kernels"],
            "gpu_launches": res["gpu_launches"], "e2e": res["e2e"], "cpu_baseline": cpu, "clocks": res["clocks"],
            "device_status": res["device_status"], "wall_s_timed": res["wall_s_timed"], "also": also,
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------------
# the oracle, timed on the host cores (reported baseline, and the --impl reference arm)
# --------------------------------------------------------------------------------------------------
def oracle_sample_step(subs, g_row_np, d_s: int, step: int):
    """One worker's compress + its aggregate share on the first d_s coordinates, for every variant; returns seconds."""
    import numpy as np
    import oracle
    from paper_2507_05508_b200 import workloads as wl
    x = np.ascontiguousarray(g_row_np[:d_s])
    t0 = time.perf_counter()
    for w in subs:
        if w.kind == "topk":
            ws = wl.shrink(w, d_s, 1)
            k = wl.topk_schedule(ws)
            p = None if w.adaptive else wl.geometric_probs(len(k))
            m = oracle.topk(x, k, p=p, seed=w.seed, step=step, worker=0)
            oracle.aggregate_topk([(m.idx, m.val)], d_s)
        elif w.kind == "stopk":
            s_len = max(1, min(w.seg_len, d_s))
            L = -(-d_s // s_len)
            m = oracle.stopk(x, s_len, p=None if w.adaptive else wl.geometric_probs(L), seed=w.seed, step=step, worker=0)
            oracle.aggregate_topk([(m.idx, m.val)], d_s)
        elif w.kind == "rtn":
            m = oracle.rtn(x, list(w.bits), p=None, seed=w.seed, step=step, worker=0)
            oracle.aggregate_dense([m.val], d_s)
        elif w.kind == "floatbits":
            m = oracle.floatbits(x, list(w.bits), p=None, seed=w.seed, step=step, worker=0)
            oracle.aggregate_dense([m.est], d_s)
        else:
            b = list(w.bits)
            p = None if w.adaptive else wl.geometric_probs(len(b))
            m = oracle.bitwise(x, b, p=p, seed=w.seed, step=step, worker=0)
            oracle.aggregate_bitwise([m], b, d_s)
    return time.perf_counter() - t0


def calibrate_sample(subs, g_row_np, budget_s: float) -> int:
    """Largest power-of-two prefix whose oracle step fits the per-step budget (extrapolated from a probe)."""
    d = subs[0].d
    probe = min(1 << 18, d)
    t = max(oracle_sample_step(subs, g_row_np, probe, 0), 1e-4)
    d_s = probe
    while d_s * 2 <= min(d, 1 << 25) and t * 2.2 <= budget_s:
        d_s *= 2
        t *= 2.2
    return d_s


def cpu_baseline(subs, g_row, budget_s: float):
    import oracle
    from paper_2507_05508_b200 import workloads as wl
    oracle.build()
    w = subs[0]
    row = wl.as_numpy_bits(g_row.unsqueeze(0))[0]
    d_s = calibrate_sample(subs, row, budget_s)
    t = oracle_sample_step(subs, row, d_s, 1)
    return {"value": round(len(subs) * d_s * elem_size(w) / t / 1e9, 5), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"1 worker, first {d_s} of d={w.d} coordinates, compress + aggregate of every variant, {t:.2f} s",
            "elements_per_s": round(len(subs) * d_s / t, 1)}


def run_reference(args):
    """Times the CPU oracle, as it stands, on bounded samples of the same workload (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2507_05508_b200 import workloads as wl
    oracle.build()
    subs = sub_workloads(args.workload)
    w = subs[0]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    d_gen = min(w.d, 1 << 25)
    wg = wl.shrink(w, d_gen, 1) if d_gen < w.d else w
    row = wl.as_numpy_bits(wl.gradients(wg, 0, dev)[:1])[0]
    per_step_budget = max(0.05, 150.0 / max(1, args.steps + args.warmup))
    d_s = min(calibrate_sample(subs, row, per_step_budget), d_gen)
    for i in range(args.warmup):
        oracle_sample_step(subs, row, d_s, i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle_sample_step(subs, row, d_s, args.warmup + i)
    t = (time.perf_counter() - t0) / args.steps
    value = len(subs) * d_s * elem_size(w) / t / 1e9
    sample = (f"each step: 1 worker, first {d_s} of d={w.d} coordinates, compress + aggregate of every variant "
              "on 1 host core")
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 5), "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(t * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if w.dtype == "f32" else "bf16", "data": "synthetic",
            "config": {"workload": describe(subs), "sample": sample},
            "cpu_baseline": {"value": round(value, 5), "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 5), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_cuda(a)
