#!/usr/bin/env python
"""Benchmark of the S2A 4-bit stash hot path on synthetic ViT-shaped activations.

One step = one pass of the whole path over one batch: for every transformer block the
softmax and GELU forward kernels (keeping each block's 4-bit stash resident), then for
every block in reverse the GELU and softmax backward kernels.  The default workload is
ViT-B/16 at 224 px, batch 64, bfloat16, 12 blocks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With N > 1 (launched by torchrun, one rank per GPU) every rank
runs an independent replica -- rows are independent, the path has no exchange step --
and the line reports the aggregate over ranks against the slowest rank's time.
"""
from __future__ import annotations

import argparse
import ctypes
import hashlib
import json
import os
import statistics
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_08154_b200 import synth  # noqa: E402

KERNELS = ("softmax_fwd", "gelu_fwd", "gelu_bwd", "softmax_bwd")
L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=synth.VIT_B16_B64.name, choices=sorted(synth.SHAPES))
    ap.add_argument("--blocks", type=int, default=0, help="override the number of blocks (0: the workload's)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--repeats", type=int, default=0,
                    help="how many times the K-step timed region is repeated (0: at least 5, and enough for about a second)")
    return ap.parse_args()


# ------------------------------------------------------------------ bytes the method must move
def algorithmic_bytes(n_elems: int, row_len: int, itemsize: int) -> int:
    """Per kernel launch: tensor in + tensor out + packed codes + per-row (min, s)."""
    return 2 * n_elems * itemsize + (n_elems + 1) // 2 + 8 * (n_elems // row_len)


def workload_tables(shape, blocks):
    item = synth.io_itemsize(shape.dtype)
    has_softmax = shape.name != synth.VIT_B16_B8_F32.name
    per_launch = {}
    elems = {}
    for k in KERNELS:
        if k.startswith("softmax"):
            if not has_softmax:
                continue
            elems[k] = shape.softmax_elems
            per_launch[k] = algorithmic_bytes(shape.softmax_elems, shape.tokens, item)
        else:
            elems[k] = shape.gelu_elems
            per_launch[k] = algorithmic_bytes(shape.gelu_elems, shape.hidden, item)
    step_bytes = blocks * sum(per_launch.values())
    # each nonlinearity's elements are counted once per step (forward+backward is one unit)
    step_elems = blocks * (shape.gelu_elems + (shape.softmax_elems if has_softmax else 0))
    stash = blocks * sum((elems[k] + 1) // 2 + 8 * (elems[k] // (shape.tokens if k.startswith("softmax") else shape.hidden))
                         for k in per_launch if k.endswith("fwd"))
    return has_softmax, per_launch, elems, step_bytes, step_elems, stash


# ------------------------------------------------------------------ host inputs
def host_inputs(shape, blocks, seed, rows_gelu=None, rows_softmax=None, with_softmax=True):
    """Per block: (gelu_x, gelu_g, softmax_x, softmax_g) as numpy arrays in I/O representation."""
    def one(b):
        gx, gg = synth.vit_gelu_inputs(shape, seed, b, rows_gelu)
        if with_softmax:
            sx, sg = synth.vit_softmax_inputs(shape, seed, b, rows_softmax)
        else:
            sx = sg = None
        return gx, gg, sx, sg

    with ThreadPoolExecutor(max_workers=max(1, min(blocks, os.cpu_count() or 1))) as pool:
        return list(pool.map(one, range(blocks)))


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
        0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, uuid, index):
        self.samples = []
        self.stop = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None
        self.thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        while not self.stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception:
                pass
            self.stop.wait(0.01)

    def start(self):
        if self.ok:
            self.thread.start()

    def finish(self, t0, t1):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        self.stop.set()
        self.thread.join()
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = "sampled during the timed region"
        if not inside:
            inside = self.samples[-3:]
            note = "timed region shorter than the sampling period: last samples under load"
        bits = 0
        for s in inside:
            bits |= s[2]
        reasons = [name for bit, name in self.REASONS.items() if bits & bit and name != "gpu_idle"]
        return {"sm_mhz": statistics.median(s[1] for s in inside) if inside else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(inside), "note": note}


# ------------------------------------------------------------------ peaks and stored traffic
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def kernel_source_digest():
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2503_08154_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def stored_traffic(kernel, workload):
    """DRAM bytes per launch from the committed ncu capture, if the kernels are unchanged since."""
    try:
        t = json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))
        e = t[workload][kernel]
        return e["dram_bytes_per_launch"] if e["source_digest"] == kernel_source_digest() else None
    except Exception:
        return None


# ------------------------------------------------------------------ the CPU oracle legs
def oracle_time_block(shape, arrays, threads):
    """Forward+backward of both nonlinearities through the oracle on one block's arrays.
    Returns (algorithmic bytes, elements, seconds, forward results)."""
    from oracle import s2a_oracle as o
    gx, gg, sx, sg = arrays
    item = synth.io_itemsize(shape.dtype)
    t0 = time.perf_counter()
    gy, gc, gm = o.gelu_fwd(gx, shape.hidden, shape.dtype, threads)
    o.gelu_bwd(gg, gc, gm, shape.hidden, shape.dtype, threads)
    nbytes = 2 * algorithmic_bytes(gx.size, shape.hidden, item)
    nelem = gx.size
    fwd = {"gelu": (gy, gc, gm)}
    if sx is not None:
        sy, sc, sm = o.softmax_fwd(sx, shape.tokens, shape.dtype, threads)
        o.softmax_bwd(sg, sc, sm, shape.tokens, shape.dtype, threads)
        nbytes += 2 * algorithmic_bytes(sx.size, shape.tokens, item)
        nelem += sx.size
        fwd["softmax"] = (sy, sc, sm)
    return nbytes, nelem, time.perf_counter() - t0, fwd


def oracle_sample_rate(shape, blocks_arrays, threads, core_seconds=12.0, on_block=None):
    """Times the oracle, as it stands, on whole blocks of the workload until about
    `core_seconds` of CPU work (threads x wall time) have been spent.  on_block(index, forward
    results) is called outside the timed part (the parity counts of the benchmark line)."""
    from oracle import s2a_oracle as o
    o.lib()
    nbytes = nelem = 0
    secs = 0.0
    used = 0
    for i, arrays in enumerate(blocks_arrays):
        b, e, t, fwd = oracle_time_block(shape, arrays, threads)
        nbytes, nelem, secs, used = nbytes + b, nelem + e, secs + t, used + 1
        if on_block is not None:
            on_block(i, arrays, fwd)
        del fwd
        if secs * threads >= core_seconds:
            break
    sample = "fwd+bwd of GELU%s on %d of the workload's blocks, full size (%.1f core-seconds)" % (
        " and softmax" if blocks_arrays[0][2] is not None else "", used, secs * threads)
    return nbytes / secs / 1e9, nelem / secs / 1e9, secs, sample


# ------------------------------------------------------------------ parity counts for the line
def _unpack4(codes, n):
    q = np.empty(2 * codes.size, dtype=np.uint8)
    q[0::2], q[1::2] = codes & 0xF, codes >> 4
    return q[:n]


def softmax_code_flips(codes_gpu, y_oracle, codes_oracle, x, L, dt):
    """Elements whose 4-bit code differs from the oracle's, and how many of them are NOT within
    reach of a bin edge.  Reach: what the output tolerance (1 bfloat16 ulp; 1e-6 relative plus
    2^-24 |x_i - max x| in binary32) allows the oracle's scaled value t = (y - min) 15 / (max - min)
    to move by, through y_i, the row minimum and the row maximum, plus 1e-5."""
    n = y_oracle.size
    rows = n // L
    qg, qo = _unpack4(codes_gpu, n), _unpack4(codes_oracle, n)
    flip = np.nonzero(qg != qo)[0]
    if flip.size == 0:
        return 0, 0
    yo = synth.io_to_f32(y_oracle, dt).astype(np.float64).reshape(rows, L)
    xw = synth.io_to_f32(x, dt).astype(np.float64).reshape(rows, L)
    r, c = flip // L, flip % L
    rows_hit = np.unique(r)
    amin = dict(zip(rows_hit, yo[rows_hit].argmin(axis=1)))
    amax = dict(zip(rows_hit, yo[rows_hit].argmax(axis=1)))
    cmin = np.array([amin[k] for k in r])
    cmax = np.array([amax[k] for k in r])

    def tol(rr, cc):
        v = yo[rr, cc]
        if dt == synth.BF16:
            return np.exp2(np.floor(np.log2(np.maximum(np.abs(v), 2.0 ** -126))) - 7)
        return (1e-6 + 2.0 ** -24 * (xw[rr].max(axis=1) - xw[rr, cc])) * np.abs(v)

    mn, mx = yo[r, cmin], yo[r, cmax]
    inv = 15.0 / (mx - mn)
    t = (yo[r, c] - mn) * inv
    w = t / 15.0
    reach = inv * (tol(r, c) + (1 - w) * tol(r, cmin) + w * tol(r, cmax)) + 1e-5
    outside = (np.abs(t - np.floor(t) - 0.5) > reach) | (np.abs(qg[flip].astype(int) - qo[flip].astype(int)) > 1)
    return int(flip.size), int(outside.sum())


def run_reference(args, shape, blocks):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    from oracle import s2a_oracle as o
    threads = o.hardware_threads()
    has_softmax = shape.name != synth.VIT_B16_B8_F32.name
    arrays = host_inputs(shape, 1, args.seed, with_softmax=has_softmax)
    rates = []
    t_all = time.perf_counter()
    sample = ""
    for i in range(args.warmup + args.steps):
        gbs, gel, dt, sample = oracle_sample_rate(shape, arrays, threads, core_seconds=0.0)
        if i >= args.warmup:
            rates.append((gbs, gel, dt))
        if time.perf_counter() - t_all > 150 and len(rates) >= 1:
            break
    gbs = statistics.mean(r[0] for r in rates)
    line = {
        "impl": "reference", "metric": "s2a_fwd_bwd_algorithmic_bandwidth", "value": gbs, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": len(rates), "warmup": args.warmup,
        "ms_per_step": 1e3 * statistics.mean(r[2] for r in rates), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": shape.name, "blocks": blocks, "sample_per_step": sample},
        "gelem_per_s": statistics.mean(r[1] for r in rates),
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ aggregation over ranks
def max_over_ranks(ms: float, world: int, device=None) -> float:
    """The slowest rank's time: every rank runs an independent replica of the same step, so
    the job's time is the maximum and its throughput is world * per-replica work / max."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(step_bytes: int, steps: int, ms: float, world: int) -> float:
    """Whole-job GB/s of `world` replicas that each moved step_bytes * steps in `ms`."""
    return world * step_bytes * steps / (ms * 1e-3) / 1e9


# ------------------------------------------------------------------ the CUDA path
def run_ours(args, shape, blocks, rank, world):
    import torch
    from paper_2503_08154_b200 import binding

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    lib = binding.lib()  # raises if the CUDA library is missing: there is no other path
    has_softmax, per_launch, elems, step_bytes, step_elems, stash = workload_tables(shape, blocks)
    item = synth.io_itemsize(shape.dtype)
    tdt = torch.float32 if shape.dtype == synth.F32 else torch.bfloat16

    def pin(a):
        t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
        return t.pin_memory()

    def dview(t):
        return t.view(tdt) if tdt == torch.bfloat16 else t

    # Distinct buffer sets, rotated step by step, so that what is touched between two uses of
    # the same buffer is several times the L2 (a workload of one small block would otherwise
    # run out of the cache).  The large workloads need one set.
    touched = blocks * (4 * item + 1) * (shape.gelu_elems + (shape.softmax_elems if has_softmax else 0))
    sets = max(1, -(-3 * L2_BYTES // touched))
    host = [tuple(pin(a) if a is not None else None for a in blk) for blk in host_inputs(
        shape, blocks * sets, args.seed + 1000 * rank, with_softmax=has_softmax)]

    class Block:
        pass

    blks = []
    for b in range(blocks * sets):
        B = Block()
        gx, gg, sx, sg = host[b]
        B.gx, B.gg = dview(gx.to(dev)), dview(gg.to(dev))
        B.gy, B.gin = torch.empty_like(B.gx), torch.empty_like(B.gg)
        B.gcodes, B.gmeta = binding.alloc_stash(shape.gelu_elems, shape.hidden, dev)
        if has_softmax:
            B.sx, B.sg = dview(sx.to(dev)), dview(sg.to(dev))
            B.sy, B.sin = torch.empty_like(B.sx), torch.empty_like(B.sg)
            B.scodes, B.smeta = binding.alloc_stash(shape.softmax_elems, shape.tokens, dev)
        blks.append(B)

    stream = torch.cuda.current_stream()
    sp = ctypes.c_void_p(stream.cuda_stream)
    dtc = shape.dtype
    ng, Lg = shape.gelu_elems, shape.hidden
    ns, Ls = shape.softmax_elems, shape.tokens

    # the sequence of C-ABI calls of one step on one buffer set, with pre-marshalled arguments
    def calls_of(set_blks):
        out = []
        for B in set_blks:
            if has_softmax:
                out.append(("softmax_fwd", lib.s2a_softmax_fwd, (B.sx.data_ptr(), B.sy.data_ptr(), B.scodes.data_ptr(), B.smeta.data_ptr(), ns, Ls, dtc, sp)))
            out.append(("gelu_fwd", lib.s2a_gelu_fwd, (B.gx.data_ptr(), B.gy.data_ptr(), B.gcodes.data_ptr(), B.gmeta.data_ptr(), ng, Lg, dtc, sp)))
        for B in reversed(set_blks):
            out.append(("gelu_bwd", lib.s2a_gelu_bwd, (B.gg.data_ptr(), B.gcodes.data_ptr(), B.gmeta.data_ptr(), B.gin.data_ptr(), ng, Lg, dtc, sp)))
            if has_softmax:
                out.append(("softmax_bwd", lib.s2a_softmax_bwd, (B.sg.data_ptr(), B.scodes.data_ptr(), B.smeta.data_ptr(), B.sin.data_ptr(), ns, Ls, dtc, sp)))
        return out

    set_calls = [calls_of(blks[i * blocks:(i + 1) * blocks]) for i in range(sets)]
    calls = set_calls[0]
    step_no = [0]

    def step():
        for _, fn, a in set_calls[step_no[0] % sets]:
            rc = fn(*a)
            if rc:
                raise RuntimeError(binding.status_string(rc))
        step_no[0] += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if binding.s2a_device_error() != 0:
        raise RuntimeError("a kernel gave up on a bounded wait during warm-up")

    # ---- timed region: K steps back to back, one event on the stream at each end.  (An
    # event between two launches would defeat programmatic dependent launch, so the
    # per-kernel figures are taken in separate loops below.)  The region is repeated R times
    # (each bracketed by a barrier and a device synchronisation on both sides); the reported
    # time is the median region, `spread` is (max - min) / median, and the clock sampler runs
    # across all repeats.
    n_calls = len(calls)
    sampler = ClockSampler(getattr(torch.cuda.get_device_properties(local), "uuid", ""), local)

    def timed_region():
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        for k in range(args.steps):
            step()
        ev1.record(stream)
        barrier()
        return max_over_ranks(ev0.elapsed_time(ev1), world, dev)

    probe_ms = timed_region()          # decides the number of repeats; not reported
    repeats = args.repeats if args.repeats > 0 else max(5, min(100, int(1000.0 / max(probe_ms, 1e-3)) + 1))
    if world > 1:                      # every rank must run the same number of regions
        t = torch.tensor([repeats], device=dev)
        dist.broadcast(t, 0)
        repeats = int(t.item())
    sampler.start()
    t0 = time.perf_counter()
    region_ms = [timed_region() for _ in range(repeats)]
    t1 = time.perf_counter()
    clocks = sampler.finish(t0, t1)
    total_ms = statistics.median(region_ms)
    spread = (max(region_ms) - min(region_ms)) / total_ms
    ordered = sorted(region_ms)
    spread_p10_p90 = (ordered[int(0.9 * (len(ordered) - 1))] - ordered[int(0.1 * (len(ordered) - 1))]) / total_ms
    if binding.s2a_device_error() != 0:
        raise RuntimeError("a kernel gave up on a bounded wait during the timed region")

    # ---- per kernel: the same launches grouped by kernel, K * blocks back to back (rotating
    # over the buffer sets like the steps do)
    per_kernel_ms = {}
    for name in per_launch:
        mine = [[(fn, a) for n_, fn, a in sc if n_ == name] for sc in set_calls]
        for grp in mine:
            for fn, a in grp:
                fn(*a)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for k in range(args.steps):
            for fn, a in mine[k % sets]:
                fn(*a)
        e1.record(stream)
        barrier()
        per_kernel_ms[name] = e0.elapsed_time(e1) / (args.steps * len(mine[0]))

    # ---- per kernel with an event before every launch of a step (for comparison: this
    # serialises the launches and adds the event's own cost to each)
    bracket_steps = min(args.steps, 20)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(n_calls + 1)] for _ in range(bracket_steps)]
    barrier()
    for k in range(bracket_steps):
        ev = events[k]
        for i, (_, fn, a) in enumerate(calls):
            ev[i].record(stream)
            fn(*a)
        ev[n_calls].record(stream)
    barrier()
    bracketed_ms = {k: [] for k in per_launch}
    for ev in events:
        for i, (name, _, _) in enumerate(calls):
            bracketed_ms[name].append(ev[i].elapsed_time(ev[i + 1]))

    # ---- end to end: pinned host inputs in, results out, every step
    e2e = None
    if not args.skip_e2e:
        hy_g = torch.empty(shape.gelu_elems * item, dtype=torch.uint8).pin_memory()
        hy_s = torch.empty(shape.softmax_elems * item, dtype=torch.uint8).pin_memory() if has_softmax else None

        # Host->device copies, kernels and device->host copies run on three streams chained
        # by events, so that the two PCIe directions and the kernels overlap; every step
        # still moves all of its inputs in and all of its results out.
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

        def staged(copies_in, launch, copies_out):
            with torch.cuda.stream(s_in):
                for dst, src in copies_in:
                    dst.copy_(dview(src), non_blocking=True)
                ready = torch.cuda.Event()
                ready.record(s_in)
            stream.wait_event(ready)
            launch()
            done = torch.cuda.Event()
            done.record(stream)
            s_out.wait_event(done)
            with torch.cuda.stream(s_out):
                for dst, src in copies_out:
                    dst.copy_(src.view(torch.uint8), non_blocking=True)

        def e2e_step():
            s_in.wait_stream(stream)  # last step's kernels have finished with the input buffers
            for B, (gx, gg, sx, sg) in zip(blks[:blocks], host[:blocks]):
                if has_softmax:
                    staged([(B.sx, sx)], lambda: binding.s2a_softmax_fwd(B.sx, B.sy, B.scodes, B.smeta, Ls),
                           [(hy_s, B.sy)])
                staged([(B.gx, gx)], lambda: binding.s2a_gelu_fwd(B.gx, B.gy, B.gcodes, B.gmeta, Lg), [(hy_g, B.gy)])
            for B, (gx, gg, sx, sg) in zip(reversed(blks[:blocks]), reversed(host[:blocks])):
                staged([(B.gg, gg)], lambda: binding.s2a_gelu_bwd(B.gg, B.gcodes, B.gmeta, B.gin, Lg), [(hy_g, B.gin)])
                if has_softmax:
                    staged([(B.sg, sg)], lambda: binding.s2a_softmax_bwd(B.sg, B.scodes, B.smeta, B.sin, Ls),
                           [(hy_s, B.sin)])
            stream.wait_stream(s_out)  # the step ends when its last result is on the host

        e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        e2e_ms = max_over_ranks(e2e_ms, world, dev)
        io_bytes = blocks * 2 * item * (shape.gelu_elems + (shape.softmax_elems if has_softmax else 0))
        e2e = {"value": aggregate_throughput(step_bytes, args.e2e_steps, e2e_ms, world), "unit": "GB/s",
               "h2d_bytes_per_step": io_bytes, "d2h_bytes_per_step": io_bytes, "steps": args.e2e_steps,
               "ms_per_step": e2e_ms / args.e2e_steps}

    if rank != 0:
        return

    peak, peak_kind = measured_peak()
    per_kernel = {}
    step_ms = total_ms / args.steps
    for k, avg in per_kernel_ms.items():
        gbs = per_launch[k] / (avg * 1e-3) / 1e9
        per_kernel[k] = {"avg_ms": avg, "launches_per_step": blocks, "algorithmic_bytes": per_launch[k], "GBps": gbs,
                         "gelem_per_s": elems[k] / (avg * 1e-3) / 1e9, "frac_of_%s_peak" % peak_kind: gbs / peak,
                         "frac_of_8TBps": gbs / NOMINAL_HBM_GBS, "share_of_step": avg * blocks / step_ms,
                         "avg_ms_event_bracketed": statistics.mean(bracketed_ms[k])}
    dominant = max(per_kernel, key=lambda k: per_kernel[k]["share_of_step"])
    roofline = {"bound": "hbm", "kernel": "s2a_" + dominant, "achieved": per_kernel[dominant]["GBps"], "peak": peak,
                "timing": "CUDA events around %d back-to-back launches of this kernel over the step's %d blocks" % (args.steps * blocks, blocks),
                "peak_source": "%s copy bandwidth" % peak_kind, "unit": "GB/s",
                "frac": per_kernel[dominant]["GBps"] / peak, "traffic": stored_traffic(dominant, shape.name)}

    value = aggregate_throughput(step_bytes, args.steps, total_ms, world)
    cpu_baseline = None
    parity = None
    if not args.skip_cpu_baseline:
        from oracle import s2a_oracle as o
        threads = o.hardware_threads()
        np_blocks = []
        for blk in host:
            np_blocks.append(tuple(None if t is None else (t.numpy().view(np.uint16) if t.dtype == torch.int16 else t.numpy())
                                   for t in blk))
        # While the oracle's forward results of a block are at hand, the stash the kernels left
        # for that block (same inputs) is compared with them: the counts go into the line.
        parity = {"blocks_checked": 0, "gelu_elements": 0, "gelu_code_mismatches": 0, "gelu_meta_mismatches": 0,
                  "softmax_elements": 0, "softmax_code_flips": 0, "softmax_flips_not_at_a_bin_edge": 0,
                  "softmax_rows_whose_range_moved_by_rounding": 0}

        def count_parity(i, arrays, fwd):
            B = blks[i]
            gy, gc, gm = fwd["gelu"]
            parity["blocks_checked"] += 1
            parity["gelu_elements"] += int(gy.size)
            parity["gelu_code_mismatches"] += int(np.count_nonzero(_unpack4(B.gcodes.cpu().numpy(), gy.size) != _unpack4(gc, gy.size)))
            parity["gelu_meta_mismatches"] += int(np.count_nonzero(B.gmeta.cpu().numpy().view(np.uint32) != gm.view(np.uint32)))
            if "softmax" in fwd:
                sy, sc, sm = fwd["softmax"]
                flips, outside = softmax_code_flips(B.scodes.cpu().numpy(), sy, sc, arrays[2], shape.tokens, shape.dtype)
                parity["softmax_elements"] += int(sy.size)
                parity["softmax_code_flips"] += flips
                parity["softmax_flips_not_at_a_bin_edge"] += outside
                parity["softmax_rows_whose_range_moved_by_rounding"] += int(np.count_nonzero(
                    (B.smeta.cpu().numpy().view(np.uint32) != sm.view(np.uint32)).reshape(-1, 2).any(axis=1)))

        gbs, gel, dtc_s, sample = oracle_sample_rate(shape, np_blocks, threads, on_block=count_parity)
        cpu_baseline = {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample,
                        "gelem_per_s": gel, "seconds": dtc_s}

    bf16_stash = blocks * 2 * (shape.gelu_elems + (shape.softmax_elems if has_softmax else 0))
    line = {
        "metric": "s2a_fwd_bwd_algorithmic_bandwidth", "value": value, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "repeats": repeats, "spread": spread, "spread_p10_p90": spread_p10_p90, "timing": "median of %d regions of %d steps each" % (repeats, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": shape.name, "blocks": blocks, "io_dtype": "bf16" if shape.dtype else "f32",
                   "gelu": [shape.gelu_rows, shape.hidden], "softmax": [shape.softmax_rows, shape.tokens] if has_softmax else None,
                   "l2": ("inputs larger than L2: %.2f GB touched per step, distinct buffers per block" % (touched / 1e9)) if sets == 1
                   else ("inputs larger than L2: steps rotate over %d distinct buffer sets, %.2f GB touched between two "
                         "uses of a buffer" % (sets, sets * touched / 1e9)),
                   "multi_gpu": "independent replicas, no collective"},
        "gelem_per_s": world * step_elems * args.steps / (total_ms * 1e-3) / 1e9,
        "frac_of_8TBps": value / world / NOMINAL_HBM_GBS,
        "frac_of_%s_peak" % peak_kind: value / world / peak,
        "saved_activation_bytes": {"stash": stash, "bf16_stash": bf16_stash, "fp32_stash": 2 * bf16_stash,
                                   "reduction_vs_bf16": bf16_stash / stash},
        "per_kernel": per_kernel, "roofline": roofline, "cpu_baseline": cpu_baseline, "parity": parity, "e2e": e2e,
        "gpu_launches": n_calls * args.steps, "clocks": clocks,
    }
    print(json.dumps(line))


def main():
    args = parse_args()
    shape = synth.SHAPES[args.workload]
    blocks = args.blocks if args.blocks > 0 else shape.blocks
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, shape, blocks)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain `python bench.py --gpus N`: start again under torch.distributed.run,
        # one rank per GPU on this node
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                  "--nproc-per-node", str(args.gpus), "--master-addr", "127.0.0.1",
                                  "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]])
    run_ours(args, shape, blocks, rank, world)


if __name__ == "__main__":
    main()
