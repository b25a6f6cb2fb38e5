"""Bandwidth sweep of the four kernels over tensor sizes and row lengths.

    python -m paper_2503_08154_b200.bandwidth_sweep [--quick] [--seeds 5]

GELU: 1e6 .. 2e9 elements (row length 4096), bfloat16 and float32.  Softmax: row lengths
64 / 197 / 257 / 1024 / 4096 with 1e4 .. 1e7 rows (combinations above 2e9 elements are
skipped).  Inputs are N(0,1), drawn on the device from seeds 0..S-1; every figure is the
median over the seeds of forward+backward algorithmic bytes per second, timed with CUDA
events over back-to-back launches on rotating buffers.  One JSON line per case.
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import binding

PEAK_NOTE = "algorithmic bytes = 2*n*itemsize + n/2 + 8*rows per kernel"


def _time_pair(kind: str, rows: int, L: int, dtype, seed: int, target_bytes: float = 1.5e9):
    n = rows * L
    item = 2 if dtype == torch.bfloat16 else 4
    per_set = 4 * n * item
    sets = max(1, min(6, int(target_bytes // per_set)))
    if per_set * sets < 3e8:  # keep the working set above the 126 MB L2
        sets = max(sets, min(8, int(3e8 // per_set) + 1))
    g = torch.Generator(device="cuda").manual_seed(seed)
    xs = [torch.randn(n, device="cuda", generator=g).to(dtype) for _ in range(sets)]
    gs = [torch.randn(n, device="cuda", generator=g).to(dtype) for _ in range(sets)]
    ys = [torch.empty_like(x) for x in xs]
    gins = [torch.empty_like(x) for x in xs]
    st = [binding.alloc_stash(n, L, "cuda") for _ in range(sets)]
    fwd = {"gelu": binding.s2a_gelu_fwd, "silu": binding.s2a_silu_fwd, "softmax": binding.s2a_softmax_fwd}[kind]
    bwd = {"gelu": binding.s2a_gelu_bwd, "silu": binding.s2a_silu_bwd, "softmax": binding.s2a_softmax_bwd}[kind]
    iters = max(4, min(200, int(2e10 // (n * item * 4))))

    def loop(fn):
        for i in range(min(3, sets)):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(i % sets)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / iters

    t_f = loop(lambda i: fwd(xs[i], ys[i], st[i][0], st[i][1], L))
    t_b = loop(lambda i: bwd(gs[i], st[i][0], st[i][1], gins[i], L))
    if binding.s2a_device_error() != 0:
        raise RuntimeError("a kernel gave up on a bounded wait")
    alg = 2 * n * item + (n + 1) // 2 + 8 * rows
    return alg / t_f / 1e9, alg / t_b / 1e9, 2 * alg / (t_f + t_b) / 1e9


def _time_relu(n: int, dtype, seed: int):
    item = 2 if dtype == torch.bfloat16 else 4
    sets = max(1, min(8, int(3e8 // (4 * n * item)) + 1))
    g = torch.Generator(device="cuda").manual_seed(seed)
    xs = [torch.randn(n, device="cuda", generator=g).to(dtype) for _ in range(sets)]
    ys = [torch.empty_like(x) for x in xs]
    ms = [torch.empty(binding.mask_bytes(n), dtype=torch.uint8, device="cuda") for _ in range(sets)]
    iters = max(4, min(200, int(2e10 // (n * item * 4))))

    def loop(fn):
        for i in range(min(3, sets)):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(i % sets)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / iters

    t_f = loop(lambda i: binding.s2a_relu_fwd(xs[i], ys[i], ms[i]))
    t_b = loop(lambda i: binding.s2a_relu_bwd(xs[i], ms[i], ys[i]))
    alg = 2 * n * item + (n + 7) // 8
    return alg / t_f / 1e9, alg / t_b / 1e9, 2 * alg / (t_f + t_b) / 1e9


def _time_tensor_range(rows: int, L: int, dtype, seed: int):
    n = rows * L
    item = 2 if dtype == torch.bfloat16 else 4
    sets = max(1, min(8, int(3e8 // (2 * n * item)) + 1))
    g = torch.Generator(device="cuda").manual_seed(seed)
    xs = [torch.randn(n, device="cuda", generator=g).to(dtype) for _ in range(sets)]
    ys = [torch.empty_like(x) for x in xs]
    st = [binding.alloc_stash(n, L, "cuda") for _ in range(sets)]
    scratch = torch.empty(binding.tensor_range_scratch_bytes(n), dtype=torch.uint8, device="cuda")
    iters = max(4, min(200, int(2e10 // (n * item * 4))))
    for i in range(min(3, sets)):
        binding.s2a_gelu_fwd_tensor_range(xs[i], ys[i], st[i][0], st[i][1], scratch, L)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        k = i % sets
        binding.s2a_gelu_fwd_tensor_range(xs[k], ys[k], st[k][0], st[k][1], scratch, L)
    e1.record()
    torch.cuda.synchronize()
    t = e0.elapsed_time(e1) * 1e-3 / iters
    alg = 3 * n * item + (n + 1) // 2 + 8 * rows   # x twice, y, codes, metadata
    return alg / t / 1e9


def _time_side(seed: int):
    """CAP (r = 8) and the LRP add on the ViT-B/16 batch-64 token stream [64*197, 768] ... [.., 3072]."""
    out = []
    g = torch.Generator(device="cuda").manual_seed(seed)
    for dtype in (torch.bfloat16, torch.float32):
        item = 2 if dtype == torch.bfloat16 else 4
        rows, ch, r = 64 * 197 * 4, 3072, 8
        xs = [torch.randn(rows * ch, device="cuda", generator=g).to(dtype) for _ in range(3)]
        ys = [torch.empty(rows * ch // r, device="cuda", dtype=dtype) for _ in range(3)]

        def timed(fn, iters=30):
            for i in range(3):
                fn(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(iters):
                fn(i % 3)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e-3 / iters

        t_f = timed(lambda i: binding.s2a_cap_fwd(xs[i], ys[i], rows, ch, r))
        t_b = timed(lambda i: binding.s2a_cap_bwd(ys[i], xs[i], rows, ch, r))
        alg = rows * ch * item * (1 + 1.0 / r)
        out.append({"kernel_pair": "cap", "rows": rows, "channels": ch, "r": r,
                    "io_dtype": "bf16" if dtype == torch.bfloat16 else "f32",
                    "fwd_GBps": round(alg / t_f / 1e9, 1), "bwd_GBps": round(alg / t_b / 1e9, 1),
                    "note": "algorithmic bytes = n*itemsize*(1 + 1/r) per kernel"})
        batch, tokens, chn, rank = 256, 197, 768, 30
        A = torch.randn(tokens * rank, device="cuda", generator=g)
        B = torch.randn(rank * chn, device="cuda", generator=g)
        xl = [torch.randn(batch * tokens * chn, device="cuda", generator=g).to(dtype) for _ in range(3)]
        yl = [torch.empty_like(x) for x in xl]
        t = timed(lambda i: binding.s2a_lrp_fwd(xl[i], A, B, yl[i], batch, tokens, chn, rank))
        out.append({"kernel": "lrp_fwd", "batch": batch, "tokens": tokens, "channels": chn, "rank": rank,
                    "io_dtype": "bf16" if dtype == torch.bfloat16 else "f32",
                    "GBps": round(2 * batch * tokens * chn * item / t / 1e9, 1),
                    "note": "algorithmic bytes = 2*n*itemsize (A and B stay in cache)"})
    return out


def _time_bits(seed: int):
    """The 2-bit and 8-bit forms on one ViT-B/16 block, bfloat16."""
    out = []
    g = torch.Generator(device="cuda").manual_seed(seed)
    for kind, rows, L in (("gelu", 12608, 3072), ("softmax", 151296, 197)):
        n = rows * L
        xs = [torch.randn(n, device="cuda", generator=g).to(torch.bfloat16) for _ in range(3)]
        ys = [torch.empty_like(x) for x in xs]
        for bits in (2, 8):
            codes = [torch.empty(binding.codes_bytes_bits(n, bits), dtype=torch.uint8, device="cuda") for _ in range(3)]
            meta = [torch.empty(2 * rows, dtype=torch.float32, device="cuda") for _ in range(3)]
            res = {}
            for name, fn in (("fwd", lambda i: binding.s2a_fwd_bits(kind, xs[i], ys[i], codes[i], meta[i], L, bits)),
                             ("bwd", lambda i: binding.s2a_bwd_bits(kind, xs[i], codes[i], meta[i], ys[i], L, bits))):
                for i in range(3):
                    fn(i)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(12):
                    fn(i % 3)
                e1.record()
                torch.cuda.synchronize()
                res[name] = (4 * n + n * bits // 8 + 8 * rows) / (e0.elapsed_time(e1) * 1e-3 / 12) / 1e9
            out.append({"kernel_pair": kind + "_bits", "bits": bits, "rows": rows, "row_len": L, "io_dtype": "bf16",
                        "fwd_GBps": round(res["fwd"], 1), "bwd_GBps": round(res["bwd"], 1),
                        "note": "pipelined path; algorithmic bytes = 4*n + n*bits/8 + 8*rows"})
    return out


def cases(quick: bool):
    out = []
    for n in ((1e6, 1e8) if quick else (1e6, 1e7, 1e8, 1e9, 2e9)):
        rows = max(2, int(n) // 4096)
        for dtype in (torch.bfloat16, torch.float32):
            out.append(("gelu", rows, 4096, dtype))
            if n == 1e8:
                out.append(("silu", rows, 4096, dtype))
    for L in (64, 197, 257, 1024, 4096):
        for rows in ((10**4, 10**6) if quick else (10**4, 10**5, 10**6, 10**7)):
            if rows * L > 2e9 or (quick and rows * L > 3e8):
                continue
            for dtype in (torch.bfloat16, torch.float32):
                out.append(("softmax", rows, L, dtype))
    # other attention widths (none a whole number of 16-byte vectors in bfloat16), about 1e8 elements
    for L in (() if quick else (49, 50, 145, 196, 198, 577, 1025)):
        for dtype in (torch.bfloat16, torch.float32):
            out.append(("softmax", max(32, 10**8 // L // 32 * 32), L, dtype))
    return out


def table(path: str) -> None:
    """Prints the compact table kept under profiles/ from the JSON lines of a sweep."""
    rows = [json.loads(l) for l in open(path) if l.startswith("{")]
    print("%-24s %-11s %-7s %-5s %9s %9s" % ("kernel pair", "rows", "row_len", "dtype", "fwd GB/s", "bwd GB/s"))
    for r in rows:
        if r.get("kernel_pair") in ("gelu", "silu", "softmax"):
            print("%-24s %-11d %-7d %-5s %9.0f %9.0f" % (r["kernel_pair"], r["rows"], r["row_len"], r["io_dtype"],
                                                         r["fwd_GBps"], r["bwd_GBps"]))
    print()
    for r in rows:
        if str(r.get("kernel_pair", "")).endswith("_bits"):
            print("%-24s %-11d %-7d %-5s %9.0f %9.0f   (Eq. 8 at %d bits)" % (r["kernel_pair"], r["rows"], r["row_len"], r["io_dtype"],
                                                                            r["fwd_GBps"], r["bwd_GBps"], r["bits"]))
    print()
    for r in rows:
        if r.get("kernel_pair") == "relu":
            print("relu (1-bit mask)        n=%-12d %-5s fwd %6.0f bwd %6.0f" % (r["elems"], r["io_dtype"], r["fwd_GBps"], r["bwd_GBps"]))
    print()
    for r in rows:
        if r.get("kernel") == "gelu_fwd_tensor_range":
            print("gelu_fwd_tensor_range    n=%-12d %-5s %6.0f GB/s (x read twice: 6.5 / 12.5 B per element)" % (r["elems"], r["io_dtype"], r["GBps"]))
    print()
    for r in rows:
        if r.get("kernel_pair") == "cap":
            print("cap                      [%d, %d] r=%d %-5s fwd %6.0f bwd %6.0f" % (r["rows"], r["channels"], r["r"], r["io_dtype"],
                                                                                     r["fwd_GBps"], r["bwd_GBps"]))
        if r.get("kernel") == "lrp_fwd":
            print("lrp_fwd                  %s" % json.dumps({k: v for k, v in r.items() if k != "note"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--seeds", type=int, default=5)
    ap.add_argument("--table", default="", help="print the compact table of a finished sweep's JSON lines and exit")
    args = ap.parse_args()
    if args.table:
        table(args.table)
        return
    for line in _time_side(0):
        print(json.dumps(line), flush=True)
    for line in _time_bits(0):
        print(json.dumps(line), flush=True)
    for n in ((10**6, 10**8) if args.quick else (10**6, 10**7, 10**8, 10**9, 2 * 10**9)):
        for dtype in (torch.bfloat16, torch.float32):
            res = []
            for seed in range(args.seeds):
                res.append(_time_relu(int(n), dtype, seed))
                torch.cuda.empty_cache()
            med = [statistics.median(r[k] for r in res) for k in range(3)]
            print(json.dumps({"kernel_pair": "relu", "elems": int(n), "io_dtype": "bf16" if dtype == torch.bfloat16 else "f32",
                              "seeds": args.seeds, "fwd_GBps": round(med[0], 1), "bwd_GBps": round(med[1], 1),
                              "fwd_bwd_GBps": round(med[2], 1),
                              "note": "algorithmic bytes = 2*n*itemsize + n/8 per kernel"}), flush=True)
    for n in ((10**6, 10**8) if args.quick else (10**6, 10**7, 10**8, 10**9)):
        for dtype in (torch.bfloat16, torch.float32):
            rows = max(2, int(n) // 4096)
            res = [_time_tensor_range(rows, 4096, dtype, seed) for seed in range(args.seeds)]
            torch.cuda.empty_cache()
            print(json.dumps({"kernel": "gelu_fwd_tensor_range", "rows": rows, "row_len": 4096, "elems": rows * 4096,
                              "io_dtype": "bf16" if dtype == torch.bfloat16 else "f32", "seeds": args.seeds,
                              "GBps": round(statistics.median(res), 1),
                              "note": "algorithmic bytes = 3*n*itemsize + n/2 + 8*rows (x is read twice)"}), flush=True)
    for kind, rows, L, dtype in cases(args.quick):
        res = []
        for seed in range(args.seeds):
            res.append(_time_pair(kind, rows, L, dtype, seed))
            torch.cuda.empty_cache()
        med = [statistics.median(r[k] for r in res) for k in range(3)]
        spread = max(r[2] for r in res) - min(r[2] for r in res)
        kid = {"gelu": binding.GELU_FWD, "silu": binding.SILU_FWD, "softmax": binding.SOFTMAX_FWD}[kind]
        print(json.dumps({
            "kernel_pair": kind, "rows": rows, "row_len": L, "elems": rows * L,
            "io_dtype": "bf16" if dtype == torch.bfloat16 else "f32", "seeds": args.seeds,
            "fwd_GBps": round(med[0], 1), "bwd_GBps": round(med[1], 1), "fwd_bwd_GBps": round(med[2], 1),
            "fwd_bwd_gelem_per_s": round(med[2] / ((2 * (2 if dtype == torch.bfloat16 else 4) + 0.5) + 8.0 / L), 2),
            "spread_GBps": round(spread, 1), "note": PEAK_NOTE,
            "plan": binding.s2a_describe_plan(kid, rows * L, L, binding.BF16 if dtype == torch.bfloat16 else binding.F32),
        }), flush=True)


if __name__ == "__main__":
    main()
