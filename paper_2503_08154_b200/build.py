"""Builds libs2a.so in-tree with nvcc for sm_100a (no GPU needed to compile).

    python -m paper_2503_08154_b200.build [--force] [-v] [--tuning]

--tuning builds a SECOND library, libs2a_tuning.so, with -DS2A_TUNING: the only build in
which the launch-shape planner honours its S2A_* environment overrides (for sweeps; load
it with binding.use_library).  libs2a.so itself reads no environment variable.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
OUT = os.path.join(HERE, "libs2a.so")
SOURCES = ["s2a_api.cu", "s2a_rowwise.cu", "s2a_relu.cu", "s2a_side.cu", "s2a_tensor_range.cu", "s2a_tile.cu", "s2a_tile_gelu_fwd.cu",
           "s2a_tile_gelu_bwd.cu", "s2a_tile_softmax_fwd.cu", "s2a_tile_softmax_bwd.cu", "s2a_tile_silu.cu", "s2a_tile_bits.cu", "s2a_tile_softmax_widths.cu"]
HEADERS = ["s2a_common.cuh", "s2a_launch.h", "s2a_tile.cuh", os.path.join("..", "..", "include", "s2a.h")]

ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
NVCC_FLAGS = [*ARCH, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _newer(deps, target) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, tuning: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    hdrs = [os.path.join(CSRC, h) for h in HEADERS] + [os.path.abspath(__file__)]
    obj_dir = OBJ + "_tuning" if tuning else OBJ
    out = os.path.join(HERE, "libs2a_tuning.so") if tuning else OUT
    os.makedirs(obj_dir, exist_ok=True)
    jobs = []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(obj_dir, src[:-3] + ".o")
        if force or _newer([path, *hdrs], obj):
            jobs.append([nvcc, *NVCC_FLAGS, *(["-DS2A_TUNING"] if tuning else []),
                         *(["-Xptxas", "-v"] if verbose else []), "-c", path, "-o", obj])

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, r

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as pool:
            for cmd, r in pool.map(run, jobs):
                if verbose or r.returncode != 0:
                    sys.stderr.write(r.stdout + r.stderr)
                if r.returncode != 0:
                    raise RuntimeError("nvcc failed: " + " ".join(cmd))
    objs = [os.path.join(obj_dir, s[:-3] + ".o") for s in SOURCES]
    if jobs or _newer(objs, out):
        subprocess.run([nvcc, *ARCH, "-shared", *objs, "-o", out + ".tmp"], check=True)
        os.replace(out + ".tmp", out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, tuning="--tuning" in sys.argv))
