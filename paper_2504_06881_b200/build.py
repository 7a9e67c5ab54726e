"""Builds libtconv.so (CUDA kernels + C ABI) for sm_100a with nvcc, in-tree.

The tiled forward kernels are compiled as one translation unit per (mode, channel
combine) family, in parallel, and linked with the API unit into one shared library.
"""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libtconv.so"
OBJ = PKG / "build"

# (exported launcher, tconv_mode_t, channel combine: 1 sum, 2 max, 3 min)
FWD_INSTANCES = [("fwd_inst_maxplus_sum", 0, 1), ("fwd_inst_maxplus_max", 0, 2),
                 ("fwd_inst_maxplus_min", 0, 3), ("fwd_inst_minplus_sum", 1, 1),
                 ("fwd_inst_minplus_max", 1, 2), ("fwd_inst_minplus_min", 1, 3),
                 ("fwd_inst_compound", 2, 1), ("fwd_inst_parallel", 3, 1)]


def _newest_source() -> float:
    files = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + \
        list((ROOT / "include").glob("*.h")) + [Path(__file__)]
    return max(f.stat().st_mtime for f in files)


def _nvcc_base(verbose: bool):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-I", str(ROOT / "include"), "-I", str(CSRC)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    return cmd


def _compile(job):
    src, obj, defs, verbose = job
    cmd = _nvcc_base(verbose) + defs + ["-c", str(src), "-o", str(obj)]
    r = subprocess.run(cmd, capture_output=True, text=True)
    return obj, r.returncode, r.stdout + r.stderr


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile the library if it is missing or older than any source file."""
    if not force and LIB.exists() and LIB.stat().st_mtime >= _newest_source():
        return LIB
    OBJ.mkdir(exist_ok=True)
    jobs = [(CSRC / "tconv_api.cu", OBJ / "tconv_api.o", [], verbose),
            (CSRC / "tconv3d_api.cu", OBJ / "tconv3d_api.o", [], verbose)]
    for name, mode, chan in FWD_INSTANCES:
        defs = [f"-DTCONV_INST_NAME={name}", f"-DTCONV_INST_MODE={mode}", f"-DTCONV_INST_CHAN={chan}"]
        jobs.append((CSRC / "tconv_fwd_inst.cu", OBJ / f"{name}.o", defs, verbose))
    log = []
    with cf.ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as ex:
        for obj, rc, out in ex.map(_compile, jobs):
            log.append(f"== {obj.name}\n{out}")
            if rc != 0:
                raise RuntimeError(f"nvcc failed for {obj.name}:\n{out}")
    if verbose:
        print("\n".join(log))
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp.so")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "--cudart", "shared"] + \
          [str(j[1]) for j in jobs] + ["-o", str(tmp)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
