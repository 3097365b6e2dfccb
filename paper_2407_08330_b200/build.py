"""Build libhdt.so (CUDA, sm_100a) in-tree with nvcc.  No GPU is needed to compile."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhdt.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--use_fast_math", "-Xcompiler", "-fPIC", "-shared", "-Xptxas", "-v",
]
# HDT_WORKBENCH=1 in the environment also compiles the instrumented instantiations (option
# "phase_stamps") and the persistent forward kept for comparisons (option "no_persistent" = 2); a
# default build leaves them out and those option values fall back to the default kernels.
if os.environ.get("HDT_WORKBENCH", "0") not in ("", "0"):
    NVCC_FLAGS.append("-DHDT_WORKBENCH")
# --use_fast_math is limited to the intrinsics it maps (exp2f/log2f/division in the kernels are
# already the approximate forms the tolerances were derived for); host code is unaffected.


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(HERE, "..", "include", "*.h")) + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu of csrc/ to an object file (in parallel; objects whose sources and headers
    are older are reused unless `force`) and link them into libhdt.so."""
    if not force and not needs_build():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    hdrs = glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h")) + \
        [os.path.abspath(__file__)]
    t_hdr = max(os.path.getmtime(h) for h in hdrs)
    flags = [f for f in NVCC_FLAGS if f != "-shared"]

    def compile_one(src):
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        log = obj + ".log"
        if not force and os.path.exists(obj) and os.path.exists(log) and \
                os.path.getmtime(obj) > max(os.path.getmtime(src), t_hdr):
            return obj, 0, open(log).read()
        res = subprocess.run([nvcc] + flags + ["-c", "-o", obj, src], capture_output=True, text=True)
        out = res.stdout + res.stderr
        if res.returncode == 0:
            with open(log, "w") as f:
                f.write(out)
        return obj, res.returncode, out

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(compile_one, sources()))
    info = "".join(out for _, _, out in results)
    failed = [r for r in results if r[1] != 0]
    if verbose or failed:
        sys.stderr.write("".join(out for _, rc, out in results if verbose or rc != 0))
    if failed:
        raise RuntimeError("nvcc failed building libhdt.so")
    tmp = LIB + f".tmp{os.getpid()}"
    res = subprocess.run([nvcc, "-shared", "-o", tmp] + [r[0] for r in results] + ["-lcudart"],
                         capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking libhdt.so")
    os.replace(tmp, LIB)
    with open(os.path.join(HERE, "ptxas_info.txt"), "w") as f:
        f.write(info)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
