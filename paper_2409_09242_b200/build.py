"""Builds libadahess.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every translation unit is compiled to an object of its own, side by side (the fused local
step is instantiated in six of them, one per combination of Hessian power and weight
decay), and the objects are linked into one shared library."""
from __future__ import annotations

import os
import shutil
import subprocess
from concurrent.futures import ThreadPoolExecutor

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
_OBJ = os.path.join(_PKG, "_build")
_INCLUDE = os.path.join(os.path.dirname(_PKG), "include")
# ADAHESS_LIB points the binding at another build of the same library (e.g. one
# compiled with different tile constants); by default the in-tree build is used.
LIB_PATH = os.environ.get("ADAHESS_LIB") or os.path.join(_PKG, "libadahess.so")
SOURCES = ["ah_kernels.cu", "ah_host.cu", "ah_noalloc.cu", "ah_exchange_async.cu", "ah_sgd.cu",
           "ah_partition.cu", "ah_dynamic.cu", "ah_selftest.cu"]
STEP_INSTANCES = 6          # ah_step_inst.cu, compiled with -DAH_STEP_INST=0 .. 5
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-ffp-contract=off"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)] + [os.path.join(_INCLUDE, "adahess.h")]
    return any(os.path.getmtime(d) > built for d in deps)


def units(defines=()):
    """(source, extra flags, object) of every translation unit."""
    out = [(s, list(defines), os.path.splitext(s)[0] + ".o") for s in SOURCES]
    out += [("ah_step_inst.cu", [*defines, f"-DAH_STEP_INST={k}"], f"ah_step_inst_{k}.o")
            for k in range(STEP_INSTANCES)]
    return out


def build(force: bool = False, verbose: bool = False, defines=(), lib_path: str | None = None,
          obj_dir: str | None = None) -> str:
    """Compile the library if it is missing or older than its sources.  `defines` (e.g.
    ["-DAH_PASSES=2"]), `lib_path` and `obj_dir` build a variant somewhere else."""
    lib_path = lib_path or LIB_PATH
    obj_dir = obj_dir or _OBJ
    if not force and lib_path == LIB_PATH and not is_stale():
        return LIB_PATH
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    logs = {}

    def compile_one(unit):
        src, extra, obj = unit
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", _INCLUDE, "-I", _CSRC, "-c", os.path.join(_CSRC, src),
               "-o", os.path.join(obj_dir, obj)]
        if verbose:
            cmd[1:1] = ["-Xptxas", "-v"]
        done = subprocess.run(cmd, capture_output=True, text=True)
        logs[obj] = done.stdout + done.stderr
        if done.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src} {extra}:\n{logs[obj][-4000:]}")
        return os.path.join(obj_dir, obj)

    todo = units(defines)
    with ThreadPoolExecutor(max_workers=min(len(todo), os.cpu_count() or 4)) as pool:
        objects = list(pool.map(compile_one, todo))
    if verbose:
        for obj in sorted(logs):
            print(f"==== {obj}\n{logs[obj]}")
    tmp = lib_path + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", *objects, "-o", tmp])
    os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force=True, verbose=True))
