"""Builds libha_la.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2609_32114_b200.build [--force] [--verbose] [--profile]

--profile builds a second library, libha_la_prof.so, with -DHA_LA_PROFILE_PHASES: the tensor-core kernels then
record clock64 / %globaltimer stamps at their phase boundaries (csrc/prof.cuh) and the library exports
ha_la_debug_read_prof_prep / _chain to read them; `python -m paper_2609_32114_b200.prof_phases` prints them.
The normal library contains none of this (the macros expand to nothing).

Objects are cached under paper_2609_32114_b200/build/ and rebuilt when their source, any
header, or this script changes; translation units compile in parallel.
"""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libha_la.so")
INCLUDE = os.path.join(ROOT, "include")

# (object name, source, extra flags)
UNITS = [("api", "api.cu", []), ("plan", "plan.cu", []), ("tc", "tc.cu", []), ("tc_prep", "tc_prep.cu", []), ("tc_chain", "tc_chain.cu", []), ("tc_seg", "tc_seg.cu", []),
         ("noalloc", "noalloc.cu", []), ("decode", "decode.cu", [])] + [
    (f"simt{u}", "simt.cu", [f"-DHA_LA_SIMT_UNIT={u}"]) for u in range(5)
]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    return os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def _headers_mtime() -> float:
    t = os.path.getmtime(os.path.abspath(__file__))
    for d in (CSRC, INCLUDE):
        for f in os.listdir(d):
            if f.endswith((".cuh", ".h")):
                t = max(t, os.path.getmtime(os.path.join(d, f)))
    return t


def _compile(unit, verbose: bool, obj_dir: str = OBJ, more=()):
    name, src, extra = unit
    extra = list(extra) + list(more)
    out = os.path.join(obj_dir, name + ".o")
    cmd = [_nvcc(), *ARCH, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-I", CSRC, "-I", INCLUDE,
           *extra, "-c", os.path.join(CSRC, src), "-o", out]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    return name, r.returncode, r.stdout + r.stderr


def build(force: bool = False, verbose: bool = False, extra_flags=(), lib_path: str = LIB, obj_dir: str = OBJ) -> str:
    """Compile what is stale and link.  `extra_flags`, `lib_path`, `obj_dir` serve developer builds."""
    os.makedirs(obj_dir, exist_ok=True)
    hdr = _headers_mtime()
    todo = []
    for unit in UNITS:
        out = os.path.join(obj_dir, unit[0] + ".o")
        src_t = os.path.getmtime(os.path.join(CSRC, unit[1]))
        if force or not os.path.exists(out) or os.path.getmtime(out) < max(src_t, hdr):
            todo.append(unit)
    if todo:
        with cf.ThreadPoolExecutor(max_workers=min(len(todo), os.cpu_count() or 4)) as ex:
            for name, rc, log in ex.map(lambda u: _compile(u, verbose, obj_dir, extra_flags), todo):
                if verbose or rc != 0:
                    sys.stderr.write(f"--- {name}\n{log}\n")
                if rc != 0:
                    raise RuntimeError(f"nvcc failed on {name}")
    objs = [os.path.join(obj_dir, u[0] + ".o") for u in UNITS]
    if todo or not os.path.exists(lib_path) or os.path.getmtime(lib_path) < max(os.path.getmtime(o) for o in objs):
        tmp = lib_path + f".tmp{os.getpid()}"
        subprocess.check_call([_nvcc(), *ARCH, "-shared", "-o", tmp, *objs])
        os.replace(tmp, lib_path)
    return lib_path


PROF_LIB = os.path.join(PKG, "libha_la_prof.so")


def build_profile(force: bool = False, verbose: bool = False) -> str:
    """The instrumented developer build (see the module docstring)."""
    return build(force=force, verbose=verbose, extra_flags=["-DHA_LA_PROFILE_PHASES"], lib_path=PROF_LIB,
                 obj_dir=os.path.join(PKG, "build_prof"))


if __name__ == "__main__":
    if "--profile" in sys.argv:
        print(build_profile(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
