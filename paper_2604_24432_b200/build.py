"""Builds the C-ABI shared library ``libksa_b200.so`` in-tree with nvcc for sm_100a."""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libksa_b200.so")
OBJ_DIR = os.path.join(HERE, "_build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr",
]


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _deps():
    hdrs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    hdrs += [os.path.join(ROOT, "include", f) for f in os.listdir(os.path.join(ROOT, "include")) if f.endswith(".h")]
    return hdrs


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


# Variants of the library for the tests (each in its own object folder, beside the product library):
#   "debug": every source with -DKSA_DEBUG -- the kernels check each global output index against the tensor's extent,
#            record a status code and skip the access instead of making it (the stand-in for a memory checker);
#   "asan":  the host logic (ksa_api.cu: validation, layout, schedule) under -fsanitize=address,undefined, the kernels
#            as in the product build; to be loaded into a process that preloads the sanitizer runtime.
VARIANTS = {
    "debug": dict(flags=("-DKSA_DEBUG",), only=None, link=()),
    "asan": dict(flags=("-Xcompiler", "-fsanitize=address", "-Xcompiler", "-fsanitize=undefined",       # (nvcc splits at commas)
                        "-Xcompiler", "-fno-omit-frame-pointer", "-g"),
                 only=("ksa_api.cu",), link=("-Xcompiler", "-fsanitize=address", "-Xcompiler", "-fsanitize=undefined")),
}


def variant_path(variant: str) -> str:
    return os.path.join(HERE, "libksa_b200_%s.so" % variant)


def build(force: bool = False, verbose: bool = False, extra_flags=(), variant: str = None) -> str:
    lib_path, obj_dir, link_flags, only = LIB, OBJ_DIR, (), None
    if variant is not None:
        if variant == "asan":
            build(force=force, verbose=verbose)          # the other objects come from the product build
        v = VARIANTS[variant]
        lib_path, obj_dir = variant_path(variant), os.path.join(HERE, "_build_" + variant)
        extra_flags, link_flags, only = tuple(extra_flags) + v["flags"], v["link"], v["only"]
    os.makedirs(obj_dir, exist_ok=True)
    newest_hdr = max(os.path.getmtime(h) for h in _deps())
    jobs = []
    objs = []
    for src in _sources():
        if only is not None and os.path.basename(src) not in only:
            objs.append(os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o"))
            continue
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), newest_hdr)
        if stale:
            jobs.append([_nvcc(), *NVCC_FLAGS, *extra_flags, "-c", src, "-o", obj])

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, len(jobs))) as ex:
        list(ex.map(run, jobs))
    newest_obj = max(os.path.getmtime(o) for o in objs)
    if jobs or not os.path.exists(lib_path) or os.path.getmtime(lib_path) < newest_obj:
        tmp = lib_path + ".tmp.%d" % os.getpid()
        run([_nvcc(), "-shared", "-o", tmp, *objs, *link_flags, "-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    variant = next((a.split("=", 1)[1] for a in sys.argv if a.startswith("--variant=")), None)
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv,
                extra_flags=("-Xptxas", "-v") if "--ptxas" in sys.argv else (), variant=variant))
