"""Builds libnb.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2211_00889_b200.build [--verbose] [--debug | --tuning]

Flavours (separate files, so that the shipped library is never replaced by one of them):
  libnb.so         the product
  libnb_debug.so   -DNB_DEBUG: every tile index, ring slot and global offset the kernels form is
                   range-checked on the device; a failed check skips the access and records a code
                   in the context's device error word (reported as NB_ERR_CUDA by nb_check_guards)
  libnb_tuning.so  -DNB_TUNING: the pipeline planner reads shape overrides from the environment
                   (NB_PIPELINE_TILE, _SLOTS, _CTAS_PER_SM, _ROWS, _GROUPS, _XSTAGES, _QPT) for sweeps
The binding loads libnb.so unless the environment variable NB_LIB_PATH names another file.
"""
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libnb.so")
SOURCES = ["nb_api.cu", "nb_kernels.cu", "nb_pipeline.cu", "nb_static.cu", "nb_host.cpp"]
FLAVOURS = {"": [], "debug": ["-DNB_DEBUG=1"], "tuning": ["-DNB_TUNING=1"]}


def lib_path(flavour=""):
    return os.path.join(HERE, "libnb%s.so" % ("_" + flavour if flavour else ""))


def _nvcc():
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(lib):
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "nb.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force=False, verbose=False, flavour=""):
    """Compiles every CUDA source of the package into libnb.so (or a flavour of it); returns its path."""
    lib = lib_path(flavour)
    if not force and not _stale(lib):
        return lib
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC,-ffp-contract=off",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-shared", "-o", lib] + FLAVOURS[flavour]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
    if verbose:
        print(r.stdout + r.stderr)
    return lib


if __name__ == "__main__":
    fl = "debug" if "--debug" in sys.argv else "tuning" if "--tuning" in sys.argv else ""
    print(build_library(force=True, verbose="--verbose" in sys.argv, flavour=fl))
