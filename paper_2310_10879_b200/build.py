"""Build libbload.so (sm_100a only) next to this file.  `python -m paper_2310_10879_b200.build`."""
from __future__ import annotations

import glob
import hashlib
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libbload.so")
DEBUG_LIB = os.path.join(PKG, "libbload_debug.so")
STAMP = LIB + ".sources"  # digest of the sources the library was built from (times of files do not survive a copy)


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def source_digest(extra: str = "") -> str:
    h = hashlib.sha256(extra.encode())
    deps = sources() + sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + sorted(glob.glob(os.path.join(ROOT, "include", "*.h")))
    for d in deps:
        h.update(os.path.basename(d).encode())
        with open(d, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def stale(lib: str = LIB, extra: str = "") -> bool:
    """True when `lib` is missing or was not built from the sources as they are now."""
    try:
        with open(lib + ".sources") as f:
            return not os.path.exists(lib) or f.read().strip() != source_digest(extra)
    except OSError:
        return True


def nvcc_path() -> str:
    for c in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if c and os.path.exists(c):
            return c
    raise RuntimeError("nvcc not found: libbload cannot be built")


def build(force: bool = False, verbose: bool = False, debug: bool = False, defines: tuple = (), out: str | None = None) -> str:
    """Compile the library.  debug=True builds libbload_debug.so with -DBLOAD_DEBUG: every global access of the
    copy, metadata and table kernels is checked against the bounds of its buffer (see bload_debug_status).
    defines / out: a variant with other tuning constants (e.g. ("BLOAD_STAGED_MAX_RUN=-1",) sends every frame size
    through the register-path copy kernel) written to `out`; load it with BLOAD_LIBRARY to compare."""
    lib = out or (DEBUG_LIB if debug else LIB)
    extra = ("debug" if debug else "") + " ".join(defines)
    if not force and not stale(lib, extra):
        return lib
    tmp = lib + ".tmp%d" % os.getpid()
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if debug:
        cmd += ["-DBLOAD_DEBUG=1"]
    cmd += ["-D" + d for d in defines]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += sources() + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    with open(lib + ".sources", "w") as f:
        f.write(source_digest(extra) + "\n")
    return lib


if __name__ == "__main__":
    argv = sys.argv[1:]
    defs = tuple(argv[i + 1] for i, a in enumerate(argv[:-1]) if a == "--define")
    out_path = next((argv[i + 1] for i, a in enumerate(argv[:-1]) if a == "--out"), None)
    if defs and not out_path:
        sys.exit("--define needs --out: the in-tree library is always built with the default constants")
    print(build(force="--force" in argv, verbose="-v" in argv, debug="--debug" in argv, defines=defs, out=out_path))
