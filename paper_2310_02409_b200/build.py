"""Compile ``csrc/*.cu`` into ``libdodo.so`` with nvcc for sm_100a (in-tree, next to this file)."""
from __future__ import annotations

import os
import subprocess
from pathlib import Path

_PKG = Path(__file__).resolve().parent
_CSRC = _PKG / "csrc"
_INCLUDE = _PKG.parent / "include"
_BUILD = _PKG / "_build"
LIB_PATH = _PKG / "libdodo.so"

NVCC_FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (cand == "nvcc" or Path(cand).exists()):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(out: Path, deps) -> bool:
    return not out.exists() or any(out.stat().st_mtime < Path(d).stat().st_mtime for d in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    """Build the shared library if any source is newer than it.  Returns its path."""
    sources = sorted(_CSRC.glob("*.cu"))
    headers = sorted(_CSRC.glob("*.cuh")) + sorted(_INCLUDE.glob("*.h"))
    _BUILD.mkdir(exist_ok=True)
    objs = []
    procs = []
    for src in sources:
        obj = _BUILD / (src.stem + ".o")
        objs.append(obj)
        if force or _stale(obj, [src] + headers):
            cmd = [_nvcc(), *NVCC_FLAGS, "-I", str(_INCLUDE), "-I", str(_CSRC), "-c", str(src), "-o", str(obj)]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for src, p in procs:
        out, _ = p.communicate()
        if verbose and out:
            print(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src.name}:\n{out}")
    if force or procs or _stale(LIB_PATH, objs):
        tmp = LIB_PATH.with_suffix(f".so.tmp{os.getpid()}")
        cmd = [_nvcc(), "-shared", "-o", str(tmp), *map(str, objs), "-cudart", "static"]
        r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"link failed:\n{r.stdout}")
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
