"""Builds liblstm_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "liblstm_b200.so"
LIB_CHECKED = PKG / "liblstm_b200_checked.so"       # same sources with -DLSTM_B200_CHECKED: index checks inside the kernels
INCLUDE = PKG.parent / "include"
SOURCES = ["api.cu", "recur.cu", "proj_simt.cu", "proj_tc.cu", "noalloc.cu", "recur_mma.cu", "hlstm_mma.cu", "recur_tc.cu", "host_tools.cu", "recur_csr.cu", "csr_pack.cu", "compact.cu", "recur_wave.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--use_fast_math=false"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(target: Path, deps) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(Path(d).stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> Path:
    """Compile every .cu under csrc/ and link the shared library next to this file (``checked``: the build
    with index checks, liblstm_b200_checked.so)."""
    sources = [s for s in SOURCES if (CSRC / s).exists()]
    headers = list(CSRC.glob("*.cuh")) + list(INCLUDE.glob("*.h"))
    objdir = PKG / ("_build_checked" if checked else "_build")
    lib = LIB_CHECKED if checked else LIB
    objdir.mkdir(exist_ok=True)
    nvcc = _nvcc()
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
    if checked:
        flags += ["-DLSTM_B200_CHECKED"]
    if verbose:
        flags += ["-Xptxas", "-v"]

    def compile_one(src: str):
        obj = objdir / (src + ".o")
        if force or _stale(obj, [CSRC / src, *headers, Path(__file__)]):
            cmd = [nvcc, *flags, "-I", str(INCLUDE), "-c", str(CSRC / src), "-o", str(obj)]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
            if verbose:
                sys.stderr.write(r.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(sources))) as ex:
        objs = list(ex.map(compile_one, sources))
    if force or _stale(lib, objs):
        tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp), *map(str, objs)]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
