"""Builds ``libccdc.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libccdc.so"
SOURCES = ["ccdc_plan.cpp", "ccdc_kernels.cu", "ccdc_map.cu", "ccdc_map_cluster.cu", "ccdc_multi.cu", "ccdc_stream.cu"]


def nvcc_command(out: Path, verbose: bool = False, defines: tuple[str, ...] = ()) -> list[str]:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "--threads", "0", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC,-Wall", "-shared", "-cudart", "static",
           "-I", str(ROOT / "include"), "-I", str(CSRC), "-o", str(out)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [f"-D{d}" for d in defines]
    return cmd + [str(CSRC / s) for s in SOURCES]


def needs_build() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*")) + [ROOT / "include" / "ccdc.h"]
    return any(d.stat().st_mtime > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> Path:
    """Compile the library if it is missing or older than its sources."""
    if not force and not needs_build():
        return LIB
    tmp = PKG / f"libccdc.{os.getpid()}.tmp.so"
    res = subprocess.run(nvcc_command(tmp, verbose), capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        tmp.unlink(missing_ok=True)
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, LIB)
    return LIB


def build_variant(out: Path, defines: tuple[str, ...]) -> Path:
    """Compile the library with extra -D options (build-time kernel choices) into ``out``."""
    res = subprocess.run(nvcc_command(out, defines=defines), capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return out


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
