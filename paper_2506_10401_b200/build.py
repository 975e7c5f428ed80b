"""Builds libhct.so in-tree.

    python -m paper_2506_10401_b200.build [--force]

Host code is C++17; device code under csrc/kernels/*.cuh is embedded as text and compiled for
sm_100a at graph-creation time, csrc/*.cu files (if any) are compiled here with nvcc for sm_100a.
"""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
BUILD = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "libhct.so")
CUDA_HOME = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def _embed_skeletons() -> str:
    os.makedirs(BUILD, exist_ok=True)
    out = os.path.join(BUILD, "skeletons.inc")
    parts = ["static const Skeleton kSkeletons[] = {\n"]
    for path in sorted(glob.glob(os.path.join(CSRC, "kernels", "*.cuh"))):
        name = os.path.splitext(os.path.basename(path))[0]
        text = open(path).read()
        assert ')HCTSRC"' not in text
        # split long sources: some compilers cap the length of one string literal
        chunks = [text[i:i + 12000] for i in range(0, len(text), 12000)] or [""]
        lit = "\n".join('R"HCTSRC(' + c + ')HCTSRC"' for c in chunks)
        parts.append('  {"%s", %s},\n' % (name, lit))
    parts.append("};\n")
    new = "".join(parts)
    if not os.path.exists(out) or open(out).read() != new:
        with open(out, "w") as f:
            f.write(new)
    return out


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cpp"))), sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = glob.glob(os.path.join(CSRC, "**", "*"), recursive=True) + [os.path.join(PKG, "..", "include", "hct.h"), __file__]
    return any(os.path.isfile(d) and os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    _embed_skeletons()
    cpp, cu = _sources()
    nvcc = shutil.which("nvcc") or os.path.join(CUDA_HOME, "bin", "nvcc")
    objs = []
    for src in cpp:
        obj = os.path.join(BUILD, os.path.basename(src) + ".o")
        cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-Wall", "-Wextra", "-fvisibility=hidden", "-I", BUILD, "-c", src, "-o", obj]
        if verbose:
            print(" ".join(cmd))
        subprocess.run(cmd, check=True)
        objs.append(obj)
    for src in cu:
        obj = os.path.join(BUILD, os.path.basename(src) + ".o")
        cmd = [nvcc, "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-Xcompiler", "-fPIC,-fvisibility=hidden",
               "-I", BUILD, "-c", src, "-o", obj]
        if verbose:
            print(" ".join(cmd))
        subprocess.run(cmd, check=True)
        objs.append(obj)
    link = ["g++", "-shared", "-o", LIB] + objs + ["-ldl", "-lpthread"]
    if cu:
        link += ["-L", os.path.join(CUDA_HOME, "lib64"), "-lcudart_static", "-lrt"]
    if verbose:
        print(" ".join(link))
    subprocess.run(link, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
