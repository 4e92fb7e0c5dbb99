"""Build the CUDA library (``libaweq.so``) in-tree with nvcc for sm_100a.

``python -m paper_2311_01305_b200.build`` compiles every ``csrc/*.cu`` to an
object file (in parallel), links them into ``paper_2311_01305_b200/libaweq.so``
and prints the ptxas resource usage when ``--verbose`` is given.  A GPU is not
needed to build.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libaweq.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--ftz=false", "--prec-div=true", "--prec-sqrt=true", "--fmad=true",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v",
]


def _cutlass_flags() -> list:
    """Include paths of a CUTLASS 3.x/4.x header tree with the sm_100 collectives (the forward
    check's tensor-core GEMMs are instantiated from them).  ``AWEQ_CUTLASS`` names the tree;
    otherwise the copies vendored inside Python packages are searched.  Without one the GEMM
    translation units compile to stubs that return AWEQ_ERR_UNSUPPORTED."""
    import sysconfig
    roots = [os.environ.get("AWEQ_CUTLASS")]
    for sp in {sysconfig.get_paths()["purelib"], sysconfig.get_paths()["platlib"]}:
        roots += [os.path.join(sp, "flashinfer", "data", "cutlass"), os.path.join(sp, "tilelang", "3rdparty", "cutlass")]
    for r in roots:
        if r and os.path.exists(os.path.join(r, "include", "cutlass", "gemm", "collective", "builders",
                                             "sm100_umma_builder.inl")):
            return ["-I" + os.path.join(r, "include"), "-I" + os.path.join(r, "tools", "util", "include"),
                    "--expt-relaxed-constexpr"]
    return ["-DAWEQ_NO_CUTLASS"]


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.isabs(c) and os.path.exists(c) or not os.path.isabs(c)):
            return c
    return "nvcc"


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in paths)


def _compile(src: str, obj: str, verbose: bool) -> str:
    extra = _cutlass_flags() if os.path.basename(src).startswith("forward_gemm") else []
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-c", src, "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, r.stdout, r.stderr))
    return r.stderr if verbose else ""


def build(force: bool = False, verbose: bool = False) -> str:
    """Build when the library is missing or older than a source; returns its path.  Serialised with
    a file lock, so that several ranks starting together compile once."""
    import fcntl
    os.makedirs(OBJ, exist_ok=True)
    with open(os.path.join(OBJ, ".lock"), "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            return _build_locked(force, verbose)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)


def _build_locked(force: bool, verbose: bool) -> str:
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    headers = glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) + [
        os.path.join(os.path.dirname(HERE), "include", "aweq.h"), os.path.abspath(__file__)]
    os.makedirs(OBJ, exist_ok=True)
    objs = [os.path.join(OBJ, os.path.basename(s)[:-3] + ".o") for s in srcs]
    # an object is stale when its source, a header it includes (directly: the headers here do not
    # include one another beyond common.cuh / kernels.h / aweq.h) or this script is newer
    def stale(src, obj):
        if force or not os.path.exists(obj):
            return True
        text = open(src).read()
        deps = [src, os.path.abspath(__file__)]
        for h in headers:
            name = os.path.basename(h)
            if name in ("common.cuh", "kernels.h", "aweq.h") or ('"%s"' % name) in text:
                deps.append(h)
        return os.path.getmtime(obj) < _newest(deps)
    todo = [(s, o) for s, o in zip(srcs, objs) if stale(s, o)]
    if not todo and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest(objs):
        return LIB
    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        logs = list(ex.map(lambda so: _compile(so[0], so[1], verbose), todo))
    if verbose:
        sys.stderr.write("\n".join(logs))
    cmd = [_nvcc(), "-shared", "-o", LIB, *objs, "-Xcompiler", "-fPIC"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("link failed:\n%s\n%s" % (r.stdout, r.stderr))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
