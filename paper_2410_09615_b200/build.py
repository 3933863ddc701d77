"""In-tree build of libslim.so (nvcc, sm_100a only)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libslim.so")
SOURCES = ["api.cu", "pack.cu", "repack.cu", "fwd_simple.cu", "fwd_decode.cu", "fwd_decode_tiled.cu", "fwd_prefill.cu",
           "fwd_noalloc.cu", "adapter_q.cu", "quant_search.cu", "mask.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC", "--use_fast_math"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "slim.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, defines=(), out: str | None = None) -> str:
    """Compile every CUDA source into ``libslim.so`` next to this file.

    ``defines``: extra ``-D`` macros, the kernels' optional hooks: ``SLIM_DECODE_TUNE`` (the environment
    variable SLIM_RING overrides the tiled decode kernel's ring depth), ``SLIM_DECODE_TRACE``,
    ``SLIM_TILED_TRACE`` and ``SLIM_PREFILL_TRACE`` (per-CTA timelines of the three kernels, read back
    with the ``slim_debug_read_*`` functions such a build exports).  A build with hooks goes to ``out``
    (required then), never to the library the package loads by default."""
    if defines and not out:
        raise ValueError("a build with extra defines needs its own output path")
    if not defines and not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    bdir = os.path.join(HERE, "_build" + ("_" + "_".join(sorted(defines)) if defines else ""))
    os.makedirs(bdir, exist_ok=True)
    procs = []
    for src in SOURCES:
        obj = os.path.join(bdir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *[f"-D{d}" for d in defines], "-I", INCLUDE, "-I", CSRC, "-c", os.path.join(CSRC, src),
               "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, pr in procs:
        log, _ = pr.communicate()
        if pr.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{log}")
        if verbose and log:
            print(log)
    target = out or LIB
    tmp = target + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-shared", "-o", tmp, *objs, "-cudart", "static"])
    os.replace(tmp, target)
    return target


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
