"""Build paper_1901_08924_b200/liblpcsvrg.so (the C-ABI library) with nvcc for sm_100a.

    python -m paper_1901_08924_b200.build [--force] [--verbose] [--trace]

--trace builds liblpcsvrg_trace.so instead: the same sources with -DLPC_TRACE, in which one CTA of the one-launch loop
and of the streaming worker kernel stamps %globaltimer at every phase boundary (read by paper_1901_08924_b200.trace).

-fmad=false: the packed codes are defined with separate round-to-nearest multiplies and adds, so
the compiler must not contract them into fused multiply-adds anywhere in the library.
"""
import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "liblpcsvrg.so")
SOURCES = ["lpc_api.cu", "lpc_quantize.cu", "lpc_aggregate.cu", "lpc_snapshot.cu", "lpc_inner.cu", "lpc_persist.cu", "lpc_noalloc.cu"]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-fmad=false",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _newest_dep():
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(os.path.dirname(HERE), "include", "lpc.h")]
    return max(os.path.getmtime(p) for p in deps)


TRACE_LIB = os.path.join(HERE, "liblpcsvrg_trace.so")


def build(force=False, verbose=False, trace=False):
    sources = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    lib = TRACE_LIB if trace else LIB
    objdir = os.path.join(OBJ, "trace") if trace else OBJ
    flags = NVCC_FLAGS + (["-DLPC_TRACE"] if trace else [])
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_dep():
        return lib
    os.makedirs(objdir, exist_ok=True)
    nvcc = _nvcc()

    def compile_one(src):
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        cmd = [nvcc, *flags, "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        with open(os.path.join(objdir, src + ".ptxas.log"), "w") as f:
            f.write(r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{r.stderr[-4000:]}")
        if verbose:
            print(r.stderr)
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        objs = list(ex.map(compile_one, sources))
    cmd = [nvcc, "-shared", "-cudart", "static", "-o", lib + ".tmp", *objs]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stderr[-4000:]}")
    os.replace(lib + ".tmp", lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, trace="--trace" in sys.argv))
