"""Builds libqevict.so (sm_100a) in-tree with nvcc: one object per .cu, compiled in parallel."""

import concurrent.futures
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libqevict.so")
# the same sources with -DQEVICT_TRACE: every step kernel stamps %globaltimer at its first CTA's start and its
# last CTA's end (qevict_kernel_timeline reads the stamps); a separate library, so that the normal one carries
# none of it
OBJ_TRACE = os.path.join(HERE, "build_trace")
LIB_TRACE = os.path.join(HERE, "libqevict_trace.so")
# the same sources with -DQEVICT_DEBUG_BOUNDS: every index a kernel reads from a table is range-checked before use
# (recorded and skipped, never trapped) and the pools start as NaN; the parity tests run against it once
OBJ_CHECK = os.path.join(HERE, "build_check")
LIB_CHECK = os.path.join(HERE, "libqevict_check.so")
_VARIANTS = {None: (OBJ, LIB, []), "trace": (OBJ_TRACE, LIB_TRACE, ["-DQEVICT_TRACE"]),
             "check": (OBJ_CHECK, LIB_CHECK, ["-DQEVICT_DEBUG_BOUNDS"])}

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
]


def _nvcc():
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _stale(lib=LIB):
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "qevict.h"))
    deps.append(os.path.abspath(__file__))
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(nvcc, src, verbose, variant=None):
    obj_dir, _, defs = _VARIANTS[variant]
    obj = os.path.join(obj_dir, src[:-3] + ".o")
    cmd = [nvcc] + NVCC_FLAGS + defs + (["-Xptxas", "-v"] if verbose else []) + ["-c", os.path.join(CSRC, src), "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s" % (src, r.stderr))
    return obj, r.stderr


def build(force=False, verbose=False, trace=False, variant=None):
    """Compile and link the library (variant "trace" or "check" for the tracing / checking build; trace=True is the
    former) if any source is newer than it.  Returns the library path."""
    if trace:
        variant = "trace"
    obj_dir, lib, _ = _VARIANTS[variant]
    if not force and not _stale(lib):
        return lib
    nvcc = _nvcc()
    os.makedirs(obj_dir, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as ex:
        results = list(ex.map(lambda s: _compile(nvcc, s, verbose, variant), _sources()))
    if verbose:
        for _, log in results:
            sys.stderr.write(log)
    objs = [o for o, _ in results]
    r = subprocess.run([nvcc, "-shared", "-o", lib] + objs + ["-Xcompiler", "-fvisibility=hidden"],
                       capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("link failed:\n" + r.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv,
                variant="trace" if "--trace" in sys.argv else ("check" if "--check" in sys.argv else None)))
