"""Compile the CUDA sources into libsparseauto.so for sm_100a (nvcc cross-compiles without a GPU)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsparseauto.so")
LIB_CHECKED = os.path.join(HERE, "libsparseauto_checked.so")
LIB_WAITTEST = os.path.join(HERE, "libsparseauto_waittest.so")
SOURCES = ["sa_api.cu", "sa_build.cu", "sa_ttm3.cu", "sa_ttm4.cu", "sa_ttm4_fis.cu", "sa_sddmm_spmm.cu", "sa_spmm_gemm.cu", "sa_ttmc3.cu", "sa_mttkrp.cu", "sa_dense_tc.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC,-fopenmp,-O3", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _stale(lib=LIB):
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "sparseauto.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False, flags=(), lib=LIB):
    """Compile the sources into ``lib``.  ``flags`` (and SA_NVCC_EXTRA in the environment) add nvcc flags."""
    extra = list(flags) + os.environ.get("SA_NVCC_EXTRA", "").split()
    if not force and not os.environ.get("SA_NVCC_EXTRA") and not _stale(lib):
        return lib
    return _compile(extra, verbose, lib, os.path.splitext(os.path.basename(lib))[0])


def build_checked(force=False):
    """The self-checking build (-DSA_DEBUG_BOUNDS): every index taken from the tensor's arrays is checked on the
    device before it becomes an address.  Loaded instead of the normal library when the environment variable
    SPARSEAUTO_LIB names it."""
    return build(force=force, flags=["-DSA_DEBUG_BOUNDS"], lib=LIB_CHECKED)


def build_waittest(force=False):
    """Test library for the bounded device-side waits of the dense stage: hand-offs give up after 2 ms instead of
    2 s, and a hook (status word 3) makes one arrival stay away so that the time-out path runs."""
    return build(force=force, flags=["-DSA_TEST_HOOKS", "-DSA_TC_WAIT_NS=2000000ull"], lib=LIB_WAITTEST)


PROBE_LIB = os.path.join(HERE, "probe", "libsaprobe.so")


def build_probe(force=False):
    """The bare row-gather kernels bench.py times as the L2-gather ceiling: a measurement aid in a library of
    its own (nothing of the product path links it)."""
    src = os.path.join(HERE, "probe", "sa_gather_probe.cu")
    if not force and os.path.exists(PROBE_LIB) and os.path.getmtime(PROBE_LIB) >= os.path.getmtime(src):
        return PROBE_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = PROBE_LIB + ".tmp%d" % os.getpid()
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
                           "-Xcompiler", "-fPIC", src, "-o", tmp])
    os.replace(tmp, PROBE_LIB)
    return PROBE_LIB


def _compile(extra, verbose, LIB, tag):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    procs = []
    os.makedirs(os.path.join(HERE, "_build", tag), exist_ok=True)
    for src in SOURCES:
        obj = os.path.join(HERE, "_build", tag, src.replace(".cu", ".o"))
        cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write("== %s\n%s\n" % (src, out))
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = LIB + ".tmp%d" % os.getpid()
    subprocess.check_call([nvcc, "-Wno-deprecated-gpu-targets", "-shared", "-o", tmp] + objs + ["-Xcompiler", "-fopenmp", "-lgomp"])
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    if "--checked" in sys.argv:
        print(build_checked(force="--force" in sys.argv))
    elif "--waittest" in sys.argv:
        print(build_waittest(force="--force" in sys.argv))
    elif "--probe" in sys.argv:
        print(build_probe(force="--force" in sys.argv))
    else:
        out = [a.split("=", 1)[1] for a in sys.argv if a.startswith("--out=")]
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, lib=os.path.abspath(out[0]) if out else LIB))
