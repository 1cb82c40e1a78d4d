"""Builds the CUDA shared library in-tree with nvcc for sm_100a.

The streaming kernels exist once per (gradient dtype, fused or not, statistics mode) and per
worker count -- several hundred instantiations.  They are spread over translation units
(stream_inst.cu compiled once per combination) that build in parallel, then linked with
abs_api.cu and the host-only sources into libabs_normtest.so.
"""
import concurrent.futures
import glob
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
_OBJ = os.path.join(_PKG, "_build")
LIB_PATH = os.path.join(_PKG, "libabs_normtest.so")
INCLUDE_DIR = os.path.join(os.path.dirname(_PKG), "include")

# -lineinfo keeps source lines for the profiler; with several hundred kernels the line tables
# triple the image, so the device code is stored compressed (52 MB -> 13 MB).
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xfatbin=-compress-all", "-Xcompiler", "-fPIC"]

# (gradient type, fused with AdamW, statistics mode: 0 sums, 1 sums + Q, 2 coordinate-wise)
STREAM_COMBINATIONS = [("BF16", 1, 0), ("F32", 1, 0), ("BF16", 0, 1), ("F32", 0, 1),
                       ("BF16", 0, 0), ("F32", 0, 0), ("BF16", 1, 2), ("F32", 1, 2),
                       ("BF16", 0, 2), ("F32", 0, 2)]


def sources():
    return sorted(glob.glob(os.path.join(_CSRC, "*.cu")))


def _deps():
    return (sources() + glob.glob(os.path.join(_CSRC, "*.cuh"))
            + glob.glob(os.path.join(INCLUDE_DIR, "*.h")) + [os.path.abspath(__file__)])


def is_stale():
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(f) > t for f in _deps())


def _jobs():
    """(object path, source, extra defines) for every translation unit."""
    jobs = []
    for src in sources():
        name = os.path.splitext(os.path.basename(src))[0]
        if name == "stream_inst":
            for gt, adam, stat in STREAM_COMBINATIONS:
                jobs.append((os.path.join(_OBJ, "stream_%s_%d_%d.o" % (gt.lower(), adam, stat)), src,
                             ["-DABS_INST_GT=%s" % gt, "-DABS_INST_ADAM=%d" % adam,
                              "-DABS_INST_STAT=%d" % stat]))
        else:
            jobs.append((os.path.join(_OBJ, name + ".o"), src, []))
    return jobs


def _compile(job, nvcc, verbose):
    obj, src, defines = job
    extra = os.environ.get("ABS_NVCC_EXTRA", "").split()  # e.g. -D switches for A/B builds
    cmd = ([nvcc] + NVCC_FLAGS + defines + extra + (["-Xptxas", "-v"] if verbose else [])
           + ["-c", "-o", obj, src])
    out = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if out.returncode != 0:
        raise RuntimeError("nvcc failed on %s %s:\n%s" % (os.path.basename(src), " ".join(defines),
                                                          out.stdout[-4000:]))
    return out.stdout


def build(force=False, verbose=False, workers=None):
    """nvcc -> libabs_normtest.so (cross-compiles without a GPU).  Returns the path."""
    if not force and not is_stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(_OBJ, exist_ok=True)
    jobs = _jobs()
    workers = workers or min(len(jobs), max(1, (os.cpu_count() or 2)))
    with concurrent.futures.ThreadPoolExecutor(max_workers=workers) as pool:
        logs = list(pool.map(lambda j: _compile(j, nvcc, verbose), jobs))
    if verbose:
        print("".join(logs))
    tmp = LIB_PATH + ".tmp.%d" % os.getpid()
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp]
                          + [j[0] for j in jobs])
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
