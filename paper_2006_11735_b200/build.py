"""Builds ``libiconv_b200.so`` (the C-ABI library) in-tree with nvcc for sm_100a."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB = os.path.join(_HERE, "libiconv_b200.so")
OBJ_DIR = os.path.join(_HERE, "_build")
# the benchmark's measurement aid (tensor-pipe issue rate): a library of its own, not part of the C ABI
PROBE_SRC = os.path.join(_HERE, "bench_probe", "probe_mma.cu")
PROBE_LIB = os.path.join(_HERE, "libiconv_probe.so")
SOURCES = ["iconv_api.cu", "plan.cu", "kernels_direct.cu", "kernel_thin.cu", "kernel_umma.cu", "kernel_stem.cu",
           "kernel_calib.cu", "kernel_chain.cu", "planner.cpp"] + ["umma_inst_conv%d.cu" % e for e in range(8)] + \
          ["umma_inst_window%d.cu" % e for e in (2, 3, 4, 5, 8)]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-diag-suppress", "128", "-Xcompiler", "-fPIC",
         "-Xcompiler", "-fvisibility=hidden", "-I", INCLUDE, "-I", CSRC]


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))] + [os.path.join(INCLUDE, "iconv.h")]


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(f) > t for f in deps)


def _compile(src: str, obj: str, verbose: bool):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + FLAGS + ["-c", src, "-o", obj]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    subprocess.run(cmd, check=True)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source for sm_100a (one object per source, in parallel; objects are
    reused while neither the source nor a header changed) and link them into one shared library
    next to this file."""
    os.makedirs(OBJ_DIR, exist_ok=True)
    headers = _headers()
    jobs = []
    for s in SOURCES:
        src, obj = os.path.join(CSRC, s), os.path.join(OBJ_DIR, s + ".o")
        if force or _stale(obj, [src] + headers):
            jobs.append((src, obj))
    jobs.sort(key=lambda j: -os.path.getsize(j[0]) if "umma_inst" not in j[0] else -10 ** 9)   # the kernel instances first: they take longest
    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as ex:
        for f in [ex.submit(_compile, src, obj, verbose) for src, obj in jobs]:
            f.result()
    objs = [os.path.join(OBJ_DIR, s + ".o") for s in SOURCES]
    if jobs or _stale(LIB, objs):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = LIB + ".%d.tmp" % os.getpid()
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs, check=True)
        os.replace(tmp, LIB)
    if force or _stale(PROBE_LIB, [PROBE_SRC]):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = PROBE_LIB + ".%d.tmp" % os.getpid()
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
                        "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-o", tmp, PROBE_SRC], check=True)
        os.replace(tmp, PROBE_LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="-f" in sys.argv, verbose="-v" in sys.argv))
