"""Build libgift.so (sm_100a) in-tree with nvcc, and the host-only check library with g++."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libgift.so")
HOSTCHECK = os.path.join(HERE, "libgift_hostcheck.so")
PROBE = os.path.join(HERE, "libgift_probe.so")
SOURCES = ["gift_lib.cu", "gift_rules.cu", "gift_hostio.cu", "gift_tokens.cu", "gift_order.cu", "gift_index.cu",
           "gift_chain.cu"]
HEADERS = ["gf128.cuh", "aes_tt.cuh", "gift_core.cuh", "gift_internal.cuh", "gift_rules.cuh", "gift_csr.cuh", "gift_seg.cuh",
           os.path.join("..", "..", "include", "gift.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def _deps(extra):
    return [os.path.join(CSRC, f) for f in list(extra) + HEADERS]


def build_lib(force=False, verbose=False):
    """Compile the CUDA library for sm_100a; returns the path of libgift.so."""
    if not force and not _stale(LIB, _deps(SOURCES)):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + \
          [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


def build_probe(force=False):
    """Compile the instruction-rate probes (diagnostics, not part of libgift.so) for sm_100a."""
    if not force and not _stale(PROBE, _deps(["pipe_probe.cu"])):
        return PROBE
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = PROBE + ".tmp.%d" % os.getpid()
    subprocess.run([nvcc] + NVCC_FLAGS + ["-o", tmp, os.path.join(CSRC, "pipe_probe.cu")], check=True)
    os.replace(tmp, PROBE)
    return PROBE


def build_hostcheck(force=False):
    """Compile the device arithmetic for the host (no GPU needed); returns the library path."""
    src = ["hostcheck.cpp"]
    if not force and not _stale(HOSTCHECK, _deps(src)):
        return HOSTCHECK
    tmp = HOSTCHECK + ".tmp.%d" % os.getpid()
    cmd = ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-Wall", "-Wno-unknown-pragmas", "-o", tmp,
           os.path.join(CSRC, "hostcheck.cpp")]
    subprocess.run(cmd, check=True)
    os.replace(tmp, HOSTCHECK)
    return HOSTCHECK


if __name__ == "__main__":
    print(build_lib(force=True, verbose=True))
    print(build_probe(force=True))
    print(build_hostcheck(force=True))
