"""Compile the CUDA sources into paper_2206_08869_b200/libiodf_b200.so (sm_100a only)."""
import glob
import hashlib
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libiodf_b200.so")
STAMP = LIB + ".sha256"      # hash of the sources the library was built from
NVCC_FLAGS = ["-shared", "-Xcompiler", "-fPIC", "-O3", "-std=c++17", "-gencode",
              "arch=compute_100a,code=sm_100a", "-lineinfo"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def source_hash():
    """SHA-256 over every file the library is compiled from (names and contents) and the flags."""
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    deps = sorted(glob.glob(os.path.join(CSRC, "*"))) + [os.path.join(HERE, "..", "include", "iodf.h")]
    for p in deps:
        if os.path.isdir(p):         # csrc/microbench: stand-alone programs, not part of the library
            continue
        h.update(os.path.basename(p).encode())
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _stale():
    """A library is current only if the hash recorded beside it equals the hash of the sources, so
    a binary built from other sources can never stand in for them, whatever the file times say."""
    if not os.path.exists(LIB) or not os.path.exists(STAMP):
        return True
    with open(STAMP) as f:
        return f.read().strip() != source_hash()


def build(force=False, verbose=False):
    """Build the shared library if it is missing or was built from other sources; return its path."""
    if force or _stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = LIB + ".tmp.%d" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
        digest = source_hash()
        subprocess.check_call(cmd)
        os.replace(tmp, LIB)
        with open(STAMP, "w") as f:
            f.write(digest + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
