"""Build ``libsfda.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

A build is current when the hash of its sources, kept in a small file beside the library, equals the hash of the
sources in the tree: file times say nothing once a source file has been put back to an earlier state."""
import glob
import hashlib
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsfda.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=true", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
    "--expt-relaxed-constexpr",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sorted(sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h"))
                  + glob.glob(os.path.join(HERE, "..", "include", "*.h")))


def source_hash(extra_flags=()) -> str:
    """SHA-256 over the compiler flags and the names and contents of every source and header of the library."""
    h = hashlib.sha256(" ".join(FLAGS + list(extra_flags)).encode())
    for path in _deps():
        h.update(os.path.basename(path).encode() + b"\0")
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _current(lib: str, extra_flags=()) -> bool:
    try:
        with open(lib + ".srchash") as f:
            return os.path.exists(lib) and f.read().strip() == source_hash(extra_flags)
    except OSError:
        return False


def is_stale() -> bool:
    """True when ``libsfda.so`` is missing or was not built from the sources now in the tree."""
    return not _current(LIB)


def _stale() -> bool:
    return is_stale()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every ``csrc/*.cu`` into ``libsfda.so`` when missing or stale."""
    if not force and not _stale():
        return LIB
    objdir = os.path.join(HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    objs = []
    procs = []
    for src in sources():
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
        procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for cmd, p in procs:
        out, _ = p.communicate()
        if verbose and out:
            print(out)
        if p.returncode != 0:
            raise RuntimeError("nvcc failed: %s\n%s" % (" ".join(cmd), out))
    tmp = LIB + ".tmp.%d" % os.getpid()
    link = [NVCC, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs
    subprocess.run(link, check=True)
    os.replace(tmp, LIB)
    with open(LIB + ".srchash", "w") as f:
        f.write(source_hash() + "\n")
    return LIB


def build_variant(name: str, extra_flags):
    """Compile every source with `extra_flags` added into ``build/<name>/`` and link ``build/libsfda_<name>.so``
    (used by the tests for the development build whose roles pause at random, ``-DSFDA_WS_CHAOS``)."""
    objdir = os.path.join(HERE, "build", name)
    lib = os.path.join(HERE, "build", "libsfda_%s.so" % name)
    if _current(lib, extra_flags):
        return lib
    os.makedirs(objdir, exist_ok=True)
    procs, objs = [], []
    for src in sources():
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        cmd = [NVCC] + FLAGS + list(extra_flags) + ["-c", src, "-o", obj]
        procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for cmd, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0:
            raise RuntimeError("nvcc failed: %s\n%s" % (" ".join(cmd), out))
    tmp = lib + ".tmp.%d" % os.getpid()
    subprocess.run([NVCC, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs, check=True)
    os.replace(tmp, lib)
    with open(lib + ".srchash", "w") as f:
        f.write(source_hash(extra_flags) + "\n")
    return lib


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
