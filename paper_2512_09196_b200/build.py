"""Builds libtf.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import fcntl
import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
INCLUDE = HERE.parent / "include"
LIB = HERE / "libtf.so"
SOURCES = ["tf_api.cu", "tf_rowreg.cu", "tf_tma.cu", "tf_stream.cu", "tf_pipe.cu", "tf_ring.cu", "tf_twopass.cu", "tf_split.cu", "tf_srows.cu", "tf_elementwise.cu", "tf_vecmat.cu", "tf_addnorm.cu", "tf_softmaxlen.cu", "tf_softmax_variants.cu", "tf_norm_bwd.cu", "tf_pipe_softmax.cu", "tf_pipe_layernorm.cu", "tf_pipe_rmsnorm.cu"]
NVCC_FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (cand == "nvcc" or Path(cand).exists()):
            return cand
    raise RuntimeError("nvcc not found")


def _digest(paths, extra=()) -> str:
    """Content hash of the inputs of a build step (file times do not survive a copy of the tree)."""
    h = hashlib.sha256()
    for x in extra:
        h.update(str(x).encode())
    for p in sorted(map(str, paths)):
        h.update(p.rsplit("/", 1)[-1].encode())
        h.update(Path(p).read_bytes())
    return h.hexdigest()


def _stale(target: Path, stamp: Path, digest: str) -> bool:
    return not target.exists() or not stamp.exists() or stamp.read_text().strip() != digest


class _Lock:
    """One builder at a time (several ranks may import the package at once)."""

    def __init__(self, path: Path):
        self.path = path

    def __enter__(self):
        self.f = open(self.path, "w")
        fcntl.flock(self.f, fcntl.LOCK_EX)

    def __exit__(self, *exc):
        fcntl.flock(self.f, fcntl.LOCK_UN)
        self.f.close()


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every .cu file to an object (in parallel) and link libtf.so.  A step is redone when the content of
    its inputs (source, headers, flags) changed."""
    headers = list(CSRC.glob("*.h")) + list(CSRC.glob("*.cuh")) + list(INCLUDE.glob("*.h"))
    objdir = HERE / "build"
    objdir.mkdir(exist_ok=True)
    with _Lock(objdir / ".lock"):
        nvcc = _nvcc()
        jobs = []
        for src in SOURCES:
            obj = objdir / (src[:-3] + ".o")
            stamp = objdir / (src[:-3] + ".stamp")
            digest = _digest([CSRC / src, *headers], NVCC_FLAGS)
            if force or _stale(obj, stamp, digest):
                jobs.append((src, obj, stamp, digest))

        def compile_one(job):
            src, obj, stamp, digest = job
            cmd = [nvcc, *NVCC_FLAGS, "-I", str(INCLUDE), "-c", str(CSRC / src), "-o", str(obj)]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            r = subprocess.run(cmd, capture_output=True, text=True)
            if r.returncode:
                raise RuntimeError(f"nvcc failed on {src}:\n{r.stdout}\n{r.stderr}")
            stamp.write_text(digest)
            return r.stderr

        with ThreadPoolExecutor(max_workers=8) as ex:
            logs = list(ex.map(compile_one, jobs))
        if verbose:
            sys.stderr.write("\n".join(logs))
        objs = [objdir / (s[:-3] + ".o") for s in SOURCES]
        link_digest = _digest(objs)
        link_stamp = objdir / "libtf.stamp"
        if force or jobs or _stale(LIB, link_stamp, link_digest):
            tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
            r = subprocess.run([nvcc, "-shared", "-o", str(tmp), *map(str, objs)], capture_output=True, text=True)
            if r.returncode:
                raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
            os.replace(tmp, LIB)
            link_stamp.write_text(link_digest)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
