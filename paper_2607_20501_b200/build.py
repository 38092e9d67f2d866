"""Builds libmk.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2607_20501_b200.build [--force] [--verbose]

Objects are rebuilt when their source or any header under csrc/ or include/ is
newer.  nvcc cross-compiles without a GPU.

The build reads ptxas' resource report and refuses a library in which one of the
hot tensor-core kernels keeps a large stack frame: their epilogues hold 32
accumulator values per thread in registers, and a single run-time index into that
array (a partially unrolled loop is enough) moves it to local memory and more than
doubles the epilogue's time without changing any result.
"""
from __future__ import annotations

import concurrent.futures as cf
import glob
import os
import re
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libmk.so")

NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr",
    "-I", INCLUDE, "-I", CSRC,
]


# (source file, pattern on the mangled kernel name, largest stack frame in bytes).  The default GEMM instantiations
# are <CG, SWIGLU, NORM=0, RING, PRE=0>; the row-norm and prefix variants spill at their register cap by design.
STACK_LIMITS = [
    ("gemm_tc.cu", r"gemm_tc_kernelILi[12]ELb[01]ELb0ELb[01]ELb0EE", 64),
    ("conv3x3_tc2.cu", r"conv3x3_tc2_kernel", 64),
    ("attention_tc2.cu", r"attention_tc2_kernel", 64),
    ("groupnorm_cluster.cu", r"groupnorm_cluster_kernel", 64),
]


def stack_frames(report):
    """{mangled kernel name: stack frame bytes} from the text ptxas -v prints."""
    out, name = {}, None
    for line in report.splitlines():
        m = re.search(r"Compiling entry function '([^']+)'", line)
        if m:
            name = m.group(1)
            continue
        m = re.search(r"(\d+) bytes stack frame", line)
        if m and name:
            out[name] = int(m.group(1))
            name = None
    return out


def check_stack(src, report):
    bad = []
    for fname, pat, limit in STACK_LIMITS:
        if os.path.basename(src) != fname:
            continue
        for k, b in stack_frames(report).items():
            if re.search(pat, k) and b > limit:
                bad.append(f"{fname}: {k} keeps a {b}-byte stack frame (limit {limit})")
    return bad


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cpp")))


def _headers_mtime():
    hs = glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(INCLUDE, "*.h"))
    return max(os.path.getmtime(h) for h in hs)


def _compile(src, obj, verbose):
    cmd = [NVCC, *FLAGS, *os.environ.get("MK_NVCC_FLAGS", "").split(), "-x", "cu", "-c", src, "-o", obj]
    if src.endswith(".cu"):
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    return src, r.returncode, r.stdout + r.stderr


def build(force=False, verbose=False):
    os.makedirs(OBJ, exist_ok=True)
    hm = _headers_mtime()
    jobs, objs = [], []
    for src in _sources():
        obj = os.path.join(OBJ, os.path.basename(src) + ".o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hm):
            jobs.append((src, obj))
    with cf.ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as ex:
        for src, rc, out in ex.map(lambda j: _compile(j[0], j[1], verbose), jobs):
            if verbose or rc != 0:
                sys.stderr.write(out)
            if rc != 0:
                raise RuntimeError(f"nvcc failed on {src}")
            bad = check_stack(src, out)
            if bad:
                os.remove(os.path.join(OBJ, os.path.basename(src) + ".o"))
                raise RuntimeError("accumulators left the register file:\n  " + "\n  ".join(bad))
    if jobs or not os.path.exists(LIB):
        cmd = [NVCC, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
               "-Xcompiler", "-fPIC"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
