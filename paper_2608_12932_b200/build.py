"""Builds libw4a8.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2608_12932_b200.build [--force]

Each .cu under csrc/ is compiled to an object, then linked into one shared library next
to this file.  The ptxas resource report of every kernel is kept in build/ptxas.txt and
checked: the tcgen05 kernel redistributes registers between warpgroups with setmaxnreg,
which only works if it was allotted the full 128 registers per thread at launch.
"""
import os
import re
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
BUILD = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libw4a8.so")

NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xptxas", "-v", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _deps_mtime():
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "w4a8.h"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def check_ptxas(report):
    """Raise if a GEMM kernel spills or the tcgen05 kernel did not get 128 registers."""
    problems = []
    for m in re.finditer(r"Compiling entry function '(\S+)' for 'sm_100a'.*?\n.*?(\d+) bytes spill stores.*?\n"
                         r".*?Used (\d+) registers", report, re.S):
        name, spill, regs = m.group(1), int(m.group(2)), int(m.group(3))
        limit = 128                               # a few stray registers are tolerable, an accumulator array is not
        m2 = re.search(r"gemm_tcgen05_kernelILi\d+ELb(\d)E", name) or re.search(r"gemm_strip_kernelILi\d+ELi\d+ELb(\d)E", name)
        if m2 and m2.group(1) == "1":
            limit = 1024                          # the debug instantiations (partials dump) may spill
        if spill > limit and "gemm_" in name:
            problems.append(f"{name}: {spill} bytes of spill stores")
        if "gemm_tcgen05_kernel" in name and regs != 128:
            problems.append(f"{name}: {regs} registers at launch, setmaxnreg budget assumes 128")
    if problems:
        raise RuntimeError("ptxas check failed:\n  " + "\n  ".join(problems))


def build(force=False, verbose=False):
    os.makedirs(BUILD, exist_ok=True)
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _deps_mtime():
        return LIB
    objs, report = [], []
    for src in _sources():
        obj = os.path.join(BUILD, src[:-3] + ".o")
        cmd = [NVCC] + FLAGS + ["-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        report.append(f"==== {src}\n{r.stderr}")
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError(f"nvcc failed on {src}")
        objs.append(obj)
    text = "\n".join(report)
    with open(os.path.join(BUILD, "ptxas.txt"), "w") as f:
        f.write(text)
    if verbose:
        print(text)
    check_ptxas(text)
    r = subprocess.run([NVCC, "-shared", "-o", LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"],
                       capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link failed")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
