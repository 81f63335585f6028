"""Builds the C-ABI library `libgdnprep.so` in-tree with nvcc for sm_100a.

`python -m paper_2606_06034_b200.build` (or `build()`), no GPU needed: nvcc
cross-compiles. The library links the CUDA runtime statically and has no other
dependency, so loading it needs neither torch nor a driver.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libgdnprep.so")
SOURCES = ["gdn_api.cu", "chunk_simt.cu", "chunk_tc_bf16.cu", "chunk_tc_int8.cu", "chunk_tc_int16.cu", "chunk_state.cu"]
HEADERS = ["common.cuh", "sm100_ptx.cuh", os.path.join("..", "..", "include", "gdnprep.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def resource_log(src: str) -> str:
    """Path of the ptxas resource report (registers, spills per kernel) written when `src` was last compiled."""
    return os.path.join(HERE, "build", src.replace(".cu", ".ptxas.log"))


def kernel_resources(src: str) -> dict:
    """{mangled kernel name: {"registers": r, "spill_stores": s, "spill_loads": l}} from the last build of `src`."""
    import re
    out = {}
    name = None
    with open(resource_log(src)) as f:
        for line in f:
            m = re.search(r"Compiling entry function '([^']+)'", line)
            if m:
                name = m.group(1)
                out[name] = {}
                continue
            if name is None:
                continue
            m = re.search(r"(\d+) bytes spill stores, (\d+) bytes spill loads", line)
            if m:
                out[name]["spill_stores"] = int(m.group(1))
                out[name]["spill_loads"] = int(m.group(2))
            m = re.search(r"Used (\d+) registers", line)
            if m:
                out[name]["registers"] = int(m.group(1))
    return out


def needs_build() -> bool:
    if not os.path.exists(LIB) or not all(os.path.exists(resource_log(s)) for s in SOURCES):
        return True
    deps = [os.path.join(CSRC, s) for s in SOURCES] + [os.path.join(CSRC, h) for h in HEADERS]
    return _newest(deps) > os.path.getmtime(LIB)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    procs = []
    os.makedirs(os.path.join(HERE, "build"), exist_ok=True)
    for src in SOURCES:
        obj = os.path.join(HERE, "build", src.replace(".cu", ".o"))
        # ptxas reports registers and spills of every kernel: kept next to the objects (`resource_log`), because the
        # tensor-core kernels run at the 128-register limit and a few bytes of spill cost them 5-10 %
        cmd = [nvcc, "-Xptxas", "-v", *NVCC_FLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode != 0:
            sys.stderr.write(out)
        if pr.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        with open(resource_log(src), "w") as f:
            f.write(out)
    cmd = [nvcc, "-shared", "-o", LIB, *objs, "-cudart", "static", "-Xcompiler", "-fPIC"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
