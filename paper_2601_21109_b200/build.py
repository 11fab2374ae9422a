"""Builds libcwl.so (CUDA, sm_100a only) in-tree with nvcc.  No GPU is needed to compile."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcwl.so")
LIB_HOOKS = os.path.join(HERE, "libcwl_hooks.so")
SOURCES = ["api.cu", "score.cu", "partition.cu", "align.cu", "stream.cu", "ladder.cu", "apply.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v", "--expt-relaxed-constexpr"]


def _newest_source() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "cwl.h"), os.path.join(ROOT, "include", "cwl_test_hooks.h"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    """Builds libcwl.so and, from the same sources plus -DCWL_TEST_HOOKS for apply.cu, the test build
    libcwl_hooks.so (it adds cwl_debug_set, which shortens the device-side wait limit and withholds H')."""
    if not force and os.path.exists(LIB) and os.path.exists(LIB_HOOKS) and \
            min(os.path.getmtime(LIB), os.path.getmtime(LIB_HOOKS)) >= _newest_source():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = os.environ.get("CWL_NVCC_EXTRA", "").split()   # e.g. -DCWL_STAGES=5 for tuning experiments
    os.makedirs(os.path.join(HERE, "_build"), exist_ok=True)
    jobs = [(src, src.replace(".cu", ".o"), []) for src in SOURCES] + \
        [("apply.cu", "apply_hooks.o", ["-DCWL_TEST_HOOKS"]), ("probe.cu", "probe_hooks.o", ["-DCWL_TEST_HOOKS"])]
    procs = []
    for src, obj, defs in jobs:
        cmd = [nvcc, *NVCC_FLAGS, *extra, *defs, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c",
               os.path.join(CSRC, src), "-o", os.path.join(HERE, "_build", obj)]
        procs.append((obj, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    log = []
    for obj, pr in procs:
        out, _ = pr.communicate()
        log.append(f"== {obj}\n{out}")
        if pr.returncode != 0:
            sys.stderr.write("\n".join(log))
            raise RuntimeError(f"nvcc failed on {obj}")
    plain = [os.path.join(HERE, "_build", s.replace(".cu", ".o")) for s in SOURCES]
    hooks = [o if not o.endswith("/apply.o") else o.replace("apply.o", "apply_hooks.o") for o in plain] + \
        [os.path.join(HERE, "_build", "probe_hooks.o")]
    for lib, objs in ((LIB, plain), (LIB_HOOKS, hooks)):
        tmp = lib + f".tmp{os.getpid()}"
        subprocess.run([nvcc, "-shared", "-o", tmp, *objs, "-lcudart_static", "-lpthread", "-ldl", "-lrt"], check=True)
        os.replace(tmp, lib)
    with open(os.path.join(HERE, "_build", "ptxas.log"), "w") as fh:
        fh.write("\n".join(log))
    if verbose:
        print("\n".join(log))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
