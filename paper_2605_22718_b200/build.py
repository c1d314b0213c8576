"""In-tree build of the CUDA libraries (sm_100a only).

``build_all()`` compiles
  * ``paper_2605_22718_b200/libworldkv.so``  -- the product: the C-ABI library declared in include/wk.h
  * ``wkinputs/libwkinputs.so``              -- the seeded input generators' device side
  * ``tests/cuda/libwk_wait_probe.so``       -- test-only: the product's bounded mbarrier wait built with a small cap
with nvcc.  nvcc cross-compiles without a GPU, so this also runs on a CPU-only machine.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2605_22718_b200", "csrc")
LIB_WORLDKV = os.path.join(ROOT, "paper_2605_22718_b200", "libworldkv.so")
LIB_INPUTS = os.path.join(ROOT, "wkinputs", "libwkinputs.so")
LIB_WAIT_PROBE = os.path.join(ROOT, "tests", "cuda", "libwk_wait_probe.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA libraries cannot be built")


def _stale(target: str, sources) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def _run(cmd, log_name: str) -> None:
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    log = os.path.join(ROOT, "build", log_name)
    os.makedirs(os.path.dirname(log), exist_ok=True)
    with open(log, "w") as f:
        f.write(" ".join(cmd) + "\n" + res.stdout)
    if res.returncode != 0:
        sys.stderr.write(res.stdout)
        raise RuntimeError("nvcc failed: " + " ".join(cmd))


def build_all(force: bool = False) -> None:
    srcs = sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))
    deps = srcs + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")] + [
        os.path.join(ROOT, "include", "wk.h")]
    if force or _stale(LIB_WORLDKV, deps):
        _run([_nvcc()] + NVCC_FLAGS + ["-I", os.path.join(ROOT, "include"), "-o", LIB_WORLDKV] + srcs, "libworldkv.log")
    gen = os.path.join(ROOT, "wkinputs", "gen.cu")
    if force or _stale(LIB_INPUTS, [gen]):
        _run([_nvcc()] + NVCC_FLAGS + ["-o", LIB_INPUTS, gen], "libwkinputs.log")
    probe = os.path.join(ROOT, "tests", "cuda", "wait_probe.cu")
    if os.path.exists(probe) and (force or _stale(LIB_WAIT_PROBE, [probe, os.path.join(CSRC, "ptx_sm100.cuh")])):
        _run([_nvcc()] + NVCC_FLAGS + ["-DWK_WAIT_CAP=4096u", "-o", LIB_WAIT_PROBE, probe], "libwk_wait_probe.log")


if __name__ == "__main__":
    build_all(force="--force" in sys.argv)
    print("built", LIB_WORLDKV, "and", LIB_INPUTS)
