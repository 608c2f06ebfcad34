"""Builds ``libsparse_engine.so`` (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libsparse_engine.so")
SOURCES = ["se_api.cu", "se_meta.cu", "se_select.cu", "se_decode.cu", "se_h2o.cu", "se_probe.cu"]
HEADERS = ["se_device.cuh", "se_internal.h", "se_topk.cuh", os.path.join("..", "..", "include", "sparse_engine.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in paths)


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    deps = [os.path.join(CSRC, s) for s in SOURCES] + [os.path.join(CSRC, h) for h in HEADERS]
    return os.path.getmtime(LIB) < _newest(deps)


def _compile(src: str, verbose: bool, extra=(), suffix: str = "") -> str:
    obj = os.path.join(OBJ, src.replace(".cu", suffix + ".o"))
    cmd = [_nvcc()] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-c", os.path.join(CSRC, src), "-o", obj]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, res.stdout, res.stderr))
    return res.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        logs = list(ex.map(lambda s: _compile(s, verbose), SOURCES))
    if verbose:
        sys.stderr.write("\n".join(logs))
    objs = [os.path.join(OBJ, s.replace(".cu", ".o")) for s in SOURCES]
    tmp = LIB + ".tmp%d" % os.getpid()
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, LIB)
    return LIB


# A second build of the same sources with -DSE_TEST_SHORT_TX: the scoring kernel's waits run out (see
# se_select.cu).  Only tests/test_gpu_timeout.py loads it.
LIB_SHORT_TX = os.path.join(HERE, "libsparse_engine_shorttx.so")


def build_short_tx(force: bool = False) -> str:
    deps = [os.path.join(CSRC, s) for s in SOURCES] + [os.path.join(CSRC, h) for h in HEADERS]
    if not force and os.path.exists(LIB_SHORT_TX) and os.path.getmtime(LIB_SHORT_TX) >= _newest(deps):
        return LIB_SHORT_TX
    os.makedirs(OBJ, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        list(ex.map(lambda s: _compile(s, False, ["-DSE_TEST_SHORT_TX"], "_shorttx"), SOURCES))
    objs = [os.path.join(OBJ, s.replace(".cu", "_shorttx.o")) for s in SOURCES]
    tmp = LIB_SHORT_TX + ".tmp%d" % os.getpid()
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, LIB_SHORT_TX)
    return LIB_SHORT_TX


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
