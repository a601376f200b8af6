"""Build libsantapp.so (sm_100a) in-tree with nvcc. Cross-compiles without a GPU."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
SOURCES = ["api.cu", "build_teams.cu", "build_parents.cu", "kmeans.cu", "score.cu", "headplan.cu", "plan.cu", "attend.cu", "latent.cu"]
HEADERS = [os.path.join(CSRC, h) for h in ("common.cuh", "pairplan.cuh", "headplan.cuh", "score_tile.cuh", "build_util.cuh", "latent_tc.cuh")] \
    + [os.path.join(ROOT, "include", h) for h in ("santapp.h", "santapp_latent.h")]
OUT = os.path.join(HERE, "libsantapp.so")


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def build(force: bool = False, verbose: bool = False) -> str:
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    if not force and os.path.exists(OUT):
        newest = max(os.path.getmtime(f) for f in srcs + HEADERS + [os.path.abspath(__file__)])
        if os.path.getmtime(OUT) >= newest:
            return OUT
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", OUT] + srcs
    if os.environ.get("SANTAPP_TUNE"):
        cmd.insert(1, "-DSANTAPP_TUNE")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
