"""Build step: compile the CUDA sources into the C-ABI shared library, in-tree.

``build()`` runs nvcc for sm_100a on every ``csrc/*.cu`` (in parallel), links
``libprunedctc.so`` next to this file and returns its path.  Objects are cached
under ``build/`` and rebuilt only when a source or header is newer.
``build_variant(tag)`` builds a test variant of the same sources (see VARIANTS).
"""

from __future__ import annotations

import concurrent.futures
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(ROOT, "build", "obj")
LIB_PATH = os.path.join(HERE, "libprunedctc.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC",
    "--expt-relaxed-constexpr",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in paths)


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def headers():
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    hs.append(os.path.join(ROOT, "include", "prunedctc.h"))
    return hs


# Variants of the library for tests: same sources, extra compile-time definitions, a file of their own.
#   shortwait  every bounded device wait gives up after a few thousand cycles, so that an ordinary
#              call exercises the give-up path (status word, drain, clean return)
#   bounds     every index that a kernel gathers or scatters through (selected classes, relabelled
#              targets, row tables) is range-checked first; a bad one is recorded in the status word
#              and the access is skipped
#   probe_*    measurement probes for `bench.py --lib-variant`: one part of the tensor-core kernel is
#              knocked out (results are wrong on purpose) to show what a launch is bound by
VARIANTS = {
    "shortwait": ("-DPCTC_WAIT_LIMIT_CYCLES=3000LL", "-DPCTC_WAIT_POLL_MASK=0u"),
    "bounds": ("-DPCTC_DEBUG_BOUNDS=1",),
    "probe_noepilogue": ("-DPCTC_PROBE=7",),      # no tensor-memory loads, no epilogue arithmetic, no chunk store
    "probe_nostore": ("-DPCTC_PROBE=4",),         # the dlogits chunk is computed but not written
    "probe_skipa": ("-DPCTC_PROBE=8",),           # the normaliser kernel reloads only its B operand per tile
    "tune_walk_a": ("-DPCTC_TUNE_WALK_HINT=1",),  # L2 evict-last on the A rows of the column-walking kernels
    "tune_walk_mb8": ("-DPCTC_TUNE_WALK_MB=8",),  # bands of the column-walking kernels whose A rows fill 8 / 16 / 66 MB
    "tune_walk_mb16": ("-DPCTC_TUNE_WALK_MB=16",),
    "tune_walk_mb66": ("-DPCTC_TUNE_WALK_MB=66",),
    "tune_lse_s22": ("-DPCTC_TUNE_LSE_SPLITS=22",),   # forced column splits of the LSE kernel (c4: 594 = 22 x 27 tiles)
    "tune_lse_s27": ("-DPCTC_TUNE_LSE_SPLITS=27",),
    "tune_lse_s9": ("-DPCTC_TUNE_LSE_SPLITS=9",),
}
TEST_VARIANTS = ("shortwait", "bounds")           # the ones the test-suite loads


def variant_path(tag: str) -> str:
    return os.path.join(HERE, f"libprunedctc_{tag}.so")


def build_variant(tag: str, verbose: bool = False) -> str:
    return build(verbose=verbose, extra_flags=VARIANTS[tag], tag=tag)


def build(verbose: bool = False, extra_flags=(), tag: str = "") -> str:
    obj_dir = OBJ_DIR + ("_" + tag if tag else "")
    lib_path = variant_path(tag) if tag else LIB_PATH
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    srcs = sources()
    hdr_time = _newest(headers() + [os.path.abspath(__file__)])
    jobs = []
    objs = []
    for src in srcs:
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if os.path.exists(obj) and os.path.getmtime(obj) >= max(os.path.getmtime(src), hdr_time):
            continue
        cmd = [nvcc, *NVCC_FLAGS, *extra_flags, "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
        return r.stderr

    if jobs:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            for out in ex.map(run, jobs):
                if verbose and out:
                    sys.stderr.write(out)
    if jobs or not os.path.exists(lib_path) or os.path.getmtime(lib_path) < _newest(objs):
        run([nvcc, "-shared", "-o", lib_path, *objs])   # static cudart (nvcc default)
    return lib_path


if __name__ == "__main__":
    print(build(verbose="-v" in sys.argv))
