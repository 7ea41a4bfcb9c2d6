"""Builds the CUDA library in-tree: ``python -m paper_2606_10415_b200.build``.

One ``nvcc`` invocation per source file (sm_100a only), then a shared link into
``paper_2606_10415_b200/liblt_attn.so``.  Objects are rebuilt when their source or
any header is newer.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
OBJ = PKG / "build"
LIB = PKG / "liblt_attn.so"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr", "-Xptxas", "-v",
]


def _extra_flags() -> list[str]:
    """Extra nvcc flags from LT_NVCC_FLAGS (development builds, e.g. -DLT_BWD_TRACE)."""
    return os.environ.get("LT_NVCC_FLAGS", "").split()


def _nvcc() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if Path(cand).exists() else "nvcc"


def build(force: bool = False, verbose: bool = False) -> Path:
    sources = sorted(CSRC.glob("*.cu"))
    headers = sorted(CSRC.glob("*.cuh")) + sorted(CSRC.glob("*.h")) + sorted((PKG.parent / "include").glob("*.h"))
    newest_header = max(h.stat().st_mtime for h in headers)
    OBJ.mkdir(exist_ok=True)
    jobs = []
    for src in sources:
        obj = OBJ / (src.stem + ".o")
        stale = force or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, newest_header)
        if stale:
            jobs.append((src, obj))

    def compile_one(job):
        src, obj = job
        cmd = [_nvcc(), *NVCC_FLAGS, *_extra_flags(), "-c", str(src), "-o", str(obj)]
        res = subprocess.run(cmd, capture_output=True, text=True)
        (OBJ / (src.stem + ".ptxas.log")).write_text(res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src.name}:\n{res.stdout}\n{res.stderr}")
        if verbose:
            print(res.stderr)

    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as pool:
        list(pool.map(compile_one, jobs))
    objs = [OBJ / (s.stem + ".o") for s in sources]
    if jobs or not LIB.exists() or LIB.stat().st_mtime < max(o.stat().st_mtime for o in objs):
        tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp), *map(str, objs)]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"link failed:\n{res.stdout}\n{res.stderr}")
        os.replace(tmp, LIB)
    return LIB


# Variant builds of the backward alone (libraries of their own that the binding never loads; whoever needs one loads
# it by path).
#  - give-up: the tensor-core issuer drops one hand-off and every device-side wait gives up after about 10 ms instead
#    of a second: the main kernel then has to leave through its give-up path (abort flag, every role out of its
#    loops, tensor memory released), which tests/test_gpu_giveup.py checks.
#  - timeline: CTA 0 stamps clock64 at every hand-off of its first 256 tile pairs; paper_2606_10415_b200/timeline.py
#    prints the table (a development aid behind the bottleneck analysis of the main kernel).
GIVEUP_LIB = PKG / "liblt_attn_giveup.so"
GIVEUP_FLAGS = ["-DLT_BWD_GIVEUP_TEST=1", "-DLT_WAIT_LIMIT_CYCLES=20000000LL"]
TIMELINE_LIB = PKG / "liblt_attn_timeline.so"
TIMELINE_FLAGS = ["-DLT_BWD_TIMELINE=0"]
VARIANT_SOURCES = ["lt_attn_bwd.cu", "lt_host.cu"]
MICROBENCH = OBJ / "sm_limits"


def _build_variant(lib: Path, flags: list[str], tag: str, force: bool) -> Path:
    obj_dir = PKG / f"build_{tag}"
    obj_dir.mkdir(exist_ok=True)
    headers = sorted(CSRC.glob("*.cuh")) + sorted(CSRC.glob("*.h")) + sorted((PKG.parent / "include").glob("*.h"))
    newest = max(h.stat().st_mtime for h in headers)
    objs = []
    for name in VARIANT_SOURCES:
        src, obj = CSRC / name, obj_dir / (Path(name).stem + ".o")
        objs.append(obj)
        if force or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, newest):
            res = subprocess.run([_nvcc(), *NVCC_FLAGS, *flags, "-c", str(src), "-o", str(obj)],
                                 capture_output=True, text=True)
            if res.returncode != 0:
                raise RuntimeError(f"nvcc failed for {name} ({tag} variant):\n{res.stdout}\n{res.stderr}")
    if force or not lib.exists() or lib.stat().st_mtime < max(o.stat().st_mtime for o in objs):
        tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
        res = subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp),
                              *map(str, objs)], capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"link failed ({tag} variant):\n{res.stdout}\n{res.stderr}")
        os.replace(tmp, lib)
    return lib


def build_giveup_variant(force: bool = False) -> Path:
    """Builds ``liblt_attn_giveup.so`` (the give-up test loads it by path)."""
    return _build_variant(GIVEUP_LIB, GIVEUP_FLAGS, "giveup", force)


def build_timeline_variant(force: bool = False) -> Path:
    """Builds ``liblt_attn_timeline.so`` (``python -m paper_2606_10415_b200.timeline`` loads it by path)."""
    return _build_variant(TIMELINE_LIB, TIMELINE_FLAGS, "timeline", force)


def build_microbench() -> Path:
    """Builds the stand-alone microbenchmark ``build/sm_limits`` from ``csrc/microbench/sm_limits.cu``."""
    OBJ.mkdir(exist_ok=True)
    src = CSRC / "microbench" / "sm_limits.cu"
    res = subprocess.run([_nvcc(), *[f for f in NVCC_FLAGS if f not in ("-Xptxas", "-v")], str(src), "-o", str(MICROBENCH)],
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src.name}:\n{res.stdout}\n{res.stderr}")
    return MICROBENCH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--giveup" in sys.argv:
        print(build_giveup_variant(force="--force" in sys.argv))
    if "--timeline" in sys.argv:
        print(build_timeline_variant(force="--force" in sys.argv))
    if "--microbench" in sys.argv:
        print(build_microbench())
