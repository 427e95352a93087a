"""Build the CUDA library in-tree: nvcc, sm_100a only, one object per source, then one shared object."""
from __future__ import annotations

import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libonela.so"
OBJ = PKG / "build"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-I", str(ROOT / "include"), "-I", str(CSRC),
] + os.environ.get("ONELA_NVCC_EXTRA", "").split()   # extra flags (e.g. -D switches) for experiments


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (cand == "nvcc" or Path(cand).exists()):
            return cand
    raise RuntimeError("nvcc not found")


def sources() -> list[Path]:
    return sorted(CSRC.glob("*.cu"))


def _stale(target: Path, deps) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(d.stat().st_mtime > t for d in deps)


# A second library for the tests of the bounded waits: the same sources with a short wait limit and a hook that
# makes one arrival go missing.  The product never loads it.
TESTHOOKS_LIB = PKG / "libonela_testhooks.so"
TESTHOOKS_FLAGS = ["-DONELA_TEST_HOOKS", "-DONELA_WAIT_LIMIT=(1<<14)"]


def build_testhooks(force: bool = False) -> Path:
    return build(force=force, lib=TESTHOOKS_LIB, obj_dir=PKG / "build_testhooks", extra=TESTHOOKS_FLAGS)


# A third one for looking INSIDE the two tensor-core decode kernels: clock stamps of CTA 0's role milestones
# (timeline.py).
TIMELINE_LIB = PKG / "libonela_timeline.so"


def build_timeline(force: bool = False) -> Path:
    return build(force=force, lib=TIMELINE_LIB, obj_dir=PKG / "build_timeline", extra=["-DONELA_WY_TL", "-DONELA_WS_TL"])


def build(force: bool = False, verbose: bool = False, lib: Path = LIB, obj_dir: Path = OBJ, extra=()) -> Path:
    """Compile every .cu under csrc/ for sm_100a and link libonela.so next to this file."""
    OBJ, LIB = obj_dir, lib
    OBJ.mkdir(exist_ok=True)
    headers = list(CSRC.glob("*.h")) + list(CSRC.glob("*.cuh")) + list((ROOT / "include").glob("*.h"))
    nvcc = _nvcc()
    jobs = []
    for src in sources():
        obj = OBJ / (src.stem + ".o")
        if force or _stale(obj, [src, *headers]):
            cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", str(src), "-o", str(obj)]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
        return r.stderr

    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as ex:
        logs = list(ex.map(run, jobs))
    if verbose:
        print("\n".join(logs))
    objs = [OBJ / (s.stem + ".o") for s in sources()]
    if force or jobs or _stale(LIB, objs):
        run([nvcc, "-shared", "-o", str(LIB), *map(str, objs), "-cudart", "shared"])
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--testhooks" in sys.argv:
        print(build_testhooks(force="--force" in sys.argv))
