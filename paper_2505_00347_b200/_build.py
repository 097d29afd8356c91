"""In-tree nvcc build of the CUDA library (sm_100a only)."""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
LIB = PKG / "libsolo_b200.so"
OBJ_DIR = PKG / "_build"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC", f"-I{INCLUDE}", f"-I{CSRC}",
]

# (source, object name, extra defines)
UNITS = [
    ("solo_api.cu", "solo_api.o", []),
    ("solo_dispatch.cu", "solo_dispatch.o", []),
    ("solo_step_inst.cu", "solo_step_bm2.o", ["-DSOLO_BM=2"]),
    ("solo_step_inst.cu", "solo_step_bm3.o", ["-DSOLO_BM=3"]),
    ("solo_step_inst.cu", "solo_step_bm4.o", ["-DSOLO_BM=4"]),
    ("solo_step_inst.cu", "solo_step_bm8.o", ["-DSOLO_BM=8"]),
    ("solo_fast_inst.cu", "solo_fast_bm2.o", ["-DSOLO_BM=2"]),
    ("solo_fast_inst.cu", "solo_fast_bm3.o", ["-DSOLO_BM=3"]),
    ("solo_fast_inst.cu", "solo_fast_bm4.o", ["-DSOLO_BM=4"]),
    ("solo_fast_inst.cu", "solo_fast_bm8.o", ["-DSOLO_BM=8"]),
    *[("solo_fast16_inst.cu", f"solo_fast16_g{g}_m{m}.o", [f"-DSOLO_G={g}", f"-DSOLO_MODES={m}"])
      for g in (4, 8, 16) for m in (0, 1, 2)],
]


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.isabs(c) and os.path.exists(c) or not os.path.isabs(c)):
            return c
    return "nvcc"


def _source_key() -> str:
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for f in sorted(list(CSRC.glob("*.cu*")) + list(CSRC.glob("*.h")) + list(INCLUDE.glob("*.h"))):
        h.update(f.name.encode())
        h.update(f.read_bytes())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False, ptxas_info: bool = False) -> Path:
    """Compile every translation unit for sm_100a and link libsolo_b200.so in-tree."""
    key = _source_key()
    stamp = OBJ_DIR / "stamp"
    if not force and LIB.exists() and stamp.exists() and stamp.read_text() == key:
        return LIB
    OBJ_DIR.mkdir(exist_ok=True)
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if ptxas_info else []

    def compile_one(unit):
        src, obj, defs = unit
        cmd = [nvcc, *NVCC_FLAGS, *extra, *defs, "-c", str(CSRC / src), "-o", str(OBJ_DIR / obj)]
        r = subprocess.run(cmd, capture_output=True, text=True)
        return unit, r

    with ThreadPoolExecutor(max_workers=min(len(UNITS), os.cpu_count() or 4)) as ex:
        for unit, r in ex.map(compile_one, UNITS):
            if verbose or ptxas_info or r.returncode:
                sys.stderr.write(f"[{unit[1]}]\n{r.stdout}{r.stderr}")
            if r.returncode:
                raise RuntimeError(f"nvcc failed on {unit[0]} ({unit[2]})")
    objs = [str(OBJ_DIR / u[1]) for u in UNITS]
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp),
                    *objs], check=True)
    os.replace(tmp, LIB)
    stamp.write_text(key)
    return LIB


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True, ptxas_info="--ptxas" in sys.argv)
    print(LIB)
