"""Builds libstief.so (sm_100a only) in-tree with nvcc.  `python -m paper_2601_21686_b200.build [--force] [--verbose]`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "libstief.so")
KEY_RANKS = (32, 48, 64, 96, 128)

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    nv = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nv):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return nv


def _units():
    """(source, object, extra flags) for every translation unit."""
    units = [(os.path.join(CSRC, f + ".cu"), os.path.join(OBJ, f + ".o"), [])
             for f in ("stief_api", "stief_small", "stief_prefill", "stief_prefill_tc", "stief_noalloc", "stief_quant", "stief_rank_select", "stief_mq", "stief_selftest")
             if os.path.exists(os.path.join(CSRC, f + ".cu"))]
    for rk in KEY_RANKS:
        units.append((os.path.join(CSRC, "stief_decode_inst.cu"), os.path.join(OBJ, f"stief_decode_rk{rk}.o"),
                      [f"-DSTIEF_RK={rk}"]))
        units.append((os.path.join(CSRC, "stief_mq_inst.cu"), os.path.join(OBJ, f"stief_mq_rk{rk}.o"),
                      [f"-DSTIEF_RK={rk}"]))
        for bits in (8, 4):
            units.append((os.path.join(CSRC, "stief_decode_q_inst.cu"), os.path.join(OBJ, f"stief_decode_q_rk{rk}_b{bits}.o"),
                          [f"-DSTIEF_RK={rk}", f"-DSTIEF_QBITS={bits}"]))
    return units


def _newest_header() -> float:
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    hs.append(os.path.join(ROOT, "include", "stief.h"))
    return max(os.path.getmtime(h) for h in hs)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    nv = _nvcc()
    hdr = _newest_header()
    todo = []
    for src, obj, extra in _units():
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr):
            todo.append((src, obj, extra))

    def compile_one(u):
        src, obj, extra = u
        cmd = [nv, *NVCC_FLAGS, *extra, "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        r = subprocess.run(cmd, capture_output=True, text=True)
        return u, r

    if todo:
        with ThreadPoolExecutor(max_workers=min(8, len(todo))) as ex:
            for (src, obj, _), r in ex.map(compile_one, todo):
                if verbose or r.returncode != 0:
                    sys.stderr.write(f"--- {os.path.basename(obj)}\n{r.stdout}{r.stderr}\n")
                if r.returncode != 0:
                    raise RuntimeError(f"nvcc failed on {src}")
    objs = [u[1] for u in _units()]
    if todo or force or not os.path.exists(LIB) or os.path.getmtime(LIB) < max(os.path.getmtime(o) for o in objs):
        r = subprocess.run([nv, "-shared", "-o", LIB, *objs, "-cudart", "static"], capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
