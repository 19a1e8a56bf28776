"""Builds the CUDA library in-tree: csrc/*.cu -> libattn_b200.so (sm_100a only)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libattn_b200.so")
SOURCES = ["attn_api.cu"]
HEADERS = ["ptx.cuh", "attn_fwd_kernel.cuh", "attn_fwd_sb3.cuh", "attn_fwd_pair.cuh", "attn_fwd_w16.cuh", "attn_merge_kernel.cuh", os.path.join("..", "..", "include", "attn.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(_CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def _compile(out_path: str, extra_flags: list[str] | None, verbose: bool) -> str:
    """nvcc -> out_path (atomically); returns the compiler's log (ptxas -v: registers, spills)."""
    tmp = out_path + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]
    cmd += list(extra_flags or [])
    cmd += [os.path.join(_CSRC, s) for s in SOURCES]
    cmd += ["-o", tmp]
    res = subprocess.run(cmd, capture_output=True, text=True)
    log = res.stdout + res.stderr
    if verbose or res.returncode != 0:
        print(log)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(out_path)}")
    os.replace(tmp, out_path)
    return log


def build(force: bool = False, verbose: bool = False, extra_flags: list[str] | None = None) -> str:
    """Compile the in-tree library for sm_100a with nvcc.  Works on a machine without a GPU."""
    if not force and not is_stale():
        return LIB_PATH
    _compile(LIB_PATH, extra_flags, verbose)
    return LIB_PATH


def build_variant(out_path: str, extra_flags: list[str], verbose: bool = False) -> dict:
    """Compile another build of the same library (e.g. another register split: -DATTN_REGS_SOFTMAX=...)
    to `out_path`, leaving the in-tree one alone.  Returns {"path", "spill_store_bytes",
    "spill_load_bytes"} with the spill figures ptxas reports for the default forward kernel."""
    import re
    log = _compile(out_path, extra_flags, verbose)
    spills = {"path": out_path, "spill_store_bytes": None, "spill_load_bytes": None}
    m = re.search(r"Function properties for \S*15attn_fwd_kernelE\S*\n\s*(\d+) bytes stack frame, (\d+) bytes spill stores, "
                  r"(\d+) bytes spill loads", log)
    if m:
        spills.update(spill_store_bytes=int(m.group(2)), spill_load_bytes=int(m.group(3)))
    return spills


if __name__ == "__main__":
    print(build(force=True, verbose=True))
