"""Compile the CUDA library for sm_100a with nvcc, in-tree.

``python -m paper_2604_18616_b200.build`` (or ``build_cuda()``) writes
``libave_attn.so`` next to this file.  nvcc cross-compiles without a GPU.

The build reads ptxas' resource report and refuses an image in which an
attention kernel got fewer registers per thread than its warp roles' register
split draws on (``setmaxnreg.inc`` beyond the CTA's allocation never returns).
The library repeats the check at run time on the loaded image.
"""
from __future__ import annotations

import os
import re
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libave_attn.so")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-shared", "-Xcompiler", "-fPIC",
    "-Xptxas", "-v",
]

# Register split of the attention kernel (WsCfg in csrc/attn_fwd_ws.cuh): 384 threads, of which one
# warpgroup keeps 64 registers per thread and two take 216.
ATTN_THREADS = 384
ATTN_REGS_NEEDED = 128 * 64 + 256 * 216
# The single-sub-tile kernel (OneCfg in csrc/attn_fwd_1t.cuh): 256 threads, 48 and 208 registers.
ONE_THREADS = 256
ONE_REGS_NEEDED = 128 * 48 + 128 * 208
# The MoE GEMM (MoeGemmCfg in csrc/moe_fp8.cuh): 384 threads, 40 and 232 registers.
MOE_THREADS = 384
MOE_REGS_NEEDED = 128 * 40 + 256 * 232


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh"))) + \
        [os.path.join(INCLUDE, h) for h in sorted(os.listdir(INCLUDE)) if h.endswith(".h")]


def kernel_registers(ptxas_report: str) -> dict:
    """{mangled kernel name: registers per thread} from ``-Xptxas -v`` output."""
    regs = {}
    current = None
    for line in ptxas_report.splitlines():
        m = re.search(r"Compiling entry function '([^']+)'", line)
        if m:
            current = m.group(1)
            continue
        m = re.search(r"Used (\d+) registers", line)
        if m and current:
            regs[current] = int(m.group(1))
            current = None
    return regs


def check_register_split(ptxas_report: str) -> dict:
    """Raise if an attention kernel of the report cannot satisfy its register split."""
    regs = {k: v for k, v in kernel_registers(ptxas_report).items() if "attn_fwd" in k or "moe_gemm" in k}
    if not regs:
        raise RuntimeError("ptxas reported no attention kernel: cannot verify the register split")
    for name, n in regs.items():
        threads, needed = (ONE_THREADS, ONE_REGS_NEEDED) if "attn_fwd_1t" in name else \
            (MOE_THREADS, MOE_REGS_NEEDED) if "moe_gemm" in name else (ATTN_THREADS, ATTN_REGS_NEEDED)
        if threads * n < needed:
            raise RuntimeError("%s was compiled with %d registers per thread; its warp roles need %d x %d >= %d" % (
                name, n, threads, n, needed))
    return regs


def build_cuda(force: bool = False, verbose: bool = False) -> str:
    newest = max(os.path.getmtime(s) for s in _sources())
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= newest:
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB_PATH + ".tmp%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + ["-o", tmp, os.path.join(CSRC, "ave_attn.cu")]
    r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout)
    if r.returncode != 0:
        raise subprocess.CalledProcessError(r.returncode, cmd)
    try:
        check_register_split(r.stdout)
    except Exception:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build_cuda(force="--force" in sys.argv, verbose="-v" in sys.argv))
