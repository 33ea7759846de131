"""Builds the C-ABI CUDA library ``libdlm.so`` in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libdlm.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-Xptxas", "-v",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ into libdlm.so (cross-compiles without a GPU)."""
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc, *NVCC_FLAGS, "-I", INCLUDE, "-I", CSRC, "-o", tmp, *sources()]
    proc = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed building libdlm.so")
    check_attention_registers(proc.stdout)
    os.replace(tmp, LIB)
    return LIB


# The attention kernel moves registers between its warpgroups with setmaxnreg: 8 softmax warps grow to 216 registers a
# thread from what the other 4 warps give up when they shrink to 72, which balances only if the kernel is launched
# with 168 (attn_step.cu: kRegsSoftmax, kRegsOther, register_budget_ok).  A compiler that allocates another number
# would make every attention call fail at run time with DLM_ERR_UNSUPPORTED; fail the build instead.
ATTENTION_REGISTERS = 168


def check_attention_registers(ptxas_log: str) -> None:
    seen, name = 0, None
    for line in ptxas_log.splitlines():
        if "Compiling entry function" in line:
            name = line.split("'")[1] if "'" in line else line
        elif "Used" in line and "registers" in line and name is not None:
            if "attn_step_sm100_kernel" in name:
                seen += 1
                regs = int(line.split("Used")[1].split("registers")[0])
                if regs != ATTENTION_REGISTERS:
                    raise RuntimeError(f"{name}: ptxas allocated {regs} registers, the kernel's register split needs "
                                       f"{ATTENTION_REGISTERS}")
            name = None
    if seen == 0:
        raise RuntimeError("no attention kernel found in the ptxas log: cannot check its register count")


if __name__ == "__main__":
    build(force=True, verbose=True)
    print(LIB)
