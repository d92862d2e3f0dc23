"""Builds libpyr.so in-tree from csrc/ with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpyr.so")
SOURCES = ["pyr_host.cu", "prefill_simt.cu", "prefill_tc.cu", "attn_tc.cu", "select_compact.cu", "decode.cu", "decode_noalloc.cu", "gen_reselect.cu", "glue.cu", "gemm_tc.cu", "gemm_skinny.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "pyr.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def _check_register_split(ptxas_log: str) -> None:
    """The attention kernel moves registers between its warpgroups (setmaxnreg) and sizes the split
    for kRegsLaunch registers per thread at launch (csrc/attn_tc.cu). If ptxas ever allocates fewer,
    the softmax warps would wait for registers that do not exist: refuse to build that. Spills in
    that kernel mean the split no longer fits the code: refuse those too."""
    import re
    with open(os.path.join(CSRC, "attn_tc.cu")) as f:
        want = int(re.search(r"kRegsLaunch\s*=\s*(\d+)", f.read()).group(1))
    m = re.search(r"attn_tc_kernel.*?(\d+) bytes spill stores.*?Used (\d+) registers", ptxas_log, re.S)
    if not m:
        raise RuntimeError("ptxas log has no register count for attn_tc_kernel")
    if int(m.group(2)) != want:
        raise RuntimeError(f"attn_tc_kernel launches with {m.group(2)} registers per thread, not the {want} its "
                           "setmaxnreg split (kRegsLaunch) assumes: adjust the split in csrc/attn_tc.cu")
    if int(m.group(1)) != 0:
        raise RuntimeError(f"attn_tc_kernel spills {m.group(1)} bytes: its register split no longer fits the code")


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    nvcc = _nvcc()
    procs = []
    for src in SOURCES:
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c",
               os.path.join(CSRC, src), "-o", obj]
        procs.append((src, obj, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    objs = []
    log = []
    for src, obj, p in procs:
        out, _ = p.communicate()
        log.append(f"== {src}\n{out}")
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{out}")
        objs.append(obj)
    with open(os.path.join(objdir, "ptxas.log"), "w") as f:
        f.write("\n".join(log))
    _check_register_split("\n".join(log))
    if verbose:
        print("\n".join(log))
    cmd = [nvcc, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}{r.stderr}")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
