"""Build the CUDA library in-tree: paper_2603_05959_b200/libovggt.so (sm_100a only)."""
import os
import re
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libovggt.so")
OUT_CHECKED = os.path.join(HERE, "libovggt_checked.so")     # the same library built with -DOVGGT_BOUNDS_CHECK
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh")))


def needs_build(out: str = OUT) -> bool:
    if not os.path.exists(out):
        return True
    deps = sources() + [os.path.join(os.path.dirname(HERE), "include", "ovggt.h")]
    return any(os.path.getmtime(d) > os.path.getmtime(out) for d in deps)


def check_register_pool(ptxas_log: str) -> None:
    """The attention kernel moves registers between its warpgroups with setmaxnreg, inside the pool it was launched
    with; an increase the pool cannot serve would wait for ever.  The source states the launch count it was budgeted
    for (kRegsLaunch); refuse a build whose ptxas report says otherwise."""
    src = open(os.path.join(CSRC, "attn_tcgen05.cuh")).read()
    want = int(re.search(r"constexpr int kRegsLaunch = (\d+);", src).group(1))
    m = re.search(r"Compiling entry function '[^']*k_attn_tcgen05[^']*'.*?Used (\d+) registers", ptxas_log, re.S)
    if not m:
        raise RuntimeError("ptxas report for k_attn_tcgen05 not found")
    if int(m.group(1)) != want:
        raise RuntimeError(f"k_attn_tcgen05 is launched with {m.group(1)} registers, budgeted for {want}")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """checked: the variant in which every index a kernel reads from device memory is range-checked (a bad one is
    skipped and reported through the status word); written to libovggt_checked.so, loaded by the binding when the
    environment says OVGGT_LIBRARY=checked."""
    OUT = OUT_CHECKED if checked else globals()["OUT"]
    if not force and not needs_build(OUT):
        return OUT
    tmp = OUT + ".tmp"
    cmd = [NVCC, "-Xptxas", "-v", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "--cudart", "static"] + (["-DOVGGT_BOUNDS_CHECK"] if checked else []) + [
           "-o", tmp, os.path.join(CSRC, "ovggt_api.cu"), "-ldl"]
    r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or r.returncode != 0:
        print(r.stdout, file=sys.stderr)
    if r.returncode != 0:
        raise subprocess.CalledProcessError(r.returncode, cmd)
    try:
        check_register_pool(r.stdout)
    except Exception:
        os.remove(tmp)
        raise
    os.replace(tmp, OUT)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
