"""Build libdet_linear.so (hand-written CUDA for sm_100a) in-tree with nvcc.

The arithmetic flags matter: no fused-multiply-add contraction the source did not write
(-fmad=false), no flush-to-zero, IEEE division and square root, never --use_fast_math.  Every
multiply-accumulate in the kernels is an explicit fma intrinsic or fma.rn PTX instruction.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libdet_linear.so")
OBJ_DIR = os.path.join(HERE, "csrc", "obj")

# (source, extra defines): the decode tilings are compiled once per weight format
SOURCES = [("plan.cpp", ()), ("capi.cu", ()), ("kernels_generic.cu", ()), ("kernels_decode.cu", ()),
           ("kernels_prefill.cu", ()), ("prefill_tma.cu", ()), ("bench_kernels.cu", ()), ("noalloc.cu", ()), ("ablation.cu", ()), ("rmsnorm.cu", ()), ("attention.cu", ())]
SOURCES += [(f"decode_inst_{i}.cu", (f"-DDET_WF={wf}",)) for wf in (0, 1, 2) for i in range(4)]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false", "-ftz=false", "-prec-div=true", "-prec-sqrt=true",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-I", INCLUDE, "-I", CSRC,
]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile what is out of date and link the shared library; return its path."""
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = os.environ.get("DET_EXTRA_NVCC_FLAGS", "").split()      # e.g. instrumentation defines for experiments
    os.makedirs(OBJ_DIR, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE) if f.endswith(".h")]
    objs, procs = [], []
    for src, defines in SOURCES:
        sp = os.path.join(CSRC, src)
        tag = "".join(d.replace("-D", "_").replace("=", "") for d in defines)
        op = os.path.join(OBJ_DIR, os.path.splitext(src)[0] + tag + ".o")
        objs.append(op)
        if force or _stale(op, [sp] + headers):
            cmd = [nvcc, *NVCC_FLAGS, *extra, *defines, "-x", "cu", "-c", sp, "-o", op]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src} ---\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if force or procs or _stale(LIB, objs):
        cmd = [nvcc, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
               "-Xcompiler", "-fPIC", "-cudart", "static"]
        subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
