"""Compile the CUDA sources into paper_2211_10438_b200/libsq.so for sm_100a (in-tree build).

nvcc cross-compiles without a GPU.  Run as `python -m paper_2211_10438_b200.build`.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsq.so")
SOURCES = ["sq_api.cu", "sq_stream_kernels.cu", "sq_gemm_sm100.cu", "sq_noalloc.cu",
           "sq_row_pipeline.cu", "sq_decode_sm100.cu", "sq_attention_sm100.cu", "sq_kv_attention.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _nvcc():
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.sep not in c or os.path.exists(c)):
            return c
    raise RuntimeError("nvcc not found")


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_trace() -> str:
    """Tuning build: libsq_trace.so, the same library with the timestamp traces of the decode-shaped GEMM
    (-DSQ_DEC_TRACE) and of the prefill GEMM's MMA warp (-DSQ_GEMM_TRACE) compiled in.  Never loaded by the binding unless LIB_PATH is pointed at it."""
    out = os.path.join(HERE, "libsq_trace.so")
    subprocess.run([_nvcc(), *NVCC_FLAGS, "-DSQ_DEC_TRACE", "-DSQ_GEMM_TRACE", "-shared", *[os.path.join(CSRC, s) for s in SOURCES], "-o", out],
                   check=True)
    return out


def build_issue_only() -> str:
    """Ceiling build: libsq_issue_only.so, in which the prefill GEMM loads no operand and stores no result
    (-DSQ_GEMM_ISSUE_ONLY): what the tensor pipe sustains on its own.  For `workloads gemm --lib ...` only."""
    out = os.path.join(HERE, "libsq_issue_only.so")
    subprocess.run([_nvcc(), *NVCC_FLAGS, "-DSQ_GEMM_ISSUE_ONLY", "-shared", *[os.path.join(CSRC, s) for s in SOURCES], "-o", out],
                   check=True)
    return out


def build_no_nsplit() -> str:
    """Tuning build: libsq_no_nsplit.so, in which the prefill GEMM never cuts the tiles of a partly filled last
    wave into column parts (-DSQ_GEMM_NO_NSPLIT): the "without" arm of that split's A/B timings."""
    out = os.path.join(HERE, "libsq_no_nsplit.so")
    subprocess.run([_nvcc(), *NVCC_FLAGS, "-DSQ_GEMM_NO_NSPLIT", "-shared", *[os.path.join(CSRC, s) for s in SOURCES], "-o", out],
                   check=True)
    return out


def build_variant(name: str, defines) -> str:
    """Tuning build: libsq_<name>.so, the library compiled with extra -D flags.  The kernels read a few of their
    constants through such macros so that the A/B timings quoted in their comments can be repeated: SQ_KV_STAGES
    (ring stages per warp of the KV-cache attention, default 2), SQ_DEC_STAGES (ring stages of the decode GEMM,
    default 10), SQ_LN_NO_TM (LayerNorm parameters in shared instead of tensor memory), SQ_GEMM_NO_L2_HINTS,
    SQ_GEMM_NO_NSPLIT.  Used through `workloads ... --lib`."""
    out = os.path.join(HERE, "libsq_%s.so" % name)
    subprocess.run([_nvcc(), *NVCC_FLAGS, *defines, "-shared", *[os.path.join(CSRC, s) for s in SOURCES], "-o", out], check=True)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "sq.h"))
    objdir = os.path.join(HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    objs, procs = [], []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(objdir, src.replace(".cu", ".o"))
        objs.append(o)
        if force or _stale(o, [s] + headers):
            cmd = [_nvcc(), *NVCC_FLAGS, "-c", s, "-o", o]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(out)
        if p.returncode:
            raise RuntimeError("nvcc failed on %s" % src)
    if force or procs or _stale(LIB, objs):
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", *objs, "-o", tmp],
                       check=True)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    if "--trace" in sys.argv:
        print(build_trace())
    elif "--issue-only" in sys.argv:
        print(build_issue_only())
    elif "--no-nsplit" in sys.argv:
        print(build_no_nsplit())
    elif "--variant" in sys.argv:  # --variant NAME -DFLAG[=VALUE] ...
        print(build_variant(sys.argv[sys.argv.index("--variant") + 1], [a for a in sys.argv if a.startswith("-D")]))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
