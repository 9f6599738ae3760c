"""Builds libd2mhe.so (the CUDA library behind the C ABI) in-tree with nvcc for sm_100a."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libd2mhe.so")
SOURCES = ["kern_pdec.cu", "kern_encrypt.cu", "kern_ntt.cu", "kern_ntt32.cu", "kern_keys.cu", "kern_stream.cu", "kern_convert.cu", "kern_bootstrap.cu", "kern_probe.cu", "kern_proto32.cu", "d2mhe_host.cu",
           "d2mhe_round_static.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--extended-lambda", "-Xcompiler", "-fPIC",
]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale():
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [
        os.path.join(HERE, "..", "include", "d2mhe.h")
    ]
    return any(os.path.getmtime(d) > built for d in deps if os.path.isfile(d))


def build(force=False, verbose=False, defines=()):
    """Compile every .cu for sm_100a and link the shared library next to this file."""
    if not force and not _stale():
        return LIB
    obj_dir = os.path.join(HERE, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    extra = (["-Xptxas", "-v"] if verbose else []) + ["-D" + d for d in defines]

    def compile_one(job):
        src, checked = job
        obj = os.path.join(obj_dir, src.replace(".cu", "_chk.o" if checked else ".o"))
        cmd = [nvcc] + NVCC_FLAGS + extra + (["-DD2MHE_CHECKED"] if checked else []) + [
            "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed for %s:\n%s" % (src, r.stderr))
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    # every kernel file is compiled twice: as it is, and with index checks in every kernel (the build
    # that contexts created with D2MHE_FLAG_DEVICE_CHECKS launch)
    jobs = [(s, False) for s in SOURCES] + [(s, True) for s in SOURCES if s.startswith("kern_")]
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as ex:
        objs = list(ex.map(compile_one, jobs))
    tmp = LIB + ".%d.tmp" % os.getpid()
    r = subprocess.run([nvcc, "-shared", "-o", tmp] + objs + ["-lcudart"], capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("link failed:\n" + r.stderr)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv,
                defines=[a[2:] for a in sys.argv if a.startswith("-D")]))
