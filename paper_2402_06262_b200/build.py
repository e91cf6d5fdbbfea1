"""Build libroco.so (hand-written CUDA for sm_100a) in-tree with nvcc."""
import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libroco.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "--expt-extended-lambda", "-Xcompiler", "-fPIC", "-shared"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) + \
        glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles every csrc/*.cu to an object (in parallel, one nvcc per file) and links libroco.so."""
    if not force and not _stale():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    compile_flags = [f for f in FLAGS if f != "-shared"] + (["-Xptxas", "-v"] if verbose else [])

    def compile_one(src):
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        res = subprocess.run([NVCC] + compile_flags + ["-c", "-o", obj, src], capture_output=True, text=True)
        return src, obj, res

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        done = list(pool.map(compile_one, sources()))
    for src, _, res in done:   # in source order, so the log reads like a serial build
        if verbose or res.returncode != 0:
            print(res.stdout, end="")
            print(res.stderr, end="")
        if res.returncode != 0:
            raise subprocess.CalledProcessError(res.returncode, res.args)
    subprocess.run([NVCC, "-shared", "-o", LIB] + [obj for _, obj, _ in done], check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
