"""Build libsysconv.so in-tree with nvcc for sm_100a.

``python -m paper_2010_15884_b200.build`` compiles every ``csrc/*.cu`` to an
object (in parallel, only when the source or one of the headers it includes,
as recorded by the compiler in a dependency file, is newer than the object)
and links them into ``paper_2010_15884_b200/libsysconv.so``.  No GPU is needed.
"""
import concurrent.futures
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "libsysconv.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _newest_header():
    deps = glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    deps.append(os.path.abspath(__file__))
    return max(os.path.getmtime(p) for p in deps)


def _recorded_deps(obj):
    """Files the object was compiled from, read from the dependency file nvcc wrote beside it (None if absent)."""
    dep = obj + ".d"
    if not os.path.exists(dep):
        return None
    with open(dep) as f:
        words = f.read().replace("\\\n", " ").split()
    files = [os.path.normpath(os.path.join(CSRC, w)) for w in words[1:] if not w.endswith(":")]
    root = os.path.abspath(os.path.join(HERE, ".."))
    mine = [w for w in files if w.startswith(root)]     # this repository's sources and headers; not the toolkit's
    return mine or None


def _stale(src, obj, hdr_time):
    if not os.path.exists(obj):
        return True
    built = os.path.getmtime(obj)
    if built < max(os.path.getmtime(src), os.path.getmtime(os.path.abspath(__file__))):
        return True
    deps = _recorded_deps(obj)
    if deps is None:
        return built < hdr_time             # no record: any newer header counts
    return any((not os.path.exists(d)) or os.path.getmtime(d) > built for d in deps)


def _compile(src, obj, verbose):
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-MD", "-MF", obj + ".d", "-c", src, "-o", obj]
    res = subprocess.run(cmd, capture_output=True, text=True, cwd=CSRC)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, res.stdout, res.stderr))
    return res.stderr


def build(force=False, verbose=False, jobs=None):
    """Compile and link the CUDA library; returns the path of the shared object."""
    os.makedirs(OBJ_DIR, exist_ok=True)
    sources = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    if not sources:
        raise RuntimeError("no CUDA sources under %s" % CSRC)
    hdr_time = _newest_header()
    todo, objs = [], []
    for src in sources:
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or _stale(src, obj, hdr_time):
            todo.append((src, obj))
    if todo:
        jobs = jobs or min(len(todo), os.cpu_count() or 4)
        with concurrent.futures.ThreadPoolExecutor(jobs) as pool:
            futs = {pool.submit(_compile, s, o, verbose): s for s, o in todo}
            for fut in concurrent.futures.as_completed(futs):
                log = fut.result()
                if verbose and log:
                    sys.stderr.write(log)
    if todo or not os.path.exists(LIB_PATH) or any(os.path.getmtime(o) > os.path.getmtime(LIB_PATH) for o in objs):
        tmp = LIB_PATH + ".tmp.%d" % os.getpid()
        cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("link failed:\n%s\n%s" % (res.stdout, res.stderr))
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
