"""Builds libwtconv_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

The kernels are spread over per-dtype instantiation units (csrc/inst_*.cu) that compile in parallel; objects
are cached under build/ (not tracked) and rebuilt when any source or header is newer."""
import concurrent.futures
import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libwtconv_b200.so")
OBJ_DIR = os.path.join(os.path.dirname(HERE), "build", "obj")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps_mtime(path, seen=None):
    """Newest modification time of a source file and of everything it includes with quotes, recursively."""
    seen = set() if seen is None else seen
    path = os.path.normpath(path)
    if path in seen or not os.path.exists(path):
        return 0.0
    seen.add(path)
    m = os.path.getmtime(path)
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line.startswith("#include \""):
                m = max(m, _deps_mtime(os.path.join(os.path.dirname(path), line.split('"')[1]), seen))
    return m


def _compile(nvcc, src, obj):
    res = subprocess.run([nvcc] + NVCC_FLAGS + ["-c", "-o", obj, src], stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                         text=True)
    return src, res.returncode, res.stdout


def build(force=False, verbose=False):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    jobs, objs = [], []
    for src in _sources():
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < _deps_mtime(src):
            jobs.append((src, obj))
    if not jobs and os.path.exists(LIB) and os.path.getmtime(LIB) >= max(os.path.getmtime(o) for o in objs):
        return LIB
    log = []
    with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 4))) as ex:
        for src, rc, out in ex.map(lambda j: _compile(nvcc, *j), jobs):
            log.append("==== %s\n%s" % (os.path.basename(src), out))
            if verbose or rc != 0:
                print(log[-1])
            if rc != 0:
                raise RuntimeError("nvcc failed compiling %s" % src)
    with open(os.path.join(os.path.dirname(OBJ_DIR), "ptxas_info.txt"), "a" if not force else "w") as f:
        f.write("\n".join(log))  # registers / spills / shared memory per kernel (not tracked)
    tmp = LIB + ".tmp%d" % os.getpid()
    res = subprocess.run([nvcc, "--shared", "-o", tmp] + objs, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if res.returncode != 0:
        print(res.stdout)
        raise RuntimeError("nvcc failed linking %s" % LIB)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
