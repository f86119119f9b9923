"""Build the DSBD CUDA library (sm_100a) in-tree with nvcc."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
BUILD_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(BUILD_DIR, "libdsbd.so")
SOURCES = ["dsbd_api.cu", "dsbd_verify.cu", "dsbd_attention.cu", "dsbd_attention_tc.cu", "dsbd_kv_commit.cu", "dsbd_forest.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xptxas=-v", "-Xcompiler", "-fPIC",
              "-I", os.path.join(ROOT, "include"), "-I", CSRC] + os.environ.get("DSBD_NVCC_EXTRA", "").split()


def _deps():
    deps = [os.path.join(ROOT, "include", "dsbd.h")]
    for name in os.listdir(CSRC):
        deps.append(os.path.join(CSRC, name))
    return deps


def stale():
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(p) > t for p in _deps())


def build(force=False, verbose=False):
    """Compile every .cu for sm_100a and link libdsbd.so; returns its path."""
    if not force and not stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(BUILD_DIR, exist_ok=True)
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(BUILD_DIR, src.replace(".cu", ".o"))
        objs.append(obj)
        cmd = [nvcc] + NVCC_FLAGS + ["-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT)))
    for src, p in procs:
        out = p.communicate()[0].decode()
        if verbose or p.returncode:
            print(out)
        if p.returncode:
            raise RuntimeError("nvcc failed on %s" % src)
    tmp = LIB_PATH + ".tmp.%d" % os.getpid()
    subprocess.run([nvcc, "-shared", "-Wno-deprecated-gpu-targets", "-o", tmp] + objs + ["-lcudart"], check=True)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


WAIT_TEST_LIB = os.path.join(BUILD_DIR, "libdsbd_waittest.so")
PHASES_LIB = os.path.join(BUILD_DIR, "libdsbd_phases.so")


def _build_variant(lib_path, tag, sources, define, force):
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= max(
            os.path.getmtime(p) for p in _deps()):
        return lib_path
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(BUILD_DIR, exist_ok=True)
    objs, procs = [], []
    for src in sources:
        obj = os.path.join(BUILD_DIR, tag + "_" + src.replace(".cu", ".o"))
        objs.append(obj)
        procs.append(subprocess.Popen([nvcc] + NVCC_FLAGS + [define, "-c", os.path.join(CSRC, src), "-o", obj],
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT))
    for pr in procs:
        out = pr.communicate()[0].decode()
        if pr.returncode:
            print(out)
            raise RuntimeError("nvcc failed building %s" % lib_path)
    tmp = lib_path + ".tmp.%d" % os.getpid()
    subprocess.run([nvcc, "-shared", "-Wno-deprecated-gpu-targets", "-o", tmp] + objs + ["-lcudart"], check=True)
    os.replace(tmp, lib_path)
    return lib_path


def build_wait_test(force=False):
    """A second library for one test: the attention kernel compiled with DSBD_TEST_WAIT_TIMEOUT
    (short bounded waits, one tile never delivered).  Nothing but that test loads it."""
    return _build_variant(WAIT_TEST_LIB, "waittest", ("dsbd_api.cu", "dsbd_attention.cu", "dsbd_attention_tc.cu"),
                          "-DDSBD_TEST_WAIT_TIMEOUT", force)


def build_phase_timing(force=False):
    """The library compiled with DSBD_PHASE_TIMING: the per-request verification kernel records
    %globaltimer stamps of its phases behind its workspace.  Loaded by `bench.py --verify-phases`
    only (a measuring aid, slower than the product library)."""
    return _build_variant(PHASES_LIB, "phases", SOURCES, "-DDSBD_PHASE_TIMING", force)


if __name__ == "__main__":
    print(build(force=True, verbose=True))
