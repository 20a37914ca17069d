"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librcp_w2a4.so")
LIB_CHECKED = os.path.join(HERE, "librcp_w2a4_checked.so")   # the guarded build (-DRCP_CHECKED), for tests
DRIVER = os.path.join(HERE, "e2e_driver")                     # host program: a decode step through the C ABI
SOURCES = ["rcp_api.cu"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    paths.append(os.path.join(os.path.dirname(HERE), "include", "rcp.h"))
    return max(os.path.getmtime(p) for p in paths)


def _compile(out: str, defines=(), verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC", "-o", out] + [f"-D{d}" for d in defines] + \
          [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source_mtime():
        return LIB
    return _compile(LIB, verbose=verbose)


def build_checked(force: bool = False) -> str:
    """The guarded build: the same sources with -DRCP_CHECKED (shared-memory addresses and TMA requests of the
    streaming kernel checked against the host's layout; a violation is reported through the status word)."""
    if not force and os.path.exists(LIB_CHECKED) and os.path.getmtime(LIB_CHECKED) >= _newest_source_mtime():
        return LIB_CHECKED
    return _compile(LIB_CHECKED, defines=("RCP_CHECKED",))


def build_driver(force: bool = False) -> str:
    """The end-to-end driver (e2e_driver.cu): a C++ host program linked against the library, run by bench.py."""
    build()
    src = os.path.join(HERE, "e2e_driver.cu")
    if not force and os.path.exists(DRIVER) and os.path.getmtime(DRIVER) >= max(os.path.getmtime(src), os.path.getmtime(LIB)):
        return DRIVER
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-std=c++17", "-o", DRIVER, src,
                           "-L" + HERE, "-lrcp_w2a4", "-Xlinker", "-rpath", "-Xlinker", "$ORIGIN"])
    return DRIVER


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose=True))
    print(build_driver(force=True))
    if "--checked" in sys.argv[1:]:
        print(build_checked(force=True))
