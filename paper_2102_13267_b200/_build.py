"""Builds liblazytensor.so (host runtime + sm_100a kernels) in-tree with nvcc and g++."""
from __future__ import annotations

import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
OBJ = HERE / "_build"
LIB = HERE / "liblazytensor.so"
CUDA_HOME = Path(os.environ.get("CUDA_HOME", "/usr/local/cuda"))

CU_SOURCES = ["kernels.cu", "compiled.cu", "static_scratch.cu", "reduce.cu", "views.cu"]
CPP_SOURCES = ["engine.cpp", "canon.cpp", "planner.cpp", "executor.cpp", "jit.cpp"]
HEADERS = ["engine.h", "vm.h", "launch.h", "vm_core.inc", "vm_ops.cuh", "compiled.h", "compiled_programs.inc", "pdl.cuh", "compiled_shells.cuh", "jit.h", "../../include/lazytensor.h"]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-diag-suppress", "177",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]
CXX_FLAGS = ["-O2", "-std=c++17", "-fPIC", "-Wall", "-Wno-unused-function", f"-I{CUDA_HOME}/include"]


def _stale(target: Path, deps) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(Path(d).stat().st_mtime > t for d in deps)


PER_SOURCE_FLAGS: dict = {}
EXTRA_NVCC = os.environ.get("LT_NVCC_FLAGS", "").split()  # e.g. -DLT_EW_MIN_BLOCKS=2 for tuning experiments


JIT_TEXTS = [("kSrcVm", "vm.h"), ("kSrcVmOps", "vm_ops.cuh"), ("kSrcPdl", "pdl.cuh"), ("kSrcShells", "compiled_shells.cuh")]


def _embed_sources() -> None:
    """jit_sources.inc (not committed): the text of the device headers, for the run-time specialiser to compile."""
    out = OBJ / "jit_sources.inc"
    deps = [CSRC / f for _, f in JIT_TEXTS]
    if not _stale(out, deps):
        return
    parts = []
    for name, f in JIT_TEXTS:
        text = (CSRC / f).read_text()
        assert ')LTSRC"' not in text
        # (string literals are limited to 64 KB pieces by some compilers: split at line ends)
        pieces, cur = [], ""
        for line in text.splitlines(keepends=True):
            if len(cur) + len(line) > 60000:
                pieces.append(cur)
                cur = ""
            cur += line
        pieces.append(cur)
        parts.append(f"const char {name}[] =\n" + "\n".join(f'R"LTSRC({p})LTSRC"' for p in pieces) + ";\n")
    out.write_text("".join(parts))


def _compile(src: str) -> Path:
    path = CSRC / src
    obj = OBJ / (src + ".o")
    deps = [path] + [CSRC / h for h in HEADERS]
    if _stale(obj, deps):
        if src.endswith(".cu"):
            cmd = [str(CUDA_HOME / "bin" / "nvcc"), *NVCC_FLAGS, *PER_SOURCE_FLAGS.get(src, []), *EXTRA_NVCC, "-c", str(path), "-o", str(obj)]
        else:
            cmd = ["g++", *CXX_FLAGS, f"-I{OBJ}", "-c", str(path), "-o", str(obj)]
        subprocess.check_call(cmd)
    return obj


def build(force: bool = False) -> Path:
    """Compile what changed and link the shared library; returns its path."""
    OBJ.mkdir(exist_ok=True)
    if force:
        for f in OBJ.glob("*.o"):
            f.unlink()
    _embed_sources()
    with ThreadPoolExecutor(max_workers=4) as pool:
        objs = list(pool.map(_compile, CU_SOURCES + CPP_SOURCES))
    if force or _stale(LIB, objs):
        tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call([str(CUDA_HOME / "bin" / "nvcc"), "-shared", "-o", str(tmp), *map(str, objs),
                               "-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static", "-ldl", "-lpthread"])
        os.replace(tmp, LIB)
    return LIB


def build_host_bench() -> Path:
    """Compile csrc/host_bench.cpp (host cost of record / flush / replay through the C ABI, no Python) against the library."""
    exe = HERE / "lt_host_bench"
    src = CSRC / "host_bench.cpp"
    if _stale(exe, [src, LIB]):
        subprocess.check_call(["g++", "-O2", "-std=c++17", f"-I{HERE.parent / 'include'}", str(src), f"-L{HERE}", "-llazytensor",
                               f"-Wl,-rpath,{HERE}", "-o", str(exe)])
    return exe


if __name__ == "__main__":
    print(build())
