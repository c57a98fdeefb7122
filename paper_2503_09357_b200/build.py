"""Build the native pieces in-tree: libpe.so (CUDA, sm_100a) and the workload generator."""
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libpe.so")
SOURCES = ["pe_graph.cu", "pe_eval.cu", "pe_lane.cu", "pe_lane_op.cu", "pe_lane_pos.cu", "pe_warp2.cu", "pe_warp2_op.cu", "pe_warp2_pos.cu", "pe_team.cu", "pe_team_nw2.cu", "pe_team_nw4.cu", "pe_team_nw6.cu", "pe_select.cu", "pe_decode.cu", "pe_coarsen.cu"]
OBJ_DIR = os.path.join(_HERE, "_build")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--compiler-options", "-fPIC", "-cudart", "shared"]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_libpe(force: bool = False, verbose: bool = False, extra_flags=()) -> str:
    """Compile every .cu of csrc/ to an object (in parallel) and link them into libpe.so."""
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(_ROOT, "include", "pe.h"))
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    jobs, objs = [], []
    for name in SOURCES:
        src = os.path.join(CSRC, name)
        obj = os.path.join(OBJ_DIR, name.replace(".cu", ".o"))
        objs.append(obj)
        if force or _stale(obj, [src] + headers):
            cmd = [nvcc] + NVCC_FLAGS + list(extra_flags) + ["-I", os.path.join(_ROOT, "include"), "-I", CSRC,
                                                              "-c", src, "-o", obj]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
                print(" ".join(cmd))
            jobs.append((name, subprocess.Popen(cmd)))
    failed = [name for name, proc in jobs if proc.wait() != 0]
    if failed:
        raise RuntimeError(f"nvcc failed for {failed}")
    if jobs or force or _stale(LIB, objs):
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "shared"] + objs + ["-o", LIB])
    return LIB


def build_all(force: bool = False, verbose: bool = False) -> None:
    build_libpe(force=force, verbose=verbose)
    from .workloads import build_generator
    build_generator(force=force)


if __name__ == "__main__":
    build_all(force="--force" in sys.argv, verbose="-v" in sys.argv)
