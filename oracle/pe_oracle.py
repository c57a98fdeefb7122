"""ctypes loader for the CPU oracle in pe_oracle.cpp.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does.  `evaluate` marshals numpy arrays and, when
asked for several threads, splits the candidate range statically; the arithmetic
is all in the C++ file.
"""
import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pe_oracle.cpp")
_LIB = os.path.join(_HERE, "libpe_oracle.so")
_lib = None

ASSIGN_BY_POS = 1
TIMES_BY_OP = 2
COMM_EXCLUSIVE = 4

STATUS_ASSIGN_RANGE = 1
STATUS_ORDER_INVALID = 2
STATUS_MEM_EXCEEDED = 4
STATUS_NO_CHANNEL = 8


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", _SRC, "-o", _LIB])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        lib.pe_oracle_eval.restype = ctypes.c_int
        lib.pe_oracle_eval.argtypes = [ctypes.c_int32, ctypes.c_int32, P, P, P, P, P, ctypes.c_int32, ctypes.c_int32,
                                       P, P, P, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, P, P, ctypes.c_int,
                                       ctypes.c_uint32, P, P, P, P, P, P]
        lib.pe_oracle_eval_hetero.restype = ctypes.c_int
        lib.pe_oracle_eval_hetero.argtypes = [ctypes.c_int32, ctypes.c_int32, P, P, P, P, P, P, ctypes.c_int32,
                                              ctypes.c_int32, P, P, P, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                              P, P, ctypes.c_int, ctypes.c_uint32, P, P, P, P, P, P]
        lib.pe_oracle_decode.restype = ctypes.c_int
        lib.pe_oracle_decode.argtypes = [ctypes.c_int32, ctypes.c_int32, P, P, ctypes.c_int64, ctypes.c_int64,
                                         ctypes.c_int64, P, ctypes.c_int, P, P]
        _lib = lib
    return _lib


def _p(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def _c(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def evaluate(w, assign, order, flags=0, want_times=True, threads=1, c_range=None):
    """Evaluate candidates of workload-like object `w` (fields as in workloads.Workload).

    assign: u8 [V, K]; order: u16/u32 [V, K].  Returns a dict of numpy arrays:
    start, finish [V, K] (None unless want_times), makespan [K], busy [D, K],
    peak_mem [D, K], status [K].  With `c_range=(b, e)` only those columns are filled.
    """
    V, D, L = int(w.num_ops), int(w.num_devices), int(w.num_link_classes)
    assign = np.ascontiguousarray(assign, dtype=np.uint8)
    order = np.ascontiguousarray(order)
    assert order.dtype in (np.uint16, np.uint32)
    K = assign.shape[1]
    assert assign.shape == (V, K) and order.shape == (V, K)
    src, dst = _c(w.edge_src, np.int32), _c(w.edge_dst, np.int32)
    dur, A, W = _c(w.dur, np.int32), _c(w.mem_delta, np.int32), _c(w.mem_weight, np.int32)
    cls, comm, cap = _c(w.link_class, np.uint8), _c(w.comm, np.int32), _c(w.mem_capacity, np.int32)
    durm = _c(getattr(w, "dur_by_machine", None), np.int32)      # [V, D]: heterogeneous machines (Section III, footnote)
    assert durm is None or durm.shape == (V, D)
    E = int(src.shape[0])
    out = dict(
        start=np.zeros((V, K), np.int32) if want_times else None,
        finish=np.zeros((V, K), np.int32) if want_times else None,
        makespan=np.zeros(K, np.int32), busy=np.zeros((D, K), np.int32),
        peak_mem=np.zeros((D, K), np.int32), status=np.zeros(K, np.uint32))
    lib = _load()
    b, e = (0, K) if c_range is None else c_range

    def run(lo, hi):
        rc = lib.pe_oracle_eval_hetero(V, E, _p(src), _p(dst), _p(dur), _p(durm), _p(A), _p(W), D, L, _p(cls), _p(comm),
                                       _p(cap), K, lo, hi, _p(assign), _p(order), order.dtype.itemsize, flags,
                                       _p(out["start"]), _p(out["finish"]), _p(out["makespan"]), _p(out["busy"]),
                                       _p(out["peak_mem"]), _p(out["status"]))
        if rc != 0:
            raise RuntimeError(f"pe_oracle_eval failed with code {rc}")

    threads = max(1, min(int(threads), e - b)) if e > b else 1
    if threads == 1:
        run(b, e)
    else:
        cuts = [b + (e - b) * t // threads for t in range(threads + 1)]
        with ThreadPoolExecutor(threads) as pool:
            list(pool.map(lambda t: run(cuts[t], cuts[t + 1]), range(threads)))
    return out


def select_best(makespan, status, reject_mask=0xFFFFFFFF):
    """The selection step written out: among candidates whose status has none of the `reject_mask`
    bits, the smallest makespan (Eq. 1), ties to the smallest index.  Returns (index or -1,
    makespan or INT32_MAX, number of qualifying candidates)."""
    best, best_c, count = 2 ** 31 - 1, -1, 0
    for c in range(len(makespan)):
        if int(status[c]) & reject_mask:
            continue
        count += 1
        if best_c < 0 or int(makespan[c]) < best:
            best, best_c = int(makespan[c]), c
    return best_c, best, count


def select_topk(makespan, status, k, reject_mask=0xFFFFFFFF):
    """The k best candidates written out (Eq. 1: smaller makespan is better; Section III: a candidate whose
    status has a `reject_mask` bit is not a valid arrangement): repeatedly take, among the qualifying
    candidates not yet taken, the one with the smallest makespan, ties to the smallest index.  Returns the
    chosen indices in INCREASING INDEX order (the selection is a set; at most k, fewer if fewer qualify)."""
    taken = []
    for _ in range(int(k)):
        best_c = -1
        for c in range(len(makespan)):
            if (int(status[c]) & reject_mask) or c in taken:
                continue
            if best_c < 0 or int(makespan[c]) < int(makespan[best_c]):
                best_c = c
        if best_c < 0:
            break
        taken.append(best_c)
    return sorted(taken)


def decode(w, plist, threads=1):
    """Priority-list decoding (see pe_oracle.cpp): plist is u16/u32 [V, K], plist[r, c] = the operation of
    rank r of candidate c.  Returns (order [V, K] of the same dtype, status [K] uint32)."""
    V = int(w.num_ops)
    plist = np.ascontiguousarray(plist)
    assert plist.dtype in (np.uint16, np.uint32) and plist.shape[0] == V
    K = plist.shape[1]
    src, dst = _c(w.edge_src, np.int32), _c(w.edge_dst, np.int32)
    order = np.zeros_like(plist)
    status = np.zeros(K, np.uint32)
    lib = _load()

    def run(lo, hi):
        rc = lib.pe_oracle_decode(V, int(src.shape[0]), _p(src), _p(dst), K, lo, hi, _p(plist), plist.dtype.itemsize,
                                  _p(order), _p(status))
        if rc != 0:
            raise RuntimeError(f"pe_oracle_decode failed with code {rc}")

    threads = max(1, min(int(threads), K)) if K > 0 else 1
    if threads == 1:
        run(0, K)
    else:
        cuts = [K * t // threads for t in range(threads + 1)]
        with ThreadPoolExecutor(threads) as pool:
            list(pool.map(lambda t: run(cuts[t], cuts[t + 1]), range(threads)))
    return order, status
