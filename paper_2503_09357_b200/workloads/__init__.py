"""Seeded synthetic workloads: operator DAGs, clusters and candidate plans.

This module only draws inputs.  It holds none of the evaluation arithmetic and is
the one piece shared by the CUDA path's tests/benchmarks and the CPU checker.
"""
import ctypes
import os
import subprocess

import numpy as np

from .graphs import (DEFAULT_SEED, SWEEP_POINTS, Workload, bidirectional_pipeline, make_config, moe_branchy,
                     multimodal_mimo, random_layered, tiny_pipeline)

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpegen.so")
_SRC_PATH = os.path.join(_HERE, "candgen.cpp")
_lib = None


def build_generator(force: bool = False) -> str:
    """Compile candgen.cpp into libpegen.so next to it (host code only, g++)."""
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC_PATH):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", _SRC_PATH, "-o", _LIB_PATH])
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_generator())
        P = ctypes.c_void_p
        lib.pegen_candidates.restype = ctypes.c_int
        lib.pegen_candidates.argtypes = [ctypes.c_int32, ctypes.c_int32, P, P, ctypes.c_int32, ctypes.c_int, P,
                                         ctypes.c_int32, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int64, P, P,
                                         ctypes.c_int, ctypes.c_int]
        lib.pegen_assign_by_pos.restype = ctypes.c_int
        lib.pegen_assign_by_pos.argtypes = [ctypes.c_int32, ctypes.c_int64, P, P, ctypes.c_int, P, ctypes.c_int]
        _lib = lib
    return _lib


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def order_dtype(num_ops: int):
    """Order entries are u16 while every op id fits (V <= 65536), else u32."""
    return np.uint16 if num_ops <= 65536 else np.uint32


def make_candidates(w: Workload, K: int = None, seed: int = DEFAULT_SEED, first: int = 0, threads: int = 0,
                    out_assign: np.ndarray = None, out_order: np.ndarray = None, order_bytes: int = None):
    """Candidates first .. first+K-1 of workload `w`.

    Returns (assign, order): `assign` is u8 [V, K] by operator (x_c[i] at [i, c]) and
    `order` is u16/u32 [V, K] by position (pi_c[k] at [k, c]).  Output arrays may be
    supplied (e.g. views of pinned memory) and are then filled in place.
    """
    K = w.num_candidates if K is None else int(K)
    V = w.num_ops
    odt = order_dtype(V) if order_bytes is None else {2: np.uint16, 4: np.uint32}[order_bytes]
    assign = np.empty((V, K), dtype=np.uint8) if out_assign is None else out_assign
    order = np.empty((V, K), dtype=odt) if out_order is None else out_order
    assert assign.shape == (V, K) and assign.dtype == np.uint8 and assign.flags.c_contiguous
    assert order.shape == (V, K) and order.dtype == odt and order.flags.c_contiguous
    mode = {"per_op": 0, "group_perm": 1}[w.assign_mode]
    group = np.ascontiguousarray(w.group, dtype=np.int32) if w.group is not None else None
    ngroups = int(group.max()) + 1 if group is not None else 0
    if mode == 1 and ngroups > w.num_devices:
        raise ValueError("group_perm needs at most one group per device")
    rc = _load().pegen_candidates(V, w.num_edges, _ptr(w.edge_src), _ptr(w.edge_dst), w.num_devices, mode,
                                  _ptr(group), ngroups, seed, K, first, _ptr(assign), _ptr(order),
                                  order.dtype.itemsize, threads)
    if rc != 0:
        raise RuntimeError(f"pegen_candidates failed with code {rc}")
    return assign, order


def assign_by_pos(assign: np.ndarray, order: np.ndarray, out: np.ndarray = None, threads: int = 0) -> np.ndarray:
    """dev_seq[k, c] = assign[order[k, c], c] (the by-position view of the same assignment)."""
    V, K = assign.shape
    out = np.empty((V, K), dtype=np.uint8) if out is None else out
    rc = _load().pegen_assign_by_pos(V, K, _ptr(assign), _ptr(order), order.dtype.itemsize, _ptr(out), threads)
    if rc != 0:
        raise RuntimeError(f"pegen_assign_by_pos failed with code {rc}")
    return out
