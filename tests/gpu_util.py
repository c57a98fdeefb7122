"""Helpers for the GPU parity tests: run the CUDA path through the C-ABI, run the oracle,
compare every output element by element (integers: bit-exact)."""
import os

import numpy as np

from oracle import pe_oracle as orc

INVALID = orc.STATUS_ASSIGN_RANGE | orc.STATUS_ORDER_INVALID
CPU_THREADS = max(1, os.cpu_count() or 1)


def as_signed(order):
    """torch has no uint16/uint32 arithmetic; ship the bits as int16/int32."""
    return order.view(np.int16 if order.dtype == np.uint16 else np.int32)


def gpu_eval(graph, assign, order, flags=0, want_times=True):
    import torch
    a = torch.from_numpy(assign).cuda(graph.device)
    o = torch.from_numpy(as_signed(order)).cuda(graph.device)
    out = graph.eval_batch(a, o, flags=flags, want_times=want_times)
    torch.cuda.synchronize(graph.device)
    res = {k: v.cpu().numpy() for k, v in out.items()}
    res["status"] = res["status"].view(np.uint32)
    return res


def compare(gpu, ref, label=""):
    """Bit-exact on every output of every valid candidate; on invalid ones only the two validity bits."""
    bad = (ref["status"] & INVALID) != 0
    assert np.array_equal((gpu["status"] & INVALID) != 0, bad), f"{label}: validity bits differ"
    assert np.array_equal(gpu["status"][bad] & INVALID, ref["status"][bad] & INVALID), f"{label}: validity bits differ"
    ok = ~bad
    assert np.array_equal(gpu["status"][ok], ref["status"][ok]), f"{label}: status"
    for key in ("makespan",):
        assert np.array_equal(gpu[key][ok], ref[key][ok]), f"{label}: {key}"
    for key in ("busy", "peak_mem", "start", "finish"):
        if ref.get(key) is None or key not in gpu:
            continue
        if not np.array_equal(gpu[key][:, ok], ref[key][:, ok]):
            diff = np.argwhere(gpu[key][:, ok] != ref[key][:, ok])
            raise AssertionError(f"{label}: {key} differs at {len(diff)} places, first {diff[:5].tolist()}")


def check(graph, w, assign, order, flags=0, want_times=True, label="", threads=None):
    ref = orc.evaluate(w, assign, order, flags=flags & 7, want_times=want_times, threads=threads or CPU_THREADS)
    gpu = gpu_eval(graph, assign, order, flags=flags, want_times=want_times)
    compare(gpu, ref, label)
    return gpu, ref
