"""ctypes binding of libpe.so: the same entry points as include/pe.h, argument marshalling only.

Every step of the evaluation runs in the library's CUDA kernels; nothing here computes.
PyTorch is used by :class:`Graph` helpers for device memory and the current stream.
Importing this module fails if the library has not been built (see build.py): there is no
CPU fallback.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpe.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_09357_b200.build` "
                      "(nvcc, sm_100a). There is no fallback path.")
_lib = ctypes.CDLL(LIB_PATH)

# ---- constants of pe.h ----
PE_OK = 0
PE_ERR_INVALID_ARG, PE_ERR_CYCLE, PE_ERR_RANGE, PE_ERR_OVERFLOW = -1, -2, -3, -4
PE_ERR_CUDA, PE_ERR_WORKSPACE, PE_ERR_TIMEOUT, PE_ERR_UNSUPPORTED = -5, -6, -7, -8
PE_ERR_SCRATCH_LIMIT = -9
PE_NOALLOC_SCRATCH_BYTES = 64 << 20
PE_ASSIGN_BY_POS, PE_TIMES_BY_OP, PE_COMM_EXCLUSIVE = 1, 2, 4
PE_VARIANT_AUTO, PE_VARIANT_GLOBAL, PE_VARIANT_SHARED, PE_VARIANT_WARP = 0 << 8, 1 << 8, 2 << 8, 3 << 8
PE_VARIANT_TEAM = 4 << 8
PE_VARIANT_MASK = 15 << 8
PE_STATUS_ASSIGN_RANGE, PE_STATUS_ORDER_INVALID, PE_STATUS_MEM_EXCEEDED, PE_STATUS_NO_CHANNEL = 1, 2, 4, 8
VARIANT_NAMES = {PE_VARIANT_GLOBAL: "global", PE_VARIANT_SHARED: "shared", PE_VARIANT_WARP: "warp", PE_VARIANT_TEAM: "team"}

_P = ctypes.c_void_p


class pe_graph_desc(ctypes.Structure):
    _fields_ = [("num_ops", ctypes.c_int32), ("num_edges", ctypes.c_int32), ("edge_src", _P), ("edge_dst", _P),
                ("dur", _P), ("mem_delta", _P), ("mem_weight", _P), ("num_devices", ctypes.c_int32),
                ("num_link_classes", ctypes.c_int32), ("link_class", _P), ("comm", _P), ("mem_capacity", _P),
                ("dur_by_machine", _P)]


class pe_outputs(ctypes.Structure):
    _fields_ = [("start", _P), ("finish", _P), ("makespan", _P), ("busy", _P), ("peak_mem", _P), ("status", _P)]


_lib.pe_graph_validate.restype = ctypes.c_int
_lib.pe_graph_validate.argtypes = [ctypes.POINTER(pe_graph_desc)]
_lib.pe_graph_create.restype = ctypes.c_int
_lib.pe_graph_create.argtypes = [ctypes.POINTER(pe_graph_desc), ctypes.c_int, ctypes.POINTER(_P)]
_lib.pe_destroy.restype = ctypes.c_int
_lib.pe_destroy.argtypes = [_P]
_lib.pe_workspace_bytes.restype = ctypes.c_size_t
_lib.pe_workspace_bytes.argtypes = [_P, ctypes.c_int64, ctypes.c_uint32]
_lib.pe_eval_variant.restype = ctypes.c_int
_lib.pe_eval_variant.argtypes = [_P, ctypes.c_int64, ctypes.c_uint32]
_lib.pe_eval_batch.restype = ctypes.c_int
_lib.pe_eval_batch.argtypes = [_P, ctypes.c_int64, _P, _P, ctypes.c_int, ctypes.c_uint32, ctypes.POINTER(pe_outputs),
                               _P, ctypes.c_size_t, _P]
_lib.pe_eval_batch_host.restype = ctypes.c_int
_lib.pe_eval_batch_host.argtypes = [_P, ctypes.c_int64, _P, _P, ctypes.c_int, ctypes.c_uint32,
                                    ctypes.POINTER(pe_outputs), _P, _P, ctypes.POINTER(pe_outputs), _P,
                                    ctypes.c_size_t, _P]
_lib.pe_eval_batch_noalloc.restype = ctypes.c_int
_lib.pe_eval_batch_noalloc.argtypes = [_P, ctypes.c_int64, _P, _P, ctypes.c_int, ctypes.c_uint32,
                                       ctypes.POINTER(pe_outputs), _P]
_lib.pe_decode_workspace_bytes.restype = ctypes.c_size_t
_lib.pe_decode_workspace_bytes.argtypes = [_P, ctypes.c_int64, ctypes.c_uint32]
_lib.pe_decode_variant.restype = ctypes.c_int
_lib.pe_decode_variant.argtypes = [_P, ctypes.c_int64, ctypes.c_uint32]
_lib.pe_decode_priority.restype = ctypes.c_int
_lib.pe_decode_priority.argtypes = [_P, ctypes.c_int64, _P, ctypes.c_int, ctypes.c_uint32, _P, _P, _P, ctypes.c_size_t, _P]
_lib.pe_select_best.restype = ctypes.c_int
_lib.pe_select_best.argtypes = [ctypes.c_int64, _P, _P, ctypes.c_uint32, _P, _P]
_lib.pe_select_topk_workspace_bytes.restype = ctypes.c_size_t
_lib.pe_select_topk_workspace_bytes.argtypes = [ctypes.c_int64]
_lib.pe_select_topk.restype = ctypes.c_int
_lib.pe_select_topk.argtypes = [ctypes.c_int64, _P, _P, ctypes.c_uint32, ctypes.c_int32, _P, _P, _P, ctypes.c_size_t, _P]
_lib.pe_graph_poll_error.restype = ctypes.c_int
_lib.pe_graph_poll_error.argtypes = [_P, _P]
_lib.pe_selftest_wait_timeout.restype = ctypes.c_int
_lib.pe_selftest_wait_timeout.argtypes = [_P, _P]
_lib.pe_kernel_launches.restype = ctypes.c_int64
_lib.pe_kernel_launches.argtypes = []
_lib.pe_strerror.restype = ctypes.c_char_p
_lib.pe_strerror.argtypes = [ctypes.c_int]


class pe_coarsen_params(ctypes.Structure):
    _fields_ = [("target_ops", ctypes.c_int32), ("max_dur_edge", ctypes.c_int32), ("max_mem_edge", ctypes.c_int32),
                ("max_dur_nonedge", ctypes.c_int32), ("max_mem_nonedge", ctypes.c_int32)]


_lib.pe_coarsen.restype = ctypes.c_int
_lib.pe_coarsen.argtypes = [ctypes.POINTER(pe_graph_desc), ctypes.POINTER(pe_coarsen_params)] + [_P] * 9


class PeError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {pe_strerror(code)} ({code})")


def pe_strerror(code: int) -> str:
    return _lib.pe_strerror(int(code)).decode()


def _np_ptr(a, dtype):
    """Host pointer of a numpy array (made contiguous with the ABI's dtype); returns (ptr, keepalive)."""
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=dtype)
    return a.ctypes.data, a


def make_desc(num_ops, edge_src, edge_dst, dur, num_devices, mem_delta=None, mem_weight=None, num_link_classes=1,
              link_class=None, comm=None, mem_capacity=None, dur_by_machine=None):
    """Fill a pe_graph_desc from numpy arrays; returns (desc, keepalive list)."""
    keep = []
    d = pe_graph_desc()
    d.num_ops = int(num_ops)
    d.num_edges = 0 if edge_src is None else int(np.asarray(edge_src).shape[0])
    d.num_devices = int(num_devices)
    d.num_link_classes = int(num_link_classes)
    for name, arr, dt in (("edge_src", edge_src, np.int32), ("edge_dst", edge_dst, np.int32), ("dur", dur, np.int32),
                          ("mem_delta", mem_delta, np.int32), ("mem_weight", mem_weight, np.int32),
                          ("link_class", link_class, np.uint8), ("comm", comm, np.int32),
                          ("mem_capacity", mem_capacity, np.int32), ("dur_by_machine", dur_by_machine, np.int32)):
        ptr, ka = _np_ptr(arr, dt)
        setattr(d, name, ptr)
        keep.append(ka)
    return d, keep


def desc_from_workload(w):
    return make_desc(w.num_ops, w.edge_src, w.edge_dst, w.dur, w.num_devices, mem_delta=w.mem_delta,
                     mem_weight=w.mem_weight, num_link_classes=w.num_link_classes, link_class=w.link_class,
                     comm=w.comm, mem_capacity=w.mem_capacity, dur_by_machine=getattr(w, "dur_by_machine", None))


def pe_coarsen(desc, target_ops, max_dur_edge, max_mem_edge, max_dur_nonedge, max_mem_nonedge):
    """Algorithm 1 on a host description (argument marshalling only).  Returns a dict of numpy arrays
    (op_map, edge_src, edge_dst, comm [E', L], dur, mem_delta, mem_weight) and num_ops."""
    V, E, L = int(desc.num_ops), int(desc.num_edges), int(desc.num_link_classes)
    prm = pe_coarsen_params(int(target_ops), int(max_dur_edge), int(max_mem_edge), int(max_dur_nonedge),
                            int(max_mem_nonedge))
    op_map = np.zeros(max(V, 1), np.int32)
    n_ops, n_edges = ctypes.c_int32(0), ctypes.c_int32(0)
    src, dst = np.zeros(max(E, 1), np.int32), np.zeros(max(E, 1), np.int32)
    comm = np.zeros(max(E * L, 1), np.int32)
    dur, A, W = (np.zeros(max(V, 1), np.int32) for _ in range(3))
    rc = _lib.pe_coarsen(ctypes.byref(desc), ctypes.byref(prm), op_map.ctypes.data, ctypes.addressof(n_ops),
                         ctypes.addressof(n_edges), src.ctypes.data, dst.ctypes.data, comm.ctypes.data,
                         dur.ctypes.data, A.ctypes.data, W.ctypes.data)
    if rc != PE_OK:
        raise PeError(rc, "pe_coarsen")
    n, m = n_ops.value, n_edges.value
    return dict(num_ops=n, op_map=op_map[:V], edge_src=src[:m], edge_dst=dst[:m], comm=comm[:m * L].reshape(m, L),
                dur=dur[:n], mem_delta=A[:n], mem_weight=W[:n])


def pe_graph_validate(desc) -> int:
    return _lib.pe_graph_validate(ctypes.byref(desc))


def pe_graph_create(desc, cuda_device: int = 0):
    """Returns the opaque handle (an int address); raises PeError on failure."""
    h = _P()
    rc = _lib.pe_graph_create(ctypes.byref(desc), int(cuda_device), ctypes.byref(h))
    if rc != PE_OK:
        raise PeError(rc, "pe_graph_create")
    return h.value


def pe_destroy(handle) -> int:
    return _lib.pe_destroy(handle)


def pe_workspace_bytes(handle, K: int, flags: int = 0) -> int:
    return int(_lib.pe_workspace_bytes(handle, int(K), int(flags)))


def pe_eval_variant(handle, K: int, flags: int = 0) -> int:
    return int(_lib.pe_eval_variant(handle, int(K), int(flags)))


def make_outputs(start=0, finish=0, makespan=0, busy=0, peak_mem=0, status=0):
    o = pe_outputs()
    o.start, o.finish, o.makespan = start or None, finish or None, makespan or None
    o.busy, o.peak_mem, o.status = busy or None, peak_mem or None, status or None
    return o


def pe_eval_batch(handle, K, assign_ptr, order_ptr, order_bytes, flags, outputs, workspace_ptr=0, workspace_bytes=0,
                  stream=0) -> int:
    """Raw call: device pointers as ints. Returns the library's code (0 = ok)."""
    return _lib.pe_eval_batch(handle, int(K), assign_ptr or None, order_ptr or None, int(order_bytes), int(flags),
                              ctypes.byref(outputs), workspace_ptr or None, int(workspace_bytes), stream or None)


def pe_eval_batch_host(handle, K, host_assign_ptr, host_order_ptr, order_bytes, flags, host_outputs, dev_assign_ptr,
                       dev_order_ptr, dev_outputs, workspace_ptr=0, workspace_bytes=0, stream=0) -> int:
    return _lib.pe_eval_batch_host(handle, int(K), host_assign_ptr, host_order_ptr, int(order_bytes), int(flags),
                                   ctypes.byref(host_outputs), dev_assign_ptr, dev_order_ptr, ctypes.byref(dev_outputs),
                                   workspace_ptr or None, int(workspace_bytes), stream or None)


def pe_eval_batch_noalloc(handle, K, assign_ptr, order_ptr, order_bytes, flags, outputs, stream=0) -> int:
    """Raw call of the entry point that brings its own scratch (for callers that cannot allocate
    device memory); same pointer conventions as pe_eval_batch, no workspace argument."""
    return _lib.pe_eval_batch_noalloc(handle, int(K), assign_ptr or None, order_ptr or None, int(order_bytes),
                                      int(flags), ctypes.byref(outputs), stream or None)


def pe_select_best(K, makespan_ptr, status_ptr, reject_mask, result_ptr, stream=0) -> int:
    """Raw call: arg-min of the makespan over the candidates whose status passes the mask (device pointers)."""
    return _lib.pe_select_best(int(K), makespan_ptr or None, status_ptr or None, int(reject_mask) & 0xFFFFFFFF,
                               result_ptr, stream or None)


def pe_select_topk_workspace_bytes(K: int) -> int:
    return int(_lib.pe_select_topk_workspace_bytes(int(K)))


def pe_select_topk(K, makespan_ptr, status_ptr, reject_mask, k, out_index_ptr, out_count_ptr, workspace_ptr,
                   workspace_bytes, stream=0) -> int:
    return _lib.pe_select_topk(int(K), makespan_ptr, status_ptr, int(reject_mask) & 0xFFFFFFFF, int(k), out_index_ptr,
                               out_count_ptr, workspace_ptr, int(workspace_bytes), stream)


def pe_decode_workspace_bytes(handle, K: int, flags: int = 0) -> int:
    return int(_lib.pe_decode_workspace_bytes(handle, int(K), int(flags)))


def pe_decode_variant(handle, K: int, flags: int = 0) -> int:
    return int(_lib.pe_decode_variant(handle, int(K), int(flags)))


def pe_decode_priority(handle, K, list_ptr, order_bytes, flags, order_ptr, status_ptr=0, workspace=0, workspace_bytes=0,
                       stream=0) -> int:
    """Raw call: priority lists -> topological priority orders (device pointers)."""
    return _lib.pe_decode_priority(handle, int(K), list_ptr or None, int(order_bytes), int(flags), order_ptr or None,
                                   status_ptr or None, workspace or None, int(workspace_bytes), stream or None)


def pe_graph_poll_error(handle, stream=0) -> int:
    return _lib.pe_graph_poll_error(handle, stream or None)


def pe_selftest_wait_timeout(handle, stream=0) -> int:
    return _lib.pe_selftest_wait_timeout(handle, stream or None)


def pe_kernel_launches() -> int:
    return int(_lib.pe_kernel_launches())


class Graph:
    """Owner of a pe_graph handle with torch-tensor conveniences (allocation and pointers only)."""

    def __init__(self, workload, device: int = 0):
        desc, self._keep = desc_from_workload(workload)
        self.V, self.D = int(workload.num_ops), int(workload.num_devices)
        self.device = int(device)
        self.handle = pe_graph_create(desc, device)

    def close(self):
        if getattr(self, "handle", None):
            _lib.pe_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:   # interpreter shutdown: the library may already be gone
            pass

    def variant(self, K, flags=0) -> str:
        v = pe_eval_variant(self.handle, K, flags)
        if v < 0:
            raise PeError(v, "pe_eval_variant")
        return VARIANT_NAMES[v]

    def alloc_outputs(self, K, want_times=True):
        import torch
        dev = torch.device("cuda", self.device)
        out = dict(makespan=torch.empty(K, dtype=torch.int32, device=dev),
                   busy=torch.empty((self.D, K), dtype=torch.int32, device=dev),
                   peak_mem=torch.empty((self.D, K), dtype=torch.int32, device=dev),
                   status=torch.empty(K, dtype=torch.int32, device=dev))
        if want_times:
            out["start"] = torch.empty((self.V, K), dtype=torch.int32, device=dev)
            out["finish"] = torch.empty((self.V, K), dtype=torch.int32, device=dev)
        return out

    def alloc_workspace(self, K, flags=0):
        import torch
        n = pe_workspace_bytes(self.handle, K, flags)
        return torch.empty(max(n, 256), dtype=torch.uint8, device=torch.device("cuda", self.device)), n

    def select_best(self, out, reject_mask=0xFFFFFFFF, stream=None):
        """Index, makespan and count of the best qualifying candidate of an eval_batch result (host ints)."""
        import torch
        res = torch.empty(4, dtype=torch.int64, device=out["makespan"].device)
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        rc = pe_select_best(out["makespan"].numel(), out["makespan"].data_ptr(), out["status"].data_ptr(), reject_mask,
                            res.data_ptr(), s)
        if rc != PE_OK:
            raise PeError(rc, "pe_select_best")
        idx, mk, cnt, _ = res.tolist()
        return idx, mk, cnt

    def select_topk(self, out, k, reject_mask=0xFFFFFFFF, stream=None):
        """The k best qualifying candidates of an eval_batch result: (indices int32 [k] on the device, listed by
        increasing candidate index and padded with -1; count, a one-element int32 device tensor).  Asynchronous."""
        import torch
        K = out["makespan"].numel()
        dev = out["makespan"].device
        idx = torch.empty(max(int(k), 1), dtype=torch.int32, device=dev)
        cnt = torch.empty(1, dtype=torch.int32, device=dev)
        n = pe_select_topk_workspace_bytes(K)
        ws = torch.empty(n, dtype=torch.uint8, device=dev)
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        rc = pe_select_topk(K, out["makespan"].data_ptr(), out["status"].data_ptr(), reject_mask, k, idx.data_ptr(),
                            cnt.data_ptr(), ws.data_ptr(), n, s)
        if rc != PE_OK:
            raise PeError(rc, "pe_select_topk")
        if stream is not None:
            ws.record_stream(torch.cuda.ExternalStream(stream, device=dev))
        return idx[:int(k)], cnt

    def decode_priority(self, plist, flags=0, stream=None):
        """plist: cuda int16 [V, K] holding u16 operator ids, plist[r, c] = operator of rank r of candidate c.
        Returns (order, status): the topological priority orders (same shape and dtype) and a uint32-bit
        status per candidate (int32 tensor).  Asynchronous on `stream` (default: torch's current stream)."""
        import torch
        K = int(plist.shape[1])
        assert plist.is_cuda and plist.is_contiguous() and tuple(plist.shape) == (self.V, K) and plist.element_size() == 2
        dev = torch.device("cuda", self.device)
        order = torch.empty_like(plist)
        status = torch.empty(K, dtype=torch.int32, device=dev)
        n = pe_decode_workspace_bytes(self.handle, K, flags)
        ws = torch.empty(max(n, 256), dtype=torch.uint8, device=dev)
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        rc = pe_decode_priority(self.handle, K, plist.data_ptr(), 2, flags, order.data_ptr(), status.data_ptr(),
                                ws.data_ptr(), n, s)
        if rc != PE_OK:
            raise PeError(rc, "pe_decode_priority")
        if stream is not None:        # the workspace dies here: keep the allocator from reusing it under the kernel
            ws.record_stream(torch.cuda.ExternalStream(stream, device=dev))
        return order, status

    def eval_batch(self, assign, order, flags=0, out=None, workspace=None, want_times=True, stream=None):
        """assign: cuda uint8 [V, K]; order: cuda int16/int32 [V, K] holding u16/u32 bits.
        Launches on `stream` (default: torch's current stream); asynchronous. Returns the dict of output tensors."""
        import torch
        K = int(assign.shape[1])
        assert assign.is_cuda and order.is_cuda and assign.is_contiguous() and order.is_contiguous()
        assert tuple(assign.shape) == (self.V, K) and tuple(order.shape) == (self.V, K)
        if out is None:
            out = self.alloc_outputs(K, want_times)
        if workspace is None:
            workspace = self.alloc_workspace(K, flags)
        ws, ws_bytes = workspace
        o = make_outputs(**{k: v.data_ptr() for k, v in out.items()})
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        rc = pe_eval_batch(self.handle, K, assign.data_ptr(), order.data_ptr(), order.element_size(), flags, o,
                           ws.data_ptr(), ws_bytes, s)
        if rc != PE_OK:
            raise PeError(rc, "pe_eval_batch")
        if stream is not None:        # a workspace allocated here dies here: keep the allocator from reusing it
            ws.record_stream(torch.cuda.ExternalStream(stream, device=torch.device("cuda", self.device)))
        return out
