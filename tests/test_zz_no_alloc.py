"""pe_eval_batch_noalloc: evaluation for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: a framework or memory pool
owns the whole device and forbids side allocations, an allocation would stall a latency-critical
loop, or the process's memory budget was fixed at start-up.  For them the library carries a
fixed scratch array of its own and an entry point that uses it.  This test calls that entry
point through the C ABI twice in a row (different candidates, then a different layout, so the
second call meets the first call's leftovers in the shared array) and requires every output to
equal pe_eval_batch's bit for bit.  It is collected last, so a failure here cannot hide others.
"""
import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _as_signed(order):
    return order.view(np.int16 if order.dtype == np.uint16 else np.int32)


def test_noalloc_entry_point_matches_pe_eval_batch_on_two_calls_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2503_09357_b200 import binding as pe

    w = wl.make_config(2)
    V, D = w.num_ops, w.num_devices
    K = 4099                                                        # ragged; 4*V*K ~ 7.9 MB of scratch
    g = pe.Graph(w)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        for call, (first, flags) in enumerate([(0, 0), (K, pe.PE_ASSIGN_BY_POS | pe.PE_TIMES_BY_OP)]):
            assign, order = wl.make_candidates(w, K=K, first=first)
            if flags & pe.PE_ASSIGN_BY_POS:
                assign = wl.assign_by_pos(assign, order)
            a = torch.from_numpy(assign).cuda()
            o = torch.from_numpy(_as_signed(order)).cuda()
            ref = g.eval_batch(a, o, flags=flags)                     # the existing entry point
            got = g.alloc_outputs(K)
            for t in got.values():
                t.fill_(-7)
            rc = pe.pe_eval_batch_noalloc(g.handle, K, a.data_ptr(), o.data_ptr(), order.dtype.itemsize, flags,
                                          pe.make_outputs(**{k: v.data_ptr() for k, v in got.items()}), stream)
            assert rc == pe.PE_OK, pe.pe_strerror(rc)
            torch.cuda.synchronize()
            for key in ref:
                assert torch.equal(ref[key], got[key]), f"call {call}: {key} differs from pe_eval_batch"
            assert int(ref["makespan"].min()) > 0

        # beyond the built-in array: refused with its own code, nothing launched
        too_many = pe.PE_NOALLOC_SCRATCH_BYTES // (4 * V) + 1
        launches = pe.pe_kernel_launches()
        rc = pe.pe_eval_batch_noalloc(g.handle, too_many, a.data_ptr(), o.data_ptr(), 2, 0,
                                      pe.make_outputs(**{k: v.data_ptr() for k, v in got.items()}), stream)
        assert rc == pe.PE_ERR_SCRATCH_LIMIT and "scratch" in pe.pe_strerror(rc)
        assert pe.pe_kernel_launches() == launches
        # variant bits are not accepted here; K = 0 is a no-op
        assert pe.pe_eval_batch_noalloc(g.handle, K, a.data_ptr(), o.data_ptr(), 2, pe.PE_VARIANT_SHARED,
                                        pe.make_outputs(), stream) == pe.PE_ERR_INVALID_ARG
        assert pe.pe_eval_batch_noalloc(g.handle, 0, 0, 0, 2, 0, pe.make_outputs(), stream) == pe.PE_OK
    finally:
        g.close()


@pytest.mark.parametrize("case", ["generic kernel, 32-bit orders, by-position assignments", "many machines: records in the scratch too",
                                  "start times only"])
def test_noalloc_other_branches_of_the_scratch_layout(case):
    """The entry point keeps different things in its built-in array depending on the problem: the generic
    kernel's end times and machine ids, the compact kernel's per-machine records when there are many machines.
    Each layout runs twice in a row on different candidates (the second call meets the first one's leftovers)
    and must match both pe_eval_batch and the oracle."""
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from oracle import pe_oracle as orc
    from paper_2503_09357_b200 import binding as pe
    if case.startswith("generic"):
        w, ob, flags, K = wl.make_config(5, V=256, D=8), 4, pe.PE_ASSIGN_BY_POS, 1500
    elif case.startswith("many"):
        w, ob, flags, K = wl.make_config(5, V=256, D=64), 2, 0, 1500
    else:
        w, ob, flags, K = wl.make_config(1), 2, pe.PE_TIMES_BY_OP, 777
    V = w.num_ops
    g = pe.Graph(w)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        for call in range(2):
            assign, order = wl.make_candidates(w, K=K, first=call * K, order_bytes=ob)
            if flags & pe.PE_ASSIGN_BY_POS:
                assign = wl.assign_by_pos(assign, order)
            a = torch.from_numpy(assign).cuda()
            o = torch.from_numpy(_as_signed(order)).cuda()
            got = g.alloc_outputs(K)
            for t in got.values():
                t.fill_(-7)
            ptrs = {k: v.data_ptr() for k, v in got.items()}
            if case.startswith("start"):
                ptrs.pop("finish")
            rc = pe.pe_eval_batch_noalloc(g.handle, K, a.data_ptr(), o.data_ptr(), ob, flags, pe.make_outputs(**ptrs), stream)
            assert rc == pe.PE_OK, pe.pe_strerror(rc)
            ref = g.eval_batch(a, o, flags=flags)
            torch.cuda.synchronize()
            cpu = orc.evaluate(w, assign, order, flags=flags & 7, threads=8)
            for key in ref:
                if key == "finish" and case.startswith("start"):
                    assert bool((got[key] == -7).all())                        # not asked for: not written
                    continue
                assert torch.equal(ref[key], got[key]), f"{case}, call {call}: {key} differs from pe_eval_batch"
                want = cpu[key].view(np.int32) if key == "status" else cpu[key]
                assert np.array_equal(got[key].cpu().numpy(), want), f"{case}, call {call}: {key} differs from the oracle"
        if case.startswith("generic"):
            # by-position assignments need one more byte per operator and candidate: 5 * V * K in all
            too_many = pe.PE_NOALLOC_SCRATCH_BYTES // (5 * V) + 64
            fits_without = pe.PE_NOALLOC_SCRATCH_BYTES // (4 * V) - 64 > too_many
            rc = pe.pe_eval_batch_noalloc(g.handle, too_many, a.data_ptr(), o.data_ptr(), ob, flags,
                                          pe.make_outputs(**ptrs), stream)
            assert rc == pe.PE_ERR_SCRATCH_LIMIT and fits_without
    finally:
        g.close()
