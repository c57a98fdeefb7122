"""Parity of the CUDA path (through the C-ABI) with the CPU oracle: bit-exact on every output."""
import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl
from tests import checkers as ck
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pe():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2503_09357_b200 import binding
    return binding


def variants_for(pe, graph, K, base_flags=0):
    out = [("auto", base_flags)]
    for name, bit in (("global", pe.PE_VARIANT_GLOBAL), ("shared", pe.PE_VARIANT_SHARED), ("warp", pe.PE_VARIANT_WARP),
                      ("team", pe.PE_VARIANT_TEAM)):
        if pe.pe_eval_variant(graph.handle, K, base_flags | bit) >= 0:
            out.append((name, base_flags | bit))
    return out


# ---- the five configurations; 1-4 at full K, the sweep at K*V = 2^23 ----
CASES = [(1, {}, None), (2, {}, None), (3, {}, None), (4, {}, None)] + \
        [(5, dict(V=V, D=D), (1 << 23) // V) for V, D in wl.SWEEP_POINTS]


@pytest.mark.parametrize("config,kw,K", CASES, ids=lambda v: str(v).replace(" ", ""))
def test_configs_match_oracle(pe, config, kw, K):
    w = wl.make_config(config, **kw)
    K = w.num_candidates if K is None else K
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        seen = set()
        for name, flags in variants_for(pe, g, K):
            v = g.variant(K, flags)
            if name == "auto":
                seen.add(v)
            elif v in seen and name != "auto" and K * w.num_ops > (1 << 24):
                continue                                   # the auto run already covered this variant at full size
            gpu, ref = gu.check(g, w, assign, order, flags=flags, label=f"config {config} {kw} {name}")
            assert (ref["status"] & gu.INVALID == 0).all()
    finally:
        g.close()


@pytest.mark.parametrize("config,kw", [(1, {}), (3, {}), (5, dict(V=256, D=64)), (5, dict(V=1024, D=8))])
@pytest.mark.parametrize("layout", ["assign_by_pos", "times_by_op", "both", "summary_only"])
def test_layout_flags(pe, config, kw, layout):
    w = wl.make_config(config, **kw)
    K = 1000                                               # ragged: not a multiple of any block size
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        base = {"assign_by_pos": pe.PE_ASSIGN_BY_POS, "times_by_op": pe.PE_TIMES_BY_OP,
                "both": pe.PE_ASSIGN_BY_POS | pe.PE_TIMES_BY_OP, "summary_only": 0}[layout]
        a = wl.assign_by_pos(assign, order) if base & pe.PE_ASSIGN_BY_POS else assign
        for name, flags in variants_for(pe, g, K, base):
            gu.check(g, w, a, order, flags=flags, want_times=layout != "summary_only", label=f"{layout} {name}")
    finally:
        g.close()


@pytest.mark.parametrize("K", [0, 1, 31, 33, 257])
def test_small_and_ragged_batches(pe, K):
    w = wl.make_config(2)
    g = pe.Graph(w)
    try:
        if K == 0:
            o = pe.make_outputs()
            assert pe.pe_eval_batch(g.handle, 0, 0, 0, 2, 0, o) == pe.PE_OK
            return
        assign, order = wl.make_candidates(w, K=K)
        for name, flags in variants_for(pe, g, K):
            gu.check(g, w, assign, order, flags=flags, label=f"K={K} {name}")
    finally:
        g.close()


def test_degenerate_graphs(pe):
    cases = [
        ck.problem(1, [], [5], 1, A=[2], cap=[1]),                                  # one op, one machine, over capacity
        ck.problem(6, [], [1, 2, 3, 4, 5, 6], 3, A=[1, 1, 1, -1, -1, -1]),          # no edges
        ck.problem(5, [(0, 4), (1, 4), (2, 4), (3, 4), (0, 4)], [1, 0, 2, 0, 3], 2, comm=2),   # duplicate edge, zero durations
        ck.problem(4, [(0, 1), (1, 2), (2, 3)], [1, 1, 1, 1], 255, comm=3),         # D = 255
    ]
    for n, w in enumerate(cases):
        w.assign_mode, w.group = "per_op", None
        K = 77
        assign, order = wl.make_candidates(w, K=K)
        g = pe.Graph(w)
        try:
            for name, flags in variants_for(pe, g, K):
                gu.check(g, w, assign, order, flags=flags, label=f"degenerate {n} {name}")
        finally:
            g.close()


def test_weights_link_classes_and_missing_channels(pe):
    w = wl.make_config(3)
    w.mem_weight = (np.arange(w.num_ops) % 7).astype(np.int32)
    w.link_class = w.link_class.copy()
    w.link_class[3, 12] = 0xFF                              # one directed pair without a channel
    w.mem_capacity = np.full(w.num_devices, 760, np.int32)   # near the typical per-machine peak: both outcomes occur
    K = 512
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        for name, flags in variants_for(pe, g, K):
            gpu, ref = gu.check(g, w, assign, order, flags=flags, label=f"weights {name}")
            assert (ref["status"] & pe.PE_STATUS_NO_CHANNEL).any()
            exceeded = (ref["status"] & pe.PE_STATUS_MEM_EXCEEDED) != 0
            assert exceeded.any() and not exceeded.all()
    finally:
        g.close()


def test_u32_orders(pe):
    w = wl.make_config(5, V=1024, D=8)
    K = 300
    assign, order = wl.make_candidates(w, K=K, order_bytes=4)
    assert order.dtype == np.uint32
    g = pe.Graph(w)
    try:
        for name, flags in variants_for(pe, g, K):
            if name == "team":                              # 16-bit orders only: refused, not mis-evaluated
                with pytest.raises(pe.PeError) as err:
                    gu.gpu_eval(g, assign, order, flags=flags)
                assert err.value.code == pe.PE_ERR_UNSUPPORTED
                continue
            gu.check(g, w, assign, order, flags=flags, label=f"u32 {name}")
    finally:
        g.close()


def test_invalid_candidates_are_flagged_and_stay_in_bounds(pe):
    w = wl.make_config(1)
    K = 64
    assign, order = wl.make_candidates(w, K=K)
    assign, order = assign.copy(), order.copy()
    order[[3, 40], 1] = order[[40, 3], 1]          # may or may not break a dependency; the oracle decides
    order[5, 2] = order[4, 2]                      # duplicate (and so a missing op)
    order[7, 3] = 60000                            # id out of range
    assign[:, 4] = 200                             # machine id out of range
    assign[9, 5] = 4                               # one machine id = D
    order[:, 6] = order[::-1, 6].copy()            # reversed: every dependency broken
    g = pe.Graph(w)
    try:
        for base in (0, pe.PE_ASSIGN_BY_POS):
            a = wl.assign_by_pos(assign, order) if base else assign
            for name, flags in variants_for(pe, g, K, base):
                gpu, ref = gu.check(g, w, a, order, flags=flags, label=f"invalid {name}")
                assert (ref["status"][[2, 3, 6]] & pe.PE_STATUS_ORDER_INVALID).all()
                assert (ref["status"][[4, 5]] & pe.PE_STATUS_ASSIGN_RANGE).all()
                assert (ref["status"][8:] == gpu["status"][8:]).all()
    finally:
        g.close()


def test_large_time_bound_falls_back_to_the_global_variant(pe):
    w = wl.make_config(5, V=256, D=8)
    w.dur = (w.dur.astype(np.int64) * 100000).astype(np.int32)       # sum of durations ~ 1.3e9 < 2^31
    K = 200
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        assert g.variant(K) == "global"
        assert pe.pe_eval_variant(g.handle, K, pe.PE_VARIANT_SHARED) == pe.PE_ERR_UNSUPPORTED
        gu.check(g, w, assign, order, label="large times")
    finally:
        g.close()


def test_workspace_is_checked(pe):
    import torch
    w = wl.make_config(1)
    K = 128
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        flags = pe.PE_VARIANT_GLOBAL
        need = pe.pe_workspace_bytes(g.handle, K, flags)
        assert need >= w.num_ops * K * 4
        a = torch.from_numpy(assign).cuda(); o = torch.from_numpy(gu.as_signed(order)).cuda()
        out = g.alloc_outputs(K)
        outs = pe.make_outputs(**{k: v.data_ptr() for k, v in out.items()})
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        assert pe.pe_eval_batch(g.handle, K, a.data_ptr(), o.data_ptr(), 2, flags, outs, ws.data_ptr(), need - 1, 0) == pe.PE_ERR_WORKSPACE
        assert pe.pe_eval_batch(g.handle, K, a.data_ptr(), o.data_ptr(), 2, flags, outs, 0, 0, 0) == pe.PE_ERR_WORKSPACE
        assert pe.pe_eval_batch(g.handle, K, a.data_ptr(), o.data_ptr(), 3, flags, outs, ws.data_ptr(), need, 0) == pe.PE_ERR_INVALID_ARG
        assert pe.pe_eval_batch(g.handle, K, a.data_ptr(), o.data_ptr(), 2, 1 << 20, outs, ws.data_ptr(), need, 0) == pe.PE_ERR_INVALID_ARG
        assert pe.pe_graph_poll_error(g.handle, 0) == pe.PE_OK
    finally:
        g.close()


def test_host_buffer_entry_point(pe):
    import torch
    w = wl.make_config(2)
    K = 4096
    V, D = w.num_ops, w.num_devices
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        h_a = torch.from_numpy(assign).pin_memory(); h_o = torch.from_numpy(gu.as_signed(order)).pin_memory()
        d_a = torch.empty_like(h_a, device="cuda"); d_o = torch.empty_like(h_o, device="cuda")
        d_out = g.alloc_outputs(K)
        h_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in d_out.items()}
        ws, ws_bytes = g.alloc_workspace(K)
        before = pe.pe_kernel_launches()
        rc = pe.pe_eval_batch_host(g.handle, K, h_a.data_ptr(), h_o.data_ptr(), 2, 0,
                                   pe.make_outputs(**{k: v.data_ptr() for k, v in h_out.items()}),
                                   d_a.data_ptr(), d_o.data_ptr(),
                                   pe.make_outputs(**{k: v.data_ptr() for k, v in d_out.items()}),
                                   ws.data_ptr(), ws_bytes, torch.cuda.current_stream().cuda_stream)
        assert rc == pe.PE_OK and pe.pe_kernel_launches() == before + 1
        res = {k: v.numpy() for k, v in h_out.items()}
        res["status"] = res["status"].view(np.uint32)
        from oracle import pe_oracle as orc
        gu.compare(res, orc.evaluate(w, assign, order, threads=gu.CPU_THREADS), "host entry point")
    finally:
        g.close()


@pytest.mark.parametrize("layout", ["default", "assign_by_pos", "times_by_op", "summary_only"])
def test_warp_variant_with_long_rows_uses_shared_tiles(pe, layout):
    """With K >= 2^19 the warp-per-candidate kernel moves order entries and times through shared tiles,
    a slab of positions at a time (block barriers, ragged last block and last slab)."""
    w = wl.make_config(5, V=256, D=8)
    K = (1 << 19) + 77
    assign, order = wl.make_candidates(w, K=K)
    base = {"default": 0, "assign_by_pos": pe.PE_ASSIGN_BY_POS, "times_by_op": pe.PE_TIMES_BY_OP, "summary_only": 0}[layout]
    a = wl.assign_by_pos(assign, order) if base & pe.PE_ASSIGN_BY_POS else assign
    g = pe.Graph(w)
    try:
        gu.check(g, w, a, order, flags=base | pe.PE_VARIANT_WARP, want_times=layout != "summary_only",
                 label=f"warp slab {layout}")
    finally:
        g.close()


def test_host_buffer_entry_point_pipelined_chunks(pe):
    """A batch large enough to be cut into chunks (ragged last chunk): uploads, kernels and downloads of
    different chunks overlap, and every output still lands in the caller's [rows][K] host layout."""
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(1)
    K = 40001
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        for flags in (0, pe.PE_ASSIGN_BY_POS | pe.PE_TIMES_BY_OP):
            a = wl.assign_by_pos(assign, order) if flags & pe.PE_ASSIGN_BY_POS else assign
            h_a = torch.from_numpy(a).pin_memory(); h_o = torch.from_numpy(gu.as_signed(order)).pin_memory()
            d_a = torch.empty_like(h_a, device="cuda"); d_o = torch.empty_like(h_o, device="cuda")
            d_out = g.alloc_outputs(K)
            h_out = {k: torch.full(v.shape, -5, dtype=v.dtype).pin_memory() for k, v in d_out.items()}
            ws, ws_bytes = g.alloc_workspace(K, flags)
            before = pe.pe_kernel_launches()
            rc = pe.pe_eval_batch_host(g.handle, K, h_a.data_ptr(), h_o.data_ptr(), 2, flags,
                                       pe.make_outputs(**{k: v.data_ptr() for k, v in h_out.items()}),
                                       d_a.data_ptr(), d_o.data_ptr(),
                                       pe.make_outputs(**{k: v.data_ptr() for k, v in d_out.items()}),
                                       ws.data_ptr(), ws_bytes, torch.cuda.current_stream().cuda_stream)
            assert rc == pe.PE_OK and pe.pe_kernel_launches() == before + 8
            res = {k: v.numpy() for k, v in h_out.items()}
            res["status"] = res["status"].view(np.uint32)
            gu.compare(res, orc.evaluate(w, a, order, flags=flags, threads=gu.CPU_THREADS), f"pipelined host call {flags}")
    finally:
        g.close()


def test_select_best_matches_the_definition(pe):
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(1)                                   # capacity 8: a mix of feasible and infeasible candidates
    K = 5000
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        out = g.eval_batch(torch.from_numpy(assign).cuda(), torch.from_numpy(gu.as_signed(order)).cuda())
        torch.cuda.synchronize()
        mk = out["makespan"].cpu().numpy(); st = out["status"].cpu().numpy().view(np.uint32)
        assert (st != 0).any() and (st == 0).any()
        for mask in (0xFFFFFFFF, 3, 4):
            assert g.select_best(out, mask) == orc.select_best(mk, st, mask)
        out["status"].fill_(4)                              # nobody qualifies
        assert g.select_best(out) == (-1, 2 ** 31 - 1, 0)
        out["status"].zero_(); out["makespan"].fill_(77)    # all tie: the first wins
        assert g.select_best(out) == (0, 77, K)
        res = torch.empty(4, dtype=torch.int64, device="cuda")
        assert pe.pe_select_best(0, 0, 0, 0xFFFFFFFF, res.data_ptr(), 0) == pe.PE_OK
        torch.cuda.synchronize()
        assert res[:3].tolist() == [-1, 2 ** 31 - 1, 0]
        # a batch larger than one pass of the grid
        big_m = torch.randint(100, 1 << 20, (1 << 21,), dtype=torch.int32, device="cuda")
        big_s = (torch.rand(1 << 21, device="cuda") < 0.5).to(torch.int32) * 4
        got = g.select_best({"makespan": big_m, "status": big_s})
        ok = big_s == 0
        best = int(big_m[ok].min())
        first = int(torch.nonzero(ok & (big_m == best))[0])
        assert got == (first, best, int(ok.sum()))
    finally:
        g.close()


def test_bench_configuration_sampled(pe):
    """The benchmark's own launch (sweep point V=16384, D=64 at its full K) on sampled candidates:
    every output of 512 randomly chosen candidates against the oracle, plus size-independent
    properties on all of them."""
    import torch
    w = wl.make_config(5, V=16384, D=64)
    K = w.num_candidates
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        gpu = gu.gpu_eval(g, assign, order)
        rs = np.random.RandomState(5)
        sample = np.sort(rs.choice(K, 512, replace=False))
        from oracle import pe_oracle as orc
        ref = orc.evaluate(w, np.ascontiguousarray(assign[:, sample]), np.ascontiguousarray(order[:, sample]),
                           threads=gu.CPU_THREADS)
        sub = {k: (v[sample] if v.ndim == 1 else v[:, sample]) for k, v in gpu.items()}
        gu.compare(sub, ref, "bench configuration sample")
        total = int(w.dur.astype(np.int64).sum())
        assert (gpu["status"] == 0).all()
        assert (gpu["busy"].sum(axis=0) == total).all()
        assert np.array_equal(gpu["makespan"], gpu["finish"].max(axis=0))
        assert (gpu["finish"] - gpu["start"] == w.dur[order.astype(np.int64)]).all()
        assert (gpu["makespan"] >= gpu["busy"].max(axis=0)).all() and (gpu["makespan"] >= ck.critical_path(w)).all()
    finally:
        g.close()


def test_bounded_wait_reports_a_timeout_and_leaves_the_graph_usable(pe):
    """The kernels' only wait (for the bulk copy that stages the graph) is bounded.  The self-test lets that wait
    run out - a barrier that expects bytes no copy brings - and the host must read PE_ERR_TIMEOUT once, then
    find the graph and the context in working order."""
    w = wl.make_config(2)
    K = 256
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        assert pe.pe_graph_poll_error(g.handle, 0) == pe.PE_OK
        assert pe.pe_selftest_wait_timeout(g.handle, 0) == pe.PE_OK
        assert pe.pe_graph_poll_error(g.handle, 0) == pe.PE_ERR_TIMEOUT
        assert pe.pe_graph_poll_error(g.handle, 0) == pe.PE_OK          # reading clears it
        gu.check(g, w, assign, order, label="after the self-test")
        assert pe.pe_graph_poll_error(g.handle, 0) == pe.PE_OK
    finally:
        g.close()


@pytest.mark.parametrize("V,D", [(256, 8), (256, 64), (1024, 8), (1024, 64), (4096, 8), (4096, 64), (16384, 8)])
def test_other_sweep_points_at_full_size_sampled(pe, V, D):
    """Sweep points at their full K (K * V = 2^30), i.e. in the launch shapes the benchmark times them in (ragged
    shared-state blocks at V = 1024 / D = 8, slab mode of the warp kernel at V = 1024 / D = 64, register slots with
    final rounds at V = 4096).  The batch repeats 8192 generated candidates; 256 sampled columns are compared
    with the oracle in full, every column with its twin and with size-independent properties."""
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(5, V=V, D=D)
    K, base = w.num_candidates, 8192
    a0, o0 = wl.make_candidates(w, K=base)
    assign = np.tile(a0, (1, K // base)); order = np.tile(o0, (1, K // base))
    g = pe.Graph(w)
    try:
        a = torch.from_numpy(assign).cuda(); o = torch.from_numpy(gu.as_signed(order)).cuda()
        out = g.eval_batch(a, o)
        torch.cuda.synchronize()
        rs = np.random.RandomState(V + D)
        sample = np.sort(rs.choice(K, 256, replace=False))
        st = torch.from_numpy(sample).cuda()
        sub = {k: (v[st] if v.dim() == 1 else v[:, st]).cpu().numpy() for k, v in out.items()}
        sub["status"] = sub["status"].view(np.uint32)
        ref = orc.evaluate(w, np.ascontiguousarray(assign[:, sample]), np.ascontiguousarray(order[:, sample]),
                           threads=gu.CPU_THREADS)
        gu.compare(sub, ref, f"V={V} D={D} full size")
        assert int(out["status"].abs().max()) == 0
        assert bool((out["busy"].sum(dim=0) == int(w.dur.astype(np.int64).sum())).all())
        assert bool((out["makespan"] == out["finish"].max(dim=0).values).all())
        first = out["makespan"][:base]
        assert bool((out["makespan"].view(K // base, base) == first).all())       # every repeat like its original
    finally:
        g.close()


def test_select_topk_matches_the_definition(pe):
    """pe_select_topk against its definition written out in the oracle (small K) and, at sizes where that loop
    is too slow, against numpy's stable sort of (makespan, index), which the oracle's pins show to be the same."""
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(1)
    g = pe.Graph(w)
    try:
        rs = np.random.RandomState(7)
        for K, k, hi in ((1, 1, 5), (37, 5, 3), (1000, 100, 50), (4097, 4097, 9), (5000, 0, 10), (3000, 4000, 10 ** 6),
                         (300000, 30000, 1 << 20), (300000, 1000, 40)):
            mk = rs.randint(0, hi, K).astype(np.int32)
            st = (rs.randint(0, 4, K) == 0).astype(np.uint32) * rs.randint(1, 16, K).astype(np.uint32)
            if K == 4097:
                mk[:] = 7                                        # all equal: the choice is by index alone
            out = dict(makespan=torch.from_numpy(mk).cuda(), status=torch.from_numpy(st.view(np.int32)).cuda())
            for mask in (0xFFFFFFFF, 3):
                idx, cnt = g.select_topk(out, k, mask)
                torch.cuda.synchronize()
                idx, cnt = idx.cpu().numpy(), int(cnt.item())
                ok = np.flatnonzero((st & np.uint32(mask)) == 0)
                want = sorted(ok[np.argsort(mk[ok], kind="stable")][:k].tolist())
                if K <= 1000:
                    assert want == orc.select_topk(mk, st, k, mask)
                assert cnt == len(want), (K, k, mask)
                assert idx[:cnt].tolist() == want, (K, k, mask)
                assert (idx[cnt:] == -1).all()
    finally:
        g.close()


@pytest.mark.parametrize("V,variant", [(256, "shared"), (256, "global"), (4096, "warp")])
def test_batches_beyond_32_bit_element_offsets(pe, V, variant):
    """K * V just above 2^32: the thread-per-candidate and warp-per-candidate kernels switch to 64-bit element
    offsets there.  The batch is built on the device by repeating 8192 generated candidates; summary outputs
    only (the times would be 34 GB); sampled columns against the oracle, every column against its twin."""
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(5, V=V, D=8)
    base = 8192
    reps = (1 << 32) // (V * base) + 1
    K = base * reps
    assert V * K > (1 << 32)
    a0, o0 = wl.make_candidates(w, K=base)
    flags = {"shared": pe.PE_VARIANT_SHARED, "global": pe.PE_VARIANT_GLOBAL, "warp": pe.PE_VARIANT_WARP}[variant]
    g = pe.Graph(w)
    try:
        assert g.variant(K, flags) == variant
        a = torch.from_numpy(a0).cuda().repeat(1, reps).contiguous()
        o = torch.from_numpy(gu.as_signed(o0)).cuda().repeat(1, reps).contiguous()
        out = g.eval_batch(a, o, flags=flags, want_times=False)
        torch.cuda.synchronize()
        del a, o
        rs = np.random.RandomState(V)
        sample = np.sort(np.concatenate([rs.choice(K, 200, replace=False), np.arange(K - 56, K)]))   # the far end too
        st = torch.from_numpy(sample).cuda()
        sub = {k: (v[st] if v.dim() == 1 else v[:, st]).cpu().numpy() for k, v in out.items()}
        sub["status"] = sub["status"].view(np.uint32)
        ref = orc.evaluate(w, np.ascontiguousarray(a0[:, sample % base]), np.ascontiguousarray(o0[:, sample % base]),
                           want_times=False, threads=gu.CPU_THREADS)
        gu.compare(sub, ref, f"64-bit offsets V={V} {variant}")
        assert int(out["status"].abs().max()) == 0
        assert bool((out["makespan"].view(reps, base) == out["makespan"][:base]).all())
        assert bool((out["busy"].view(-1, reps, base) == out["busy"][:, :base].unsqueeze(1)).all())
        assert bool((out["peak_mem"].view(-1, reps, base) == out["peak_mem"][:, :base].unsqueeze(1)).all())
    finally:
        g.close()
        torch.cuda.empty_cache()


def test_many_sources_of_one_operator_inside_its_window(pe):
    """Operators with five to eight incoming edges whose sources all sit in the same 32-position window, two
    link classes: the warp kernel then has to go back to the edge list for the sources beyond its inline
    slots.  Orders: the identity (sources right in front of their sink) and random topological ones."""
    rs = np.random.RandomState(42)
    V, D, L = 96, 5, 2
    edges = []
    for sink, fan in ((8, 8), (20, 6), (29, 5), (40, 7), (70, 8)):
        edges += [(sink - 1 - q, sink) for q in range(fan)]            # sources sink-fan .. sink-1
    edges += [(i, i + 1) for i in range(0, V - 1, 3)]                  # some chains across windows
    edges += [(int(a), int(b)) for a, b in zip(rs.randint(0, 40, 30), rs.randint(41, V, 30))]
    edges = sorted(set(edges))
    cls = rs.randint(0, L, (D, D)).astype(np.uint8)
    w = ck.problem(V, edges, rs.randint(1, 20, V), D, comm=rs.randint(0, 9, (len(edges), L)), L=L, link_class=cls,
                   A=rs.randint(-3, 4, V), cap=rs.randint(5, 30, D))
    w.assign_mode, w.group = "per_op", None
    K = 256
    assign, order = wl.make_candidates(w, K=K)
    order[:, :K // 2] = np.arange(V, dtype=order.dtype)[:, None]       # identity order for half of them
    g = pe.Graph(w)
    try:
        names = []
        for name, flags in variants_for(pe, g, K):
            gu.check(g, w, assign, order, flags=flags, label=f"many in-window sources {name}")
            names.append(name)
        assert "warp" in names
        a_pos = wl.assign_by_pos(assign, order)
        gu.check(g, w, a_pos, order, flags=pe.PE_VARIANT_WARP | pe.PE_ASSIGN_BY_POS, label="many in-window sources by-pos")
    finally:
        g.close()


@pytest.mark.parametrize("K", [333, 332])
def test_team_kernel_with_and_without_staging_copies(pe, K):
    """The block-per-candidate kernel reads the interleaved arrays directly when K is not a multiple of 4 (K = 333)
    and goes through candidate-major staging copies otherwise (K = 332); both, in every layout, on a graph large
    enough for it to be the automatic choice, and on the MoE graph (operators with eight incoming edges)."""
    for w in (wl.make_config(5, V=4096, D=8), wl.make_config(3)):
        assign, order = wl.make_candidates(w, K=K)
        g = pe.Graph(w)
        try:
            assert g.variant(K) == "team"
            for base in (0, pe.PE_ASSIGN_BY_POS, pe.PE_TIMES_BY_OP, pe.PE_ASSIGN_BY_POS | pe.PE_TIMES_BY_OP):
                a = wl.assign_by_pos(assign, order) if base & pe.PE_ASSIGN_BY_POS else assign
                gu.check(g, w, a, order, flags=base | pe.PE_VARIANT_TEAM, label=f"team K={K} flags={base}")
            gu.check(g, w, assign, order, flags=pe.PE_VARIANT_TEAM, want_times=False, label=f"team K={K} summary")
        finally:
            g.close()


def test_two_host_threads_share_a_graph(pe):
    """pe.h promises that a graph may be used from several host threads and streams.  The block-per-candidate
    variant forks onto side streams owned by the graph, so two threads, each with its own stream, workspace and
    outputs, evaluate different batches at the same time, several times over; both must get the oracle's result."""
    import threading
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(5, V=4096, D=64)
    K = 8000                                                   # more than one chunk: the side streams are used
    g = pe.Graph(w)
    try:
        batches = [wl.make_candidates(w, K=K, first=n * K) for n in range(2)]
        refs = [orc.evaluate(w, a, o, threads=gu.CPU_THREADS) for a, o in batches]
        errors = []

        def work(n):
            try:
                a, o = batches[n]
                s = torch.cuda.Stream()
                with torch.cuda.stream(s):
                    da = torch.from_numpy(a).cuda(); do = torch.from_numpy(gu.as_signed(o)).cuda()
                    ws = g.alloc_workspace(K, 0)
                    for _ in range(4):
                        out = g.eval_batch(da, do, workspace=ws, stream=s.cuda_stream)
                    s.synchronize()
                res = {k: v.cpu().numpy() for k, v in out.items()}
                res["status"] = res["status"].view(np.uint32)
                gu.compare(res, refs[n], f"thread {n}")
            except Exception as e:                               # reported by the main thread
                errors.append(e)

        threads = [threading.Thread(target=work, args=(n,)) for n in range(2)]
        for t in threads:
            t.start()
        for t in threads:
            t.join()
        assert not errors, errors
    finally:
        g.close()
