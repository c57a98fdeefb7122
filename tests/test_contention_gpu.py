"""Parity of the exclusive-channel communication model (PE_COMM_EXCLUSIVE, Eqs. 14-15) with the oracle."""
import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pe():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2503_09357_b200 import binding
    return binding


CASES = [(1, {}, 1024), (2, {}, 4099), (3, {}, 1031), (4, {}, 2049), (5, dict(V=256, D=64), 2000), (5, dict(V=1024, D=8), 1500)]


@pytest.mark.parametrize("config,kw,K", CASES, ids=lambda v: str(v).replace(" ", ""))
def test_exclusive_channels_match_the_oracle(pe, config, kw, K):
    w = wl.make_config(config, **kw)
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        seen = set()
        for name, bit in (("auto", 0), ("shared", pe.PE_VARIANT_SHARED), ("global", pe.PE_VARIANT_GLOBAL)):
            if pe.pe_eval_variant(g.handle, K, pe.PE_COMM_EXCLUSIVE | bit) < 0:
                continue
            gpu, ref = gu.check(g, w, assign, order, flags=pe.PE_COMM_EXCLUSIVE | bit, label=f"exclusive {config} {kw} {name}")
            seen.add(g.variant(K, pe.PE_COMM_EXCLUSIVE | bit))
        assert "global" in seen and (config not in (1, 2) or "shared" in seen)
        plain = gu.gpu_eval(g, assign, order)
        assert (gpu["finish"] >= plain["finish"]).all()
        if config >= 3:
            assert (gpu["makespan"] > plain["makespan"]).any()      # the channels do bind on these workloads
    finally:
        g.close()


@pytest.mark.parametrize("layout", ["assign_by_pos", "times_by_op", "summary_only"])
def test_exclusive_channels_with_layout_flags(pe, layout):
    w = wl.make_config(3)
    K = 333
    assign, order = wl.make_candidates(w, K=K)
    base = {"assign_by_pos": pe.PE_ASSIGN_BY_POS, "times_by_op": pe.PE_TIMES_BY_OP, "summary_only": 0}[layout]
    a = wl.assign_by_pos(assign, order) if base & pe.PE_ASSIGN_BY_POS else assign
    g = pe.Graph(w)
    try:
        gu.check(g, w, a, order, flags=base | pe.PE_COMM_EXCLUSIVE, want_times=layout != "summary_only", label=layout)
    finally:
        g.close()
    w = wl.make_config(2)                                    # small enough for the shared-state kernel
    assign, order = wl.make_candidates(w, K=K)
    a = wl.assign_by_pos(assign, order) if base & pe.PE_ASSIGN_BY_POS else assign
    g = pe.Graph(w)
    try:
        assert g.variant(K, base | pe.PE_COMM_EXCLUSIVE) == "shared"
        gu.check(g, w, a, order, flags=base | pe.PE_COMM_EXCLUSIVE, want_times=layout != "summary_only", label=layout + " shared")
    finally:
        g.close()


def test_which_kernels_offer_it(pe):
    w = wl.make_config(1)
    g = pe.Graph(w)
    try:
        K = 64
        assert pe.pe_eval_variant(g.handle, K, pe.PE_COMM_EXCLUSIVE | pe.PE_VARIANT_SHARED) == pe.PE_VARIANT_SHARED
        assert pe.pe_eval_variant(g.handle, K, pe.PE_COMM_EXCLUSIVE | pe.PE_VARIANT_WARP) == pe.PE_ERR_UNSUPPORTED
        assert pe.pe_eval_variant(g.handle, K, pe.PE_COMM_EXCLUSIVE | pe.PE_VARIANT_GLOBAL) == pe.PE_VARIANT_GLOBAL
        assert pe.pe_workspace_bytes(g.handle, K, pe.PE_COMM_EXCLUSIVE | pe.PE_VARIANT_GLOBAL) >= w.num_devices ** 2 * K * 4
        # the size query covers every form of the call (e.g. 32-bit orders, which take the global-state kernel)
        assert pe.pe_workspace_bytes(g.handle, K, pe.PE_COMM_EXCLUSIVE) >= w.num_devices ** 2 * K * 4
    finally:
        g.close()


def test_host_buffer_entry_point_with_exclusive_channels(pe):
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(4)
    K = 3000
    assign, order = wl.make_candidates(w, K=K)
    flags = pe.PE_COMM_EXCLUSIVE
    g = pe.Graph(w)
    try:
        h_a = torch.from_numpy(assign).pin_memory(); h_o = torch.from_numpy(gu.as_signed(order)).pin_memory()
        d_a = torch.empty_like(h_a, device="cuda"); d_o = torch.empty_like(h_o, device="cuda")
        d_out = g.alloc_outputs(K)
        h_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in d_out.items()}
        ws, ws_bytes = g.alloc_workspace(K, flags)
        rc = pe.pe_eval_batch_host(g.handle, K, h_a.data_ptr(), h_o.data_ptr(), 2, flags,
                                   pe.make_outputs(**{k: v.data_ptr() for k, v in h_out.items()}),
                                   d_a.data_ptr(), d_o.data_ptr(),
                                   pe.make_outputs(**{k: v.data_ptr() for k, v in d_out.items()}),
                                   ws.data_ptr(), ws_bytes, torch.cuda.current_stream().cuda_stream)
        assert rc == pe.PE_OK
        res = {k: v.numpy() for k, v in h_out.items()}
        res["status"] = res["status"].view(np.uint32)
        gu.compare(res, orc.evaluate(w, assign, order, flags=orc.COMM_EXCLUSIVE, threads=gu.CPU_THREADS), "host call, exclusive")
    finally:
        g.close()
