"""Parity of pe_decode_priority (through the C-ABI) with the oracle's priority-list decoding: bit-exact."""
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


def random_lists(V, K, seed):
    """K uniformly random permutations of the operators, [V, K] u16."""
    rs = np.random.RandomState(seed)
    return np.argsort(rs.randint(0, 1 << 30, size=(V, K)), axis=0, kind="stable").astype(np.uint16)


def decode_variants(pe, g, K):
    out = [("auto", 0)]
    for name, bit in (("shared", pe.PE_VARIANT_SHARED), ("global", pe.PE_VARIANT_GLOBAL)):
        if pe.pe_decode_variant(g.handle, K, bit) >= 0:
            out.append((name, bit))
    return out


def gpu_decode(g, plist, flags=0):
    import torch
    order, status = g.decode_priority(torch.from_numpy(gu.as_signed(plist)).cuda(g.device), flags=flags)
    torch.cuda.synchronize(g.device)
    return order.cpu().numpy().view(np.uint16), status.cpu().numpy().view(np.uint32)


def check(pe, w, plist, label):
    from oracle import pe_oracle as orc
    ref_order, ref_status = orc.decode(w, plist, threads=gu.CPU_THREADS)
    g = pe.Graph(w)
    try:
        for name, flags in decode_variants(pe, g, plist.shape[1]):
            order, status = gpu_decode(g, plist, flags)
            assert np.array_equal(status, ref_status), f"{label} {name}: status"
            ok = ref_status == 0
            assert np.array_equal(order[:, ok], ref_order[:, ok]), f"{label} {name}: order"
    finally:
        g.close()
    return ref_order, ref_status


CASES = [(1, {}, 1000), (2, {}, 4099), (3, {}, 1031), (4, {}, 2049)] + \
        [(5, dict(V=V, D=8), max(257, (1 << 21) // V)) for V in (256, 1024, 4096, 16384)]


@pytest.mark.parametrize("config,kw,K", CASES, ids=lambda v: str(v).replace(" ", ""))
def test_random_lists_decode_like_the_oracle(pe, config, kw, K):
    w = wl.make_config(config, **kw)
    check(pe, w, random_lists(w.num_ops, K, config), f"config {config} {kw}")


@pytest.mark.parametrize("K", [0, 1, 31, 33, 129])
def test_small_and_ragged_batches(pe, K):
    w = wl.make_config(2)
    if K == 0:
        g = pe.Graph(w)
        try:
            assert pe.pe_decode_priority(g.handle, 0, 0, 2, 0, 0) == pe.PE_OK
        finally:
            g.close()
        return
    check(pe, w, random_lists(w.num_ops, K, K), f"K={K}")


def test_topological_lists_come_back_unchanged_and_lists_that_are_no_permutation_are_flagged(pe):
    w = wl.make_config(3)
    K = 300
    _, order = wl.make_candidates(w, K=K)
    plist = order.copy()
    plist[5, 1] = plist[6, 1]             # an operator twice
    plist[0, 2] = 60000                   # no such operator
    plist[:, 3] = plist[::-1, 3].copy()   # reversed: still a permutation
    ref_order, ref_status = check(pe, w, plist, "lists")
    assert ref_status[[1, 2]].tolist() == [pe.PE_STATUS_ORDER_INVALID] * 2 and ref_status[3] == 0
    keep = np.ones(K, bool); keep[[1, 2, 3]] = False
    assert np.array_equal(ref_order[:, keep], order[:, keep])


def test_decoded_orders_evaluate_as_valid_candidates(pe):
    """Decoder and evaluator back to back on the device: every decoded order is accepted (status 0 up to
    the capacity flag) and evaluates like the oracle's decoding of the same list."""
    import torch
    from oracle import pe_oracle as orc
    w = wl.make_config(5, V=1024, D=8)
    K = 2048
    assign, _ = wl.make_candidates(w, K=K)
    plist = random_lists(w.num_ops, K, 7)
    g = pe.Graph(w)
    try:
        order, status = g.decode_priority(torch.from_numpy(gu.as_signed(plist)).cuda())
        out = g.eval_batch(torch.from_numpy(assign).cuda(), order)
        torch.cuda.synchronize()
        assert (status == 0).all()
        gpu = {k: v.cpu().numpy() for k, v in out.items()}
        gpu["status"] = gpu["status"].view(np.uint32)
        ref_order, _ = orc.decode(w, plist, threads=gu.CPU_THREADS)
        gu.compare(gpu, orc.evaluate(w, assign, ref_order, threads=gu.CPU_THREADS), "decode then evaluate")
        assert (gpu["status"] & gu.INVALID == 0).all()
    finally:
        g.close()


def test_unsupported_forms_are_refused(pe):
    w = wl.make_config(1)
    g = pe.Graph(w)
    try:
        assert pe.pe_decode_priority(g.handle, 4, 1, 4, 0, 1) == pe.PE_ERR_UNSUPPORTED      # 32-bit entries
        assert pe.pe_decode_priority(g.handle, 4, 1, 3, 0, 1) == pe.PE_ERR_INVALID_ARG
        assert pe.pe_decode_priority(g.handle, 4, 1, 2, 1, 1) == pe.PE_ERR_INVALID_ARG      # a flag that is no variant
        assert pe.pe_decode_priority(g.handle, 4, 0, 2, 0, 1) == pe.PE_ERR_INVALID_ARG      # NULL list
        need = pe.pe_decode_workspace_bytes(g.handle, 4, pe.PE_VARIANT_GLOBAL)
        assert need > 0
        assert pe.pe_decode_priority(g.handle, 4, 1, 2, pe.PE_VARIANT_GLOBAL, 1, 0, 0, 0) == pe.PE_ERR_WORKSPACE
    finally:
        g.close()
