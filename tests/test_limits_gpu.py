"""The largest sizes the 16-bit forms admit: V = 65535 (the last size with a compact graph encoding: the
sentinel row still has a 16-bit id) and V = 65536 (16-bit order entries still cover every operator)."""
import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl
from tests import checkers as ck
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def big_dag(V, D, seed):
    """Each operator after the first 64 draws 1-3 predecessors among the 4096 operators before it."""
    rs = np.random.RandomState(seed)
    dst = np.repeat(np.arange(64, V), 3)
    keep = rs.rand(dst.size) < 0.6
    keep[::3] = True
    dst = dst[keep]
    src = dst - 1 - rs.randint(0, np.minimum(dst, 4096))
    edges = sorted(set(zip(src.tolist(), dst.tolist())))
    w = ck.problem(V, edges, rs.randint(1, 20, V), D, comm=rs.randint(0, 5, (len(edges), 1)), A=rs.randint(-3, 4, V),
                   cap=[1 << 20] * D)
    w.assign_mode, w.group = "per_op", None
    return w


@pytest.fixture(scope="module")
def pe():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2503_09357_b200 import binding
    return binding


@pytest.mark.parametrize("V", [65535, 65536])
def test_evaluation_at_the_largest_sizes(pe, V):
    w = big_dag(V, 3, V)
    K = 48
    assign, order = wl.make_candidates(w, K=K, order_bytes=2)
    g = pe.Graph(w)
    try:
        seen = set()
        for name, bit in (("auto", 0), ("global", pe.PE_VARIANT_GLOBAL), ("warp", pe.PE_VARIANT_WARP),
                          ("team", pe.PE_VARIANT_TEAM)):
            if pe.pe_eval_variant(g.handle, K, bit) < 0:
                continue
            gu.check(g, w, assign, order, flags=bit, label=f"V={V} {name}")
            seen.add(name)
        assert "global" in seen
    finally:
        g.close()


def test_decoding_at_the_largest_size(pe):
    import torch
    from oracle import pe_oracle as orc
    V, K = 65536, 40
    w = big_dag(V, 3, 1)
    rs = np.random.RandomState(2)
    plist = np.stack([rs.permutation(V) for _ in range(K)], axis=1).astype(np.uint16)
    plist[:, 3] = np.arange(V, dtype=np.uint16)[::-1]      # rank 0 is operator 65535
    ref_order, ref_status = orc.decode(w, plist, threads=gu.CPU_THREADS)
    g = pe.Graph(w)
    try:
        order, status = g.decode_priority(torch.from_numpy(gu.as_signed(plist)).cuda())
        torch.cuda.synchronize()
        assert (status.cpu().numpy() == 0).all() and (ref_status == 0).all()
        assert np.array_equal(order.cpu().numpy().view(np.uint16), ref_order)
    finally:
        g.close()
