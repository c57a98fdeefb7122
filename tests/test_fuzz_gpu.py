"""Randomised parity: small random problems (shapes, link classes, missing channels, weights, capacities,
zero durations, duplicate edges) through every kernel variant and flag combination, against the oracle."""
import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl
from tests import checkers as ck
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def random_problem(rs):
    V = int(rs.choice([1, 2, 5, 17, 33, 64, 100, 257, 300]))
    D = int(rs.choice([1, 2, 3, 8, 9, 31, 32, 33, 64, 70]))
    L = int(rs.choice([1, 1, 2]))
    n_edges = int(rs.randint(0, 3 * V + 1)) if V > 1 else 0
    edges = []
    for _ in range(n_edges):
        b = int(rs.randint(1, V)); a = int(rs.randint(max(0, b - 40), b))
        edges.append((a, b))                                  # duplicates allowed
    if rs.rand() < 0.3 and V > 12:                            # one operator with many incoming edges
        edges += [(int(a), V - 1) for a in rs.choice(V - 1, size=min(V - 1, 9), replace=False)]
    dur = rs.randint(0, 30, V)
    comm = rs.randint(0, 12, (len(edges), L))
    cls = None
    if L == 2 or rs.rand() < 0.4:
        cls = rs.randint(0, L, (D, D)).astype(np.uint8)
        if rs.rand() < 0.5 and D > 1:
            cls[rs.randint(0, D), rs.randint(0, D)] = 0xFF
    W = rs.randint(0, 5, V) if rs.rand() < 0.4 else None
    cap = rs.randint(0, 40, D) if rs.rand() < 0.7 else None
    w = ck.problem(V, edges, dur, D, comm=comm if len(edges) else None, L=L, link_class=cls, A=rs.randint(-4, 5, V), W=W, cap=cap)
    w.assign_mode, w.group = "per_op", None
    return w


@pytest.mark.parametrize("seed", range(24))
def test_random_problems_match_the_oracle_in_every_variant(seed):
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from oracle import pe_oracle as orc
    from paper_2503_09357_b200 import binding as pe
    rs = np.random.RandomState(1000 + seed)
    w = random_problem(rs)
    K = int(rs.choice([1, 31, 97, 200]))
    assign, order = wl.make_candidates(w, K=K, seed=seed)
    base = int(rs.choice([0, pe.PE_ASSIGN_BY_POS, pe.PE_TIMES_BY_OP, pe.PE_ASSIGN_BY_POS | pe.PE_TIMES_BY_OP]))
    a = wl.assign_by_pos(assign, order) if base & pe.PE_ASSIGN_BY_POS else assign
    g = pe.Graph(w)
    try:
        for name, bit in (("auto", 0), ("global", pe.PE_VARIANT_GLOBAL), ("shared", pe.PE_VARIANT_SHARED),
                          ("warp", pe.PE_VARIANT_WARP), ("team", pe.PE_VARIANT_TEAM), ("exclusive", pe.PE_COMM_EXCLUSIVE),
                          ("exclusive shared", pe.PE_COMM_EXCLUSIVE | pe.PE_VARIANT_SHARED),
                          ("exclusive global", pe.PE_COMM_EXCLUSIVE | pe.PE_VARIANT_GLOBAL)):
            if pe.pe_eval_variant(g.handle, K, base | bit) < 0:
                continue
            gu.check(g, w, a, order, flags=base | bit, want_times=bool(rs.rand() < 0.8), label=f"seed {seed} {name}")
        plist = np.stack([rs.permutation(w.num_ops) for _ in range(K)], axis=1).astype(np.uint16)
        ref_order, ref_status = orc.decode(w, plist)
        for bit in (0, pe.PE_VARIANT_SHARED, pe.PE_VARIANT_GLOBAL):
            if pe.pe_decode_variant(g.handle, K, bit) < 0:
                continue
            dorder, dstatus = g.decode_priority(torch.from_numpy(gu.as_signed(plist)).cuda(), flags=bit)
            torch.cuda.synchronize()
            assert (dstatus.cpu().numpy() == 0).all() and (ref_status == 0).all()
            assert np.array_equal(dorder.cpu().numpy().view(np.uint16), ref_order), f"seed {seed} decode {bit}"
    finally:
        g.close()
