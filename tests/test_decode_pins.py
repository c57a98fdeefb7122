"""Pins of the oracle's priority-list decoding (oracle/pe_oracle.cpp::pe_oracle_decode) against
things fixed without it: brute force over all topological orders, special cases with an
obvious answer, and the input generator's independent random-key Kahn sort."""
import itertools

import numpy as np
import pytest

from oracle import pe_oracle as orc
from paper_2503_09357_b200 import workloads as wl
from paper_2503_09357_b200.workloads import rng
from tests import checkers as ck


class _G:
    def __init__(self, V, edges):
        self.num_ops = V
        self.edge_src = np.array([a for a, _ in edges], np.int32)
        self.edge_dst = np.array([b for _, b in edges], np.int32)


TINY = [
    (5, [(0, 2), (1, 2), (2, 3), (1, 4)]),
    (6, [(0, 3), (1, 3), (1, 4), (2, 4), (3, 5), (4, 5)]),
    (6, [(5, 0), (4, 0), (0, 1), (3, 2)]),            # edges against the numbering
    (7, [(0, 1), (1, 2), (3, 4), (4, 5), (2, 6), (5, 6)]),
    (4, []),
]


def _is_topological(order, V, edges):
    pos = np.empty(V, np.int64)
    pos[order] = np.arange(V)
    return sorted(order) == list(range(V)) and all(pos[a] < pos[b] for a, b in edges)


@pytest.mark.parametrize("V,edges", TINY)
def test_decoded_order_is_the_rank_wise_smallest_topological_order(V, edges):
    """Always taking the smallest rank among the available operations yields, of all topological orders,
    the one whose sequence of ranks is lexicographically smallest (exchange argument).  Checked by
    enumerating every topological order, for every priority list (V <= 5) or 200 random ones."""
    g = _G(V, edges)
    topo = ck.topological_orders(V, edges)
    if V <= 5:
        lists = list(itertools.permutations(range(V)))
    else:
        rs = np.random.RandomState(V)
        lists = [rs.permutation(V) for _ in range(200)]
    plist = np.array(lists, np.uint16).T.copy()
    order, status = orc.decode(g, plist)
    assert (status == 0).all()
    for c, lst in enumerate(lists):
        rank = np.empty(V, np.int64)
        rank[list(lst)] = np.arange(V)
        best = min(topo, key=lambda t: [int(rank[i]) for i in t])
        assert order[:, c].tolist() == best


def test_without_edges_the_list_itself_and_on_a_chain_the_chain():
    rs = np.random.RandomState(0)
    V, K = 9, 50
    plist = np.stack([rs.permutation(V) for _ in range(K)], axis=1).astype(np.uint16)
    order, _ = orc.decode(_G(V, []), plist)
    assert np.array_equal(order, plist)
    chain = [(i + 1, i) for i in range(V - 1)]                # 8 -> 7 -> ... -> 0
    order, _ = orc.decode(_G(V, chain), plist)
    assert np.array_equal(order, np.repeat(np.arange(V - 1, -1, -1, dtype=np.uint16)[:, None], K, axis=1))


@pytest.mark.parametrize("config,kw", [(1, {}), (2, {}), (3, {}), (4, {}), (5, dict(V=256, D=8)), (5, dict(V=1024, D=64))])
def test_topological_lists_come_back_unchanged_and_any_list_gives_a_topological_order(config, kw):
    w = wl.make_config(config, **kw)
    K = 24
    _, order = wl.make_candidates(w, K=K)
    back, status = orc.decode(w, order)
    assert (status == 0).all() and np.array_equal(back, order)
    rs = np.random.RandomState(config)
    plist = np.stack([rs.permutation(w.num_ops) for _ in range(K)], axis=1).astype(order.dtype)
    dec, status = orc.decode(w, plist)
    assert (status == 0).all()
    edges = list(zip(w.edge_src.tolist(), w.edge_dst.tolist()))
    for c in range(K):
        assert _is_topological(dec[:, c].astype(np.int64), w.num_ops, edges)
    again, _ = orc.decode(w, dec)
    assert np.array_equal(again, dec)                         # decoding is idempotent


@pytest.mark.parametrize("config,kw", [(1, {}), (3, {}), (5, dict(V=1024, D=8))])
def test_agrees_with_the_generators_random_key_sort(config, kw):
    """The input generator draws a 32-bit key per operation and runs its own Kahn sort with a heap of
    (key, id) pairs.  Ranking the operations by (key, id) and decoding that list must give the same order."""
    w = wl.make_config(config, **kw)
    V, K, first = w.num_ops, 12, 5
    _, order = wl.make_candidates(w, K=K, first=first)
    plist = np.empty((V, K), order.dtype)
    for c in range(K):
        keys = (rng.rand64(wl.DEFAULT_SEED, 101, first + c, np.arange(V)) >> np.uint64(32)).astype(np.uint64)
        plist[:, c] = np.lexsort((np.arange(V), keys))        # by key, ties by id
    dec, status = orc.decode(w, plist)
    assert (status == 0).all() and np.array_equal(dec, order)


def test_lists_that_are_no_permutation_are_flagged():
    V, edges = TINY[1]
    plist = np.repeat(np.arange(V, dtype=np.uint16)[:, None], 4, axis=1)
    plist[2, 1] = 3                  # operation 3 twice, 2 missing
    plist[0, 2] = 60000              # no such operation
    _, status = orc.decode(_G(V, edges), plist)
    assert status.tolist() == [0, orc.STATUS_ORDER_INVALID, orc.STATUS_ORDER_INVALID, 0]
