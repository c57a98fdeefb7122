"""The seeded generators produce the shapes the benchmark configurations state and valid candidates."""
import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl


@pytest.mark.parametrize("config,V,E,D,L,K", [(1, 64, 56, 4, 1, 1024), (2, 480, 460, 8, 1, 65536),
                                              (3, 2816, 4604, 16, 2, 16384), (4, 1536, 1528, 32, 2, 65536)])
def test_fixed_config_shapes(config, V, E, D, L, K):
    w = wl.make_config(config)
    assert (w.num_ops, w.num_edges, w.num_devices, w.num_link_classes, w.num_candidates) == (V, E, D, L, K)
    assert w.comm.shape == (E, L) and w.dur.shape == (V,) and w.mem_delta.shape == (V,)
    assert (w.dur >= 1).all() and (w.comm >= 0).all()
    if config >= 3:
        assert int(w.mem_delta.sum()) == 0                     # every allocation has its matching release
        assert np.bincount(w.edge_dst, minlength=V).max() == (8 if config == 3 else 2)


@pytest.mark.parametrize("V,D", wl.SWEEP_POINTS)
def test_sweep_point_shapes(V, D):
    w = wl.make_config(5, V=V, D=D)
    side = int(round(V ** 0.5))
    indeg = np.bincount(w.edge_dst, minlength=V)
    assert w.num_candidates * V == 1 << 30
    assert (indeg[:side] == 0).all() and (indeg[side:] >= 1).all() and indeg.max() <= 3
    assert (w.edge_src // side < w.edge_dst // side).all()      # predecessors come from earlier layers
    assert len(set(zip(w.edge_src.tolist(), w.edge_dst.tolist()))) == w.num_edges   # distinct predecessors
    assert w.dur.min() >= 1 and w.dur.max() <= 100 and w.comm.max() <= 20
    assert w.mem_delta.min() >= -3 and w.mem_delta.max() <= 3


@pytest.mark.parametrize("config,kw", [(1, {}), (2, {}), (3, {}), (4, {}), (5, dict(V=1024, D=64))])
def test_candidates_are_topological_permutations(config, kw):
    w = wl.make_config(config, **kw)
    K = 200
    assign, order = wl.make_candidates(w, K=K)
    V = w.num_ops
    assert assign.max() < w.num_devices
    for c in range(0, K, 7):
        pi = order[:, c].astype(np.int64)
        assert np.array_equal(np.sort(pi), np.arange(V))
        pos = np.empty(V, np.int64); pos[pi] = np.arange(V)
        assert (pos[w.edge_src] < pos[w.edge_dst]).all()
    if w.assign_mode == "group_perm":
        for c in range(0, K, 7):
            sigma = {}
            for g, j in zip(w.group.tolist(), assign[:, c].tolist()):
                assert sigma.setdefault(g, j) == j               # one machine per pipeline slot
            assert sorted(sigma.values()) == list(range(w.num_devices))
    assert len({order[:, c].tobytes() for c in range(K)}) > K // 2   # candidates differ


def test_candidates_are_counter_based():
    """Candidate c is the same whichever batch it is generated in, and whatever the thread count."""
    w = wl.make_config(3)
    a1, o1 = wl.make_candidates(w, K=96, threads=1)
    a2, o2 = wl.make_candidates(w, K=32, first=40, threads=3)
    assert np.array_equal(a1[:, 40:72], a2) and np.array_equal(o1[:, 40:72], o2)
    a3, o3 = wl.make_candidates(w, K=96, seed=7)
    assert not np.array_equal(o1, o3)


def test_assign_by_pos_is_a_gather():
    w = wl.make_config(4)
    assign, order = wl.make_candidates(w, K=50)
    seq = wl.assign_by_pos(assign, order)
    assert np.array_equal(seq, assign[order.astype(np.int64), np.arange(50)[None, :]])
