"""Graph coarsening (Section IV, Algorithm 1): the oracle against what the paper and graph theory fix,
then the library's pe_coarsen against the oracle.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import pe_coarsen_oracle as co
from tests import checkers as ck
from tests.conftest import ROOT

BIG = 10 ** 6


def random_dag(rs, V, p_edge=0.25, L=1):
    edges = [(a, b) for a in range(V) for b in range(a + 1, V) if rs.rand() < p_edge]
    perm = rs.permutation(V)                                   # labels do not follow the topological order
    edges = [(int(perm[a]), int(perm[b])) for a, b in edges]
    w = ck.problem(V, edges, rs.randint(1, 9, V), 2, comm=rs.randint(0, 5, (max(len(edges), 1), L))[:len(edges)], L=L,
                   A=rs.randint(-3, 4, V), W=rs.randint(0, 3, V))
    return w


def closure(n, edges):
    """Reachability by brute force (Warshall)."""
    r = np.zeros((n, n), bool)
    for a, b in edges:
        r[a, b] = True
    for k in range(n):
        r |= np.outer(r[:, k], r[k, :])
    return r


def critical_path(n, edges, dur):
    """Longest duration-weighted path, by the textbook recurrence over a topological order found by
    repeated source removal (also proves the graph is acyclic)."""
    indeg = [0] * n
    for _, b in edges:
        indeg[b] += 1
    ready = [i for i in range(n) if indeg[i] == 0]
    dist = [int(d) for d in dur]
    seen = 0
    while ready:
        u = ready.pop()
        seen += 1
        for a, b in edges:
            if a == u:
                dist[b] = max(dist[b], dist[u] + int(dur[b]))
                indeg[b] -= 1
                if indeg[b] == 0:
                    ready.append(b)
    assert seen == n, "the graph has a cycle"
    return max(dist)


def edges_of(w):
    return [(int(a), int(b)) for a, b in zip(w.edge_src, w.edge_dst)]


@pytest.mark.parametrize("seed", range(12))
def test_oracle_invariants(seed):
    rs = np.random.RandomState(seed)
    V = int(rs.randint(6, 13))
    w = random_dag(rs, V, L=int(rs.choice([1, 2])))
    N = int(rs.randint(2, V))
    r = co.coarsen(w, N, int(rs.randint(8, 40)), BIG, int(rs.randint(6, 20)), BIG)
    n = r.num_ops
    ce = edges_of(r)
    critical_path(n, ce, r.dur)                                   # a DAG
    assert len(set(ce)) == len(ce) and all(a != b for a, b in ce)
    # attributes are sums over the members
    for arr, src in ((r.dur, w.dur), (r.mem_delta, w.mem_delta), (r.mem_weight, w.mem_weight)):
        assert np.array_equal(np.bincount(r.op_map, weights=src, minlength=n).astype(np.int64), arr)
    # numbering: by smallest member
    firsts = [int(np.flatnonzero(r.op_map == g)[0]) for g in range(n)]
    assert firsts == sorted(firsts)
    # every original precedence is still implied, and nothing else is: group a reaches group b exactly when
    # some member of a reached some member of b
    ro, rc = closure(V, edges_of(w)), closure(n, ce)
    want = np.zeros((n, n), bool)
    for a, b in itertools.product(range(V), repeat=2):
        if ro[a, b] and r.op_map[a] != r.op_map[b]:
            want[r.op_map[a], r.op_map[b]] = True
    assert np.array_equal(rc, closure(n, list(zip(*np.nonzero(want)))))
    # a merged edge carries the largest communication duration of the edges it stands for
    for e, (a, b) in enumerate(ce):
        members = [k for k, (x, y) in enumerate(edges_of(w)) if r.op_map[x] == a and r.op_map[y] == b]
        assert members and np.array_equal(r.comm[e], w.comm[members].max(axis=0))


def test_edge_merges_are_safe_and_respect_the_rules():
    """Replaying the merge list: at the time of an edge merge the head had a single input and the tail a
    single output once two-hop shortcuts are set aside, the pair with the smallest merged duration went
    first, and the critical path kept its length (Section IV)."""
    for seed in range(10):
        rs = np.random.RandomState(100 + seed)
        V = int(rs.randint(7, 12))
        w = random_dag(rs, V, p_edge=0.2)
        r = co.coarsen(w, 2, 30, BIG, 0, BIG)                      # edge merges only
        group = {i: i for i in range(V)}
        dur = {i: int(w.dur[i]) for i in range(V)}
        edges = set(edges_of(w))
        for u, v, kind in r.merges:
            assert kind == "edge"
            live = sorted(set(group.values()))
            ge = {(group[a], group[b]) for a, b in edges if group[a] != group[b]}
            cp_before = critical_path(V, [(a, b) for a, b in ge], [dur.get(i, 0) for i in range(V)])
            red = {(a, b) for a, b in ge if any((a, c) in ge and (c, b) in ge for c in live)}
            kept = ge - red
            tail, head = (u, v) if (u, v) in ge else (v, u)
            assert (tail, head) in kept
            assert sum(1 for a, b in kept if a == tail) == 1 and sum(1 for a, b in kept if b == head) == 1
            cands = [(dur[a] + dur[b], a, b) for a, b in kept
                     if sum(1 for x, y in kept if x == a) == 1 and sum(1 for x, y in kept if y == b) == 1
                     and dur[a] + dur[b] <= 30]
            assert min(cands) == (dur[tail] + dur[head], tail, head)
            keep, gone = min(u, v), max(u, v)
            for i in group:
                if group[i] == gone:
                    group[i] = keep
            dur[keep] += dur.pop(gone)
            ge2 = {(group[a], group[b]) for a, b in edges if group[a] != group[b]}
            assert critical_path(V, list(ge2), [dur.get(i, 0) for i in range(V)]) == cp_before


def test_nonedge_merges_join_unrelated_operators_only():
    for seed in range(8):
        rs = np.random.RandomState(200 + seed)
        V = int(rs.randint(6, 11))
        w = random_dag(rs, V, p_edge=0.3)
        r = co.coarsen(w, 2, 0, BIG, 25, BIG)                      # non-edge merges only
        group = {i: i for i in range(V)}
        edges = edges_of(w)
        for u, v, kind in r.merges:
            assert kind == "nonedge"
            ge = [(group[a], group[b]) for a, b in edges if group[a] != group[b]]
            reach = closure(V, ge)
            assert not reach[u, v] and not reach[v, u]
            for i in group:
                if group[i] == v:
                    group[i] = u


def test_special_cases():
    chain = ck.problem(6, [(i, i + 1) for i in range(5)], [1, 2, 3, 4, 5, 6], 1, comm=1)
    r = co.coarsen(chain, 1, BIG, BIG, 0, 0)
    assert r.num_ops == 1 and r.dur.tolist() == [21] and len(r.edge_src) == 0        # a chain folds into one operator
    r = co.coarsen(chain, 6, BIG, BIG, BIG, BIG)
    assert r.num_ops == 6 and r.op_map.tolist() == list(range(6))                     # already small enough
    r = co.coarsen(chain, 1, 4, BIG, 0, 0)                                            # threshold: only 0+1 (3) and then nothing
    assert r.op_map.tolist() == [0, 0, 1, 2, 3, 4]
    free = ck.problem(4, [], [4, 3, 2, 1], 1)
    r = co.coarsen(free, 2, 0, 0, BIG, BIG)                                           # no edges: smallest pairs first
    assert r.merges == [(2, 3, "nonedge"), (1, 2, "nonedge")] and r.dur.tolist() == [4, 6]
    mem = ck.problem(3, [(0, 1), (1, 2)], [1, 1, 1], 1, A=[5, -5, 5], W=[1, 1, 1])
    r = co.coarsen(mem, 1, BIG, 7, 0, 0)                                              # requirement W + max(A, 0): 6, 1, 6
    assert r.op_map.tolist() == [0, 0, 1] and r.mem_delta.tolist() == [0, 5] and r.mem_weight.tolist() == [2, 1]


def read_golden():
    out = {"merges": []}
    mode = None
    for line in open(os.path.join(ROOT, "tests", "golden", "worked_example_coarsening.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        t = line.split()
        if t[0] == "merges":
            mode = "merges"
        elif t[0] in ("op_map", "dur", "edges"):
            mode = None
            out[t[0]] = [int(x) for x in t[1:]]
        elif mode == "merges":
            out["merges"].append((int(t[0]), int(t[1]), t[2]))
    return out


def golden_problem():
    return ck.problem(8, [(0, 1), (1, 2), (0, 2), (2, 3), (2, 4), (3, 5), (4, 5), (5, 6), (6, 7)],
                      [1, 2, 3, 4, 5, 6, 7, 8], 2, comm=1)


def test_hand_worked_example():
    g = read_golden()
    r = co.coarsen(golden_problem(), 3, 100, BIG, 12, BIG)
    assert r.merges == g["merges"]
    assert r.op_map.tolist() == g["op_map"] and r.dur.tolist() == g["dur"]
    assert [x for e in zip(r.edge_src, r.edge_dst) for x in map(int, e)] == g["edges"]


# ---- the library against the oracle ----
@pytest.fixture(scope="module")
def pe():
    from paper_2503_09357_b200.build import build_libpe
    build_libpe()
    from paper_2503_09357_b200 import binding
    return binding


def same(lib, ref):
    assert lib["num_ops"] == ref.num_ops
    for key in ("op_map", "edge_src", "edge_dst", "comm", "dur", "mem_delta", "mem_weight"):
        assert np.array_equal(lib[key], getattr(ref, key)), key


@pytest.mark.parametrize("seed", range(20))
def test_library_matches_the_oracle(pe, seed):
    rs = np.random.RandomState(300 + seed)
    V = int(rs.randint(5, 40))
    w = random_dag(rs, V, p_edge=float(rs.choice([0.05, 0.15, 0.3])), L=int(rs.choice([1, 2])))
    args = (int(rs.randint(1, V + 1)), int(rs.randint(0, 40)), int(rs.randint(0, 30)), int(rs.randint(0, 25)),
            int(rs.randint(0, 30)))
    desc, keep = pe.desc_from_workload(w)
    same(pe.pe_coarsen(desc, *args), co.coarsen(w, *args))


def test_library_on_the_benchmark_shapes_and_the_golden_case(pe):
    from paper_2503_09357_b200 import workloads as wl
    g = golden_problem()
    desc, keep = pe.desc_from_workload(g)
    same(pe.pe_coarsen(desc, 3, 100, BIG, 12, BIG), co.coarsen(g, 3, 100, BIG, 12, BIG))
    w = wl.make_config(1)                                          # the tiny pipeline: 64 operators
    desc, keep = pe.desc_from_workload(w)
    lib = pe.pe_coarsen(desc, 16, 12, BIG, 8, BIG)
    same(lib, co.coarsen(w, 16, 12, BIG, 8, BIG))
    assert lib["num_ops"] <= 64
    w = wl.make_config(5, V=256, D=8)                              # shaped like the paper's random graph (Section V-B)
    desc, keep = pe.desc_from_workload(w)
    lib = pe.pe_coarsen(desc, 40, 400, BIG, 150, BIG)
    same(lib, co.coarsen(w, 40, 400, BIG, 150, BIG))
    # the result is a valid problem description again
    d2, k2 = pe.make_desc(lib["num_ops"], lib["edge_src"], lib["edge_dst"], lib["dur"], w.num_devices,
                          mem_delta=lib["mem_delta"], mem_weight=lib["mem_weight"], comm=lib["comm"])
    assert pe.pe_graph_validate(d2) == pe.PE_OK


def test_library_argument_checks(pe):
    w = golden_problem()
    desc, keep = pe.desc_from_workload(w)
    with pytest.raises(pe.PeError) as e:
        pe.pe_coarsen(desc, 0, 1, 1, 1, 1)
    assert e.value.code == pe.PE_ERR_INVALID_ARG
    cyc = ck.problem(2, [(0, 1), (1, 0)], [1, 1], 1)
    desc, keep = pe.desc_from_workload(cyc)
    with pytest.raises(pe.PeError) as e:
        pe.pe_coarsen(desc, 1, 1, 1, 1, 1)
    assert e.value.code == pe.PE_ERR_CYCLE
