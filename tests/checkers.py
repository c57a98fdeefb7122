"""Independent checks of a schedule against the scheduling model's constraints.

Nothing here calls the oracle or the CUDA path: these functions restate the
constraints (Eqs. 3, 7-8, 11-13 and the memory chain of Eqs. 16-19) directly on
(x, pi, s, e), enumerate tiny instances exhaustively, or hand the explicit
disjunctive graph to a library shortest-path routine.
"""
import itertools
from types import SimpleNamespace

import numpy as np


def problem(V, edges, dur, D, comm=None, L=1, link_class=None, A=None, W=None, cap=None):
    """A small workload-like object from Python lists. `comm` is [E][L] or a scalar."""
    E = len(edges)
    src = np.array([a for a, _ in edges], dtype=np.int32).reshape(E)
    dst = np.array([b for _, b in edges], dtype=np.int32).reshape(E)
    if comm is None:
        comm = 0
    comm = np.broadcast_to(np.asarray(comm, dtype=np.int32).reshape(-1, L) if np.ndim(comm) else
                           np.full((E, L), comm, dtype=np.int32), (E, L)).copy()
    return SimpleNamespace(
        num_ops=V, num_devices=D, num_link_classes=L, edge_src=src, edge_dst=dst,
        dur=np.asarray(dur, dtype=np.int32), mem_delta=np.zeros(V, np.int32) if A is None else np.asarray(A, np.int32),
        mem_weight=None if W is None else np.asarray(W, np.int32), comm=comm,
        link_class=None if link_class is None else np.asarray(link_class, np.uint8),
        mem_capacity=None if cap is None else np.asarray(cap, np.int32), num_edges=E)


def columns(xs, pis, V):
    """Stack per-candidate lists into candidate-interleaved [V, K] arrays."""
    assign = np.array(xs, dtype=np.uint8).T.copy().reshape(V, len(xs))
    order = np.array(pis, dtype=np.uint16).T.copy().reshape(V, len(pis))
    return assign, order


def edge_delay(w, b, jp, ji):
    """Delay of edge number b when its endpoints run on machines jp -> ji."""
    if jp == ji:
        return 0
    cls = 0 if w.link_class is None else int(w.link_class[jp, ji])
    return 0 if cls == 0xFF else int(w.comm[b, cls])


def lower_bounds(w, x, pi, s, e):
    """For every op, the list of lower bounds the constraints put on its start time."""
    V = w.num_ops
    pos = np.empty(V, dtype=np.int64)
    pos[np.asarray(pi)] = np.arange(V)
    lbs = [[0] for _ in range(V)]                               # machines are free from time 0
    for b in range(w.num_edges):                                # Eqs. 11-13
        p, i = int(w.edge_src[b]), int(w.edge_dst[b])
        lbs[i].append(int(e[p]) + edge_delay(w, b, int(x[p]), int(x[i])))
    for a in range(V):                                          # Eqs. 7-8: y from pi, same machine
        for c in range(V):
            if a != c and x[a] == x[c] and pos[a] < pos[c]:
                lbs[c].append(int(e[a]))
    return lbs


def check_feasible(w, x, pi, s, e):
    V = w.num_ops
    assert sorted(int(v) for v in pi) == list(range(V)), "pi must be a permutation"
    for i in range(V):
        assert int(e[i]) - int(s[i]) == int(w.dur[i]), f"Eq. 3 fails at op {i}"
    for i, lb in enumerate(lower_bounds(w, x, pi, s, e)):
        assert int(s[i]) >= max(lb), f"op {i} starts at {s[i]} before bound {max(lb)}"


def check_left_shifted(w, x, pi, s, e):
    """Every start time is tight: lowering any s_i by one breaks a constraint."""
    for i, lb in enumerate(lower_bounds(w, x, pi, s, e)):
        assert int(s[i]) == max(lb), f"op {i} could start at {max(lb)} but starts at {s[i]}"


def machine_memory(w, x, pi):
    """Peak level per machine from its own op sequence (Eqs. 16-19), empty prefix included."""
    D = w.num_devices
    lvl = np.zeros(D, dtype=np.int64)
    if w.mem_weight is not None:
        for i in range(w.num_ops):
            lvl[x[i]] += int(w.mem_weight[i])
    peak = lvl.copy()
    for i in pi:
        lvl[x[i]] += int(w.mem_delta[i])
        peak[x[i]] = max(peak[x[i]], lvl[x[i]])
    return peak


def topological_orders(V, edges):
    """All topological orders of a small DAG."""
    preds = [set() for _ in range(V)]
    for a, b in edges:
        preds[b].add(a)
    out = []

    def rec(prefix, placed):
        if len(prefix) == V:
            out.append(list(prefix))
            return
        for i in range(V):
            if i not in placed and preds[i] <= placed:
                prefix.append(i); placed.add(i)
                rec(prefix, placed)
                prefix.pop(); placed.remove(i)

    rec([], set())
    return out


def all_assignments(V, D):
    return [list(t) for t in itertools.product(range(D), repeat=V)]


def min_makespan_over_start_vectors(w, horizon):
    """min over x and all integer start vectors in [0, horizon]^V of the makespan of the
    schedules that satisfy Eqs. 3, 7 (for some order), 11-13.  Exponential: tiny cases only."""
    V, D = w.num_ops, w.num_devices
    dur = [int(d) for d in w.dur]
    best = None
    for x in all_assignments(V, D):
        for s in itertools.product(range(horizon + 1), repeat=V):
            e = [s[i] + dur[i] for i in range(V)]
            z = max(e)
            if best is not None and z >= best:
                continue
            ok = True
            for b in range(w.num_edges):
                p, i = int(w.edge_src[b]), int(w.edge_dst[b])
                if s[i] < e[p] + edge_delay(w, b, x[p], x[i]):
                    ok = False
                    break
            if not ok:
                continue
            for a in range(V):
                for c in range(a + 1, V):
                    if x[a] == x[c] and not (e[a] <= s[c] or e[c] <= s[a]):
                        ok = False
                        break
                if not ok:
                    break
            if ok:
                best = z
    return best


def longest_path_starts(w, x, pi):
    """Start times as longest-path distances in the explicit disjunctive graph
    H(x, pi) = B joined with consecutive same-machine pairs of pi, computed by scipy's
    Bellman-Ford on negated weights.  A source node reaches every op with weight -1
    (so that no stored weight is zero); the 1 is taken off again at the end."""
    from scipy.sparse import csr_matrix
    from scipy.sparse.csgraph import bellman_ford
    V = w.num_ops
    weights = {}

    def add(a, b, wt):
        weights[(a, b)] = max(weights.get((a, b), 0), wt)

    for b in range(w.num_edges):
        p, i = int(w.edge_src[b]), int(w.edge_dst[b])
        add(p, i, int(w.dur[p]) + edge_delay(w, b, int(x[p]), int(x[i])))
    last = {}
    for i in pi:
        j = int(x[i])
        if j in last:
            add(last[j], int(i), int(w.dur[last[j]]))
        last[j] = int(i)
    rows, cols, vals = [], [], []
    for (a, b), wt in weights.items():
        assert wt > 0, "library route needs positive durations"
        rows.append(a); cols.append(b); vals.append(-float(wt))
    for i in range(V):
        rows.append(V); cols.append(i); vals.append(-1.0)
    g = csr_matrix((vals, (rows, cols)), shape=(V + 1, V + 1))
    dist = bellman_ford(g, directed=True, indices=V)
    return (-dist[:V] - 1).astype(np.int64)


def critical_path(w):
    """Longest dur-weighted path of G_m (no communication), by the same library routine."""
    from scipy.sparse import csr_matrix
    from scipy.sparse.csgraph import bellman_ford
    V = w.num_ops
    rows = [int(a) for a in w.edge_src] + [V] * V
    cols = [int(b) for b in w.edge_dst] + list(range(V))
    vals = [-float(w.dur[int(a)]) for a in w.edge_src] + [-1.0] * V
    agg = {}
    for r, c, v in zip(rows, cols, vals):
        agg[(r, c)] = min(agg.get((r, c), 0.0), v)
    g = csr_matrix((list(agg.values()), ([k[0] for k in agg], [k[1] for k in agg])), shape=(V + 1, V + 1))
    dist = bellman_ford(g, directed=True, indices=V)
    starts = -dist[:V] - 1
    return int(np.max(starts + np.asarray(w.dur)))


def exclusive_channel_starts(w, x, pi):
    """Start times under exclusive channels (Eqs. 11-15) as longest-path distances in the explicit
    constraint graph, by scipy's Bellman-Ford on negated weights.  Nodes: one per operation (its start)
    and one per cross-machine edge with a channel (the start c of its transfer).  Arcs:
      machine chain (Eqs. 7-8)   s_next >= s_prev + dur_prev      for consecutive same-machine ops of pi
      Eq. 13                     c_b    >= s_p + dur_p
      Eqs. 11-12                 s_i    >= c_b + D^c_b
      Eq. 14                     c_b'   >= c_b + D^c_b             for consecutive transfers of a channel,
                                 sequenced by the position of the receiving op in pi, then by edge number
      same machine / no channel  s_i    >= s_p + dur_p
    Needs durations and communication times >= 1 (the sparse matrix drops zero weights)."""
    from scipy.sparse import csr_matrix
    from scipy.sparse.csgraph import bellman_ford
    V, E = w.num_ops, w.num_edges
    pos = np.empty(V, dtype=np.int64)
    pos[np.asarray(pi)] = np.arange(V)
    weights = {}

    def add(a, b, wt):
        assert wt > 0
        weights[(a, b)] = max(weights.get((a, b), 0), wt)

    last = {}
    for i in pi:
        j = int(x[i])
        if j in last:
            add(last[j], int(i), int(w.dur[last[j]]))
        last[j] = int(i)
    per_channel = {}
    for b in range(E):
        p, i = int(w.edge_src[b]), int(w.edge_dst[b])
        jp, ji = int(x[p]), int(x[i])
        cls = 0 if w.link_class is None else int(w.link_class[jp, ji])
        if jp == ji or cls == 0xFF:
            add(p, i, int(w.dur[p]))
            continue
        t = V + 1 + b                                      # node of this edge's transfer
        add(p, t, int(w.dur[p]))
        add(t, i, int(w.comm[b, cls]))
        per_channel.setdefault((jp, ji), []).append((int(pos[i]), b, int(w.comm[b, cls])))
    for seq in per_channel.values():
        seq.sort()
        for (_, b0, c0), (_, b1, _) in zip(seq, seq[1:]):
            add(V + 1 + b0, V + 1 + b1, c0)
    n = V + 1 + E
    rows = [a for a, _ in weights] + [V] * V
    cols = [b for _, b in weights] + list(range(V))
    vals = [-float(v) for v in weights.values()] + [-1.0] * V
    g = csr_matrix((vals, (rows, cols)), shape=(n, n))
    dist = bellman_ford(g, directed=True, indices=V)
    return (-dist[:V] - 1).astype(np.int64)
