"""Oracle of the graph-coarsening heuristic (Section IV, Algorithm 1).  TEST INFRASTRUCTURE ONLY:
plain Python sets and loops, slow on purpose, used by tests/ to check the library's pe_coarsen.
It shares no code with the library.

What the paper fixes, and how it is read here where it is silent or garbled:

* Algorithm 1 alternates two loops until the graph has at most N nodes: merges of pairs joined by an
  edge (GetCandidateEdge), then merges of pairs not joined by an edge (GetCandidateNonEdge).  The
  printed condition of the second loop repeats the first loop's test; it is read as "while
  GetCandidateNonEdge returns a pair".  The printed outer loop has no exit; it ends here when
  |I| <= N or when a whole pass merged nothing.
* Before candidates are looked for, the topologically redundant edges
  {(i1, i2) in B : exists i3 with (i1, i3) in B and (i3, i2) in B} are set aside (Section IV gives
  exactly this two-hop definition); the merge itself works on the full edge set.
* GetCandidateEdge: an edge (u, v) of the remaining graph whose head v has a single input and whose
  tail u has a single output, with the merged duration and memory requirement within the thresholds.
  Such a merge cannot create a cycle and leaves the length of the critical path unchanged
  (Section IV calls these merges safe).
* GetCandidateNonEdge: two nodes with no directed path between them in either direction (so that the
  merge cannot create a cycle; the paper only says "without a direct edge"), within its own,
  stricter, thresholds.
* Which of several candidates comes first is not stated.  Here: the pair with the smallest merged
  duration, ties to the smallest (u, v) by node label, where a merged node carries the smallest
  original operator id among its members as its label.
* MergeNodes: duration, A and W of the new node are the sums over its members (Section IV); it
  inherits every edge of either member to or from a third node; edges that become parallel are
  combined into one whose communication duration is, per link class, the larger of the two: with
  communication as a delay (Eqs. 11-13) the merged operation can start once the later of the two
  transfers has arrived.  The memory requirement tested against the thresholds is not defined in the paper;
  here it is W + max(A, 0) summed over the members.
"""
from types import SimpleNamespace

import numpy as np


def _two_hop_redundant(succ):
    """Edges (a, b) for which some c has (a, c) and (c, b)."""
    red = set()
    for a, outs in succ.items():
        for c in outs:
            for b in succ[c]:
                if b in outs:
                    red.add((a, b))
    return red


def _reachable(succ, nodes):
    """reach[u] = set of nodes reachable from u by one or more edges."""
    reach = {}

    def visit(u):
        if u in reach:
            return reach[u]
        r = set()
        for v in succ[u]:
            r.add(v)
            r |= visit(v)
        reach[u] = r
        return r

    for u in nodes:
        visit(u)
    return reach


def coarsen(w, N, max_dur_edge, max_mem_edge, max_dur_nonedge, max_mem_nonedge):
    """Run Algorithm 1 on workload-like `w` (num_ops, edge_src, edge_dst, dur, mem_delta, mem_weight,
    comm [E][L], num_link_classes).  Returns a SimpleNamespace with
      op_map [V]   coarse node of every original operator (coarse nodes numbered by smallest member),
      num_ops, edge_src, edge_dst (sorted by (src, dst)), dur, mem_delta, mem_weight, comm [E'][L],
      merges       the list of (u, v, kind) merges in the order they happened (labels, 'edge'/'nonedge')."""
    V, L = int(w.num_ops), int(w.num_link_classes)
    dur = {i: int(w.dur[i]) for i in range(V)}
    A = {i: int(w.mem_delta[i]) for i in range(V)}
    W = {i: 0 if w.mem_weight is None else int(w.mem_weight[i]) for i in range(V)}
    req = {i: W[i] + max(A[i], 0) for i in range(V)}          # memory requirement tested against thresholds
    members = {i: [i] for i in range(V)}
    succ = {i: {} for i in range(V)}                          # succ[u][v] = per-class communication durations
    pred = {i: set() for i in range(V)}
    for b in range(len(w.edge_src)):
        u, v = int(w.edge_src[b]), int(w.edge_dst[b])
        c = [int(x) for x in np.asarray(w.comm[b]).reshape(L)]
        if v in succ[u]:
            succ[u][v] = [max(a, b_) for a, b_ in zip(succ[u][v], c)]   # parallel input edges are combined too
        else:
            succ[u][v] = c
        pred[v].add(u)
    merges = []

    def candidate_edge():
        red = _two_hop_redundant(succ)
        best = None
        for u in succ:
            outs = [v for v in succ[u] if (u, v) not in red]
            if len(outs) != 1:
                continue                                      # the tail must have a single output
            v = outs[0]
            ins = [p for p in pred[v] if (p, v) not in red]
            if len(ins) != 1:
                continue                                      # the head must have a single input
            if dur[u] + dur[v] > max_dur_edge or req[u] + req[v] > max_mem_edge:
                continue
            key = (dur[u] + dur[v], u, v)
            if best is None or key < best:
                best = key
        return None if best is None else (best[1], best[2])

    def candidate_nonedge():
        reach = _reachable(succ, list(succ))
        best = None
        nodes = sorted(succ)
        for a_i, u in enumerate(nodes):
            for v in nodes[a_i + 1:]:
                if v in reach[u] or u in reach[v]:
                    continue
                if dur[u] + dur[v] > max_dur_nonedge or req[u] + req[v] > max_mem_nonedge:
                    continue
                key = (dur[u] + dur[v], u, v)
                if best is None or key < best:
                    best = key
        return None if best is None else (best[1], best[2])

    def merge(u, v):
        """v is folded into u (u < v or (u, v) an edge); the node keeps the smaller label."""
        keep, gone = (u, v) if u < v else (v, u)
        succ[u].pop(v, None); pred[v].discard(u)
        succ[v].pop(u, None); pred[u].discard(v)
        for x, c in list(succ[gone].items()):                  # outgoing edges of the node that disappears
            pred[x].discard(gone)
            if x in succ[keep]:
                succ[keep][x] = [max(a, b_) for a, b_ in zip(succ[keep][x], c)]
            else:
                succ[keep][x] = c
            pred[x].add(keep)
        for p in list(pred[gone]):                             # incoming edges
            c = succ[p].pop(gone)
            if keep in succ[p]:
                succ[p][keep] = [max(a, b_) for a, b_ in zip(succ[p][keep], c)]
            else:
                succ[p][keep] = c
            pred[keep].add(p)
        del succ[gone], pred[gone]
        dur[keep] += dur.pop(gone); A[keep] += A.pop(gone); W[keep] += W.pop(gone); req[keep] += req.pop(gone)
        members[keep] = sorted(members[keep] + members.pop(gone))

    while len(succ) > N:
        merged_this_pass = 0
        while len(succ) > N:                                   # loop over to merge edges
            c = candidate_edge()
            if c is None:
                break
            merge(*c); merges.append((min(c), max(c), "edge")); merged_this_pass += 1
        while len(succ) > N:                                   # loop over to merge non-edges
            c = candidate_nonedge()
            if c is None:
                break
            merge(*c); merges.append((min(c), max(c), "nonedge")); merged_this_pass += 1
        if merged_this_pass == 0:
            break

    labels = sorted(succ)                                      # label = smallest member: this is the numbering
    index = {lab: n for n, lab in enumerate(labels)}
    op_map = np.empty(V, np.int32)
    for lab in labels:
        for i in members[lab]:
            op_map[i] = index[lab]
    edges = sorted((index[u], index[v], tuple(c)) for u in succ for v, c in succ[u].items())
    return SimpleNamespace(
        op_map=op_map, num_ops=len(labels),
        edge_src=np.array([e[0] for e in edges], np.int32), edge_dst=np.array([e[1] for e in edges], np.int32),
        comm=np.array([e[2] for e in edges], np.int32).reshape(len(edges), L),
        dur=np.array([dur[l] for l in labels], np.int32), mem_delta=np.array([A[l] for l in labels], np.int32),
        mem_weight=np.array([W[l] for l in labels], np.int32), num_link_classes=L, merges=merges)
