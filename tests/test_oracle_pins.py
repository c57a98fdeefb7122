"""Pins for the CPU oracle: it is checked against the constraints themselves, exhaustive
enumeration, closed forms, a library longest-path routine and hand-computed fixtures,
never against itself or the CUDA path."""
import itertools
import os

import numpy as np
import pytest

from oracle import pe_oracle as orc
from paper_2503_09357_b200 import workloads as wl
from tests import checkers as ck

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def run(w, xs, pis, flags=0):
    assign, order = ck.columns(xs, pis, w.num_ops)
    return orc.evaluate(w, assign, order, flags=flags)


def by_op(out, pis, c):
    """by-position outputs of candidate c re-indexed by operation."""
    V = len(pis[c])
    s = np.empty(V, np.int64); e = np.empty(V, np.int64)
    s[np.asarray(pis[c])] = out["start"][:, c]
    e[np.asarray(pis[c])] = out["finish"][:, c]
    return s, e


TINY = [
    # (V, edges, dur, comm per edge)
    (4, [(0, 1), (0, 2), (1, 3), (2, 3)], [1, 2, 1, 1], [1, 2, 1, 1]),          # diamond
    (4, [(0, 2), (1, 2), (1, 3)], [2, 1, 1, 2], [1, 1, 2]),                      # two sources
    (5, [(0, 1), (1, 2), (0, 3), (3, 4), (2, 4)], [1, 1, 2, 1, 1], [2, 1, 1, 1, 1]),
    (5, [(0, 4), (1, 4), (2, 4), (3, 4)], [1, 2, 1, 1, 1], [1, 1, 3, 1]),        # fan-in
    (4, [], [1, 2, 1, 2], []),                                                   # no edges
]


# ---- P1 (i): every assignment x every topological order, checked by the constraint predicate ----
@pytest.mark.parametrize("case", range(len(TINY)))
@pytest.mark.parametrize("D", [1, 2, 3])
def test_exhaustive_candidates_satisfy_constraints_and_are_left_shifted(case, D):
    V, edges, dur, comm = TINY[case]
    A = [((3 * i) % 5) - 2 for i in range(V)]
    w = ck.problem(V, edges, dur, D, comm=np.array(comm, np.int32).reshape(-1, 1) if comm else None, A=A)
    xs, pis = [], []
    for x in ck.all_assignments(V, D):
        for pi in ck.topological_orders(V, edges):
            xs.append(x); pis.append(pi)
    out = run(w, xs, pis)
    assert not out["status"].any()
    for c in range(len(xs)):
        s, e = by_op(out, pis, c)
        ck.check_feasible(w, xs[c], pis[c], s, e)
        ck.check_left_shifted(w, xs[c], pis[c], s, e)
        assert out["makespan"][c] == e.max()
        assert np.array_equal(out["peak_mem"][:, c], ck.machine_memory(w, xs[c], pis[c]))
        for j in range(D):
            assert out["busy"][j, c] == sum(dur[i] for i in range(V) if xs[c][i] == j)


# ---- P1 (ii): the best candidate equals the best of ALL feasible integer schedules ----
@pytest.mark.parametrize("case", [0, 1, 4])
def test_best_candidate_matches_brute_force_over_start_vectors(case):
    V, edges, dur, comm = TINY[case]
    D = 2
    w = ck.problem(V, edges, dur, D, comm=np.array(comm, np.int32).reshape(-1, 1) if comm else None)
    xs, pis = [], []
    for x in ck.all_assignments(V, D):
        for pi in ck.topological_orders(V, edges):
            xs.append(x); pis.append(pi)
    out = run(w, xs, pis)
    assert int(out["makespan"].min()) == ck.min_makespan_over_start_vectors(w, horizon=sum(dur) - min(dur))


# ---- P2: closed forms for a uniform pipeline (stage s on machine s) ----
def pipeline_orders(S, M):
    """Per-machine GPipe and 1F1B sequences merged into global topological orders."""
    F = lambda s, m: s * M + m
    B = lambda s, m: S * M + s * M + m
    gpipe = [[F(s, m) for m in range(M)] + [B(s, m) for m in range(M)] for s in range(S)]
    f1b1 = []
    for s in range(S):
        warm = min(S - s, M)
        seq = [F(s, m) for m in range(warm)]
        nf, nb = warm, 0
        while nb < M:
            seq.append(B(s, nb)); nb += 1
            if nf < M:
                seq.append(F(s, nf)); nf += 1
        f1b1.append(seq)
    return gpipe, f1b1


def merge_device_sequences(w, seqs):
    """A topological order of B joined with the per-machine chains (plain Kahn, smallest id first)."""
    V = w.num_ops
    succ = [[] for _ in range(V)]
    indeg = [0] * V
    for a, b in zip(w.edge_src.tolist(), w.edge_dst.tolist()):
        succ[a].append(b); indeg[b] += 1
    for seq in seqs:
        for a, b in zip(seq[:-1], seq[1:]):
            succ[a].append(b); indeg[b] += 1
    ready = sorted(i for i in range(V) if indeg[i] == 0)
    pi = []
    while ready:
        i = ready.pop(0)
        pi.append(i)
        for t in succ[i]:
            indeg[t] -= 1
            if indeg[t] == 0:
                ready.append(t); ready.sort()
    assert len(pi) == V
    return pi


@pytest.mark.parametrize("S,M", [(1, 1), (1, 5), (2, 2), (3, 4), (4, 8), (4, 2), (6, 11)])
@pytest.mark.parametrize("f,b", [(1, 1), (2, 4), (3, 7), (5, 2)])
@pytest.mark.parametrize("c", [0, 1, 3])
def test_uniform_pipeline_closed_forms(S, M, f, b, c):
    w = wl.tiny_pipeline(S=S, M=M, f=f, b=b, c=c, capacity=M)
    x = [int(g) for g in w.group]                       # stage s on machine s
    gpipe, f1b1 = pipeline_orders(S, M)
    pis = [merge_device_sequences(w, gpipe), merge_device_sequences(w, f1b1)]
    out = run(w, [x, x], pis)
    assert out["makespan"][0] == (M + S - 1) * (f + b) + 2 * (S - 1) * c      # GPipe, comm on every hop
    if c == 0:
        assert out["makespan"][1] == (M + S - 1) * (f + b)                    # 1F1B, zero comm
    for s in range(S):
        assert out["busy"][s, 0] == M * (f + b) and out["busy"][s, 1] == M * (f + b)
        assert out["peak_mem"][s, 0] == M                                     # GPipe holds every microbatch
        assert out["peak_mem"][s, 1] == min(S - s, M)                         # 1F1B holds the warm-up depth
    assert out["status"][0] == 0                                              # capacity M is just enough
    w.mem_capacity[:] = M - 1
    out = run(w, [x, x], pis)
    assert out["status"][0] == orc.STATUS_MEM_EXCEEDED


def test_config1_identity_placement_gpipe_is_72():
    w = wl.make_config(1)
    x = [int(g) for g in w.group]
    gpipe, _ = pipeline_orders(4, 8)
    out = run(w, [x], [merge_device_sequences(w, gpipe)])
    assert out["makespan"][0] == 72 and out["status"][0] == 0 and (out["peak_mem"][:, 0] == 8).all()


# ---- P3: a single machine is a prefix sum ----
@pytest.mark.parametrize("config", [1, 2, 3])
def test_single_machine_is_prefix_sums(config):
    w = wl.make_config(config)
    K = 16
    _, order = wl.make_candidates(w, K=K)
    assign = np.zeros((w.num_ops, K), np.uint8)
    w.mem_weight = (np.arange(w.num_ops) % 3).astype(np.int32)
    out = orc.evaluate(w, assign, order)
    dur = w.dur.astype(np.int64)
    for c in range(K):
        pi = order[:, c].astype(np.int64)
        ends = np.cumsum(dur[pi])
        assert np.array_equal(out["finish"][:, c], ends)
        assert np.array_equal(out["start"][:, c], ends - dur[pi])
        assert out["makespan"][c] == dur.sum() and out["busy"][0, c] == dur.sum()
        assert (out["busy"][1:, c] == 0).all() and (out["peak_mem"][1:, c] == 0).all()
        wsum = int(w.mem_weight.sum())
        assert out["peak_mem"][0, c] == wsum + max(0, int(np.cumsum(w.mem_delta[pi].astype(np.int64)).max()))


# ---- P4: bounds that hold for every candidate ----
@pytest.mark.parametrize("config,kw", [(1, {}), (2, {}), (3, {}), (4, {}), (5, dict(V=256, D=8)), (5, dict(V=1024, D=64))])
def test_bounds_on_random_candidates(config, kw):
    w = wl.make_config(config, **kw)
    K = 64
    assign, order = wl.make_candidates(w, K=K)
    out = orc.evaluate(w, assign, order)
    total = int(w.dur.astype(np.int64).sum())
    cp = ck.critical_path(w)
    upper = total + int(w.comm.max(axis=1).astype(np.int64).sum())
    assert (out["status"] & 3 == 0).all()
    assert (out["start"] >= 0).all()
    assert (out["makespan"] >= cp).all()
    assert (out["makespan"] >= -(-total // w.num_devices)).all()
    assert (out["makespan"] >= out["busy"].max(axis=0)).all()
    assert (out["makespan"] <= upper).all()
    assert (out["busy"].sum(axis=0) == total).all()
    assert np.array_equal(out["makespan"], out["finish"].max(axis=0))


# ---- P5: one op per machine, zero communication: ASAP times, makespan = critical path ----
def test_one_op_per_machine_gives_critical_path():
    w = wl.random_layered(V=144, D=144)
    w.comm[:] = 0
    K = 8
    _, order = wl.make_candidates(w, K=K)
    assign = np.repeat(np.arange(144, dtype=np.uint8)[:, None], K, axis=1)
    out = orc.evaluate(w, assign, order, flags=orc.TIMES_BY_OP)
    asap = ck.longest_path_starts(w, list(range(144)), list(range(144)))   # machine chains are empty here
    for c in range(K):
        assert np.array_equal(out["start"][:, c], asap)
    assert (out["makespan"] == ck.critical_path(w)).all()


# ---- P7: library longest path on the explicit disjunctive graph ----
@pytest.mark.parametrize("config,kw", [(1, {}), (2, {}), (3, {}), (4, {}), (5, dict(V=256, D=8)), (5, dict(V=1024, D=64))])
def test_longest_path_library_agrees(config, kw):
    w = wl.make_config(config, **kw)
    K = 6
    assign, order = wl.make_candidates(w, K=K)
    out = orc.evaluate(w, assign, order, flags=orc.TIMES_BY_OP)
    for c in range(K):
        s = ck.longest_path_starts(w, assign[:, c].astype(int), order[:, c].astype(int))
        assert np.array_equal(out["start"][:, c], s)
        assert np.array_equal(out["finish"][:, c], s + w.dur)
        assert np.array_equal(out["peak_mem"][:, c], ck.machine_memory(w, assign[:, c].astype(int), order[:, c].astype(int)))


# ---- P6: metamorphic relations ----
def test_same_machine_sequences_give_same_schedule():
    w = wl.make_config(1)
    K = 32
    assign, order = wl.make_candidates(w, K=K)
    out = orc.evaluate(w, assign, order, flags=orc.TIMES_BY_OP)
    # re-merge each candidate's per-machine sequences into a different global order
    pis2 = []
    for c in range(K):
        seqs = [[int(i) for i in order[:, c] if assign[i, c] == j] for j in range(w.num_devices)]
        pis2.append(merge_device_sequences(w, seqs))
    order2 = np.array(pis2, dtype=np.uint16).T.copy()
    assert (order2 != order).any()
    out2 = orc.evaluate(w, assign, order2, flags=orc.TIMES_BY_OP)
    for key in ("start", "finish", "makespan", "busy", "peak_mem", "status"):
        assert np.array_equal(out[key], out2[key]), key


def test_relabelling_machines_within_a_node_permutes_outputs():
    w = wl.make_config(3)
    K = 16
    assign, order = wl.make_candidates(w, K=K)
    perm = np.array([3, 0, 1, 2, 7, 6, 5, 4, 8, 10, 9, 11, 15, 12, 13, 14], dtype=np.uint8)   # keeps nodes of 8
    out = orc.evaluate(w, assign, order)
    out2 = orc.evaluate(w, perm[assign], order)
    assert np.array_equal(out["start"], out2["start"]) and np.array_equal(out["makespan"], out2["makespan"])
    assert np.array_equal(out["busy"], out2["busy"][perm]) and np.array_equal(out["peak_mem"], out2["peak_mem"][perm])


def test_scaling_durations_scales_times():
    w = wl.make_config(4)
    K = 8
    assign, order = wl.make_candidates(w, K=K)
    out = orc.evaluate(w, assign, order)
    w.dur *= 3; w.comm *= 3
    out3 = orc.evaluate(w, assign, order)
    for key in ("start", "finish", "makespan", "busy"):
        assert np.array_equal(out3[key], 3 * out[key])
    assert np.array_equal(out3["peak_mem"], out["peak_mem"])


def test_layout_flags_are_re_indexings():
    w = wl.make_config(5, V=256, D=8)
    K = 32
    assign, order = wl.make_candidates(w, K=K)
    a = orc.evaluate(w, assign, order)
    b = orc.evaluate(w, assign, order, flags=orc.TIMES_BY_OP)
    c = orc.evaluate(w, wl.assign_by_pos(assign, order), order, flags=orc.ASSIGN_BY_POS)
    cols = np.arange(K)[None, :]
    assert np.array_equal(b["start"][order.astype(np.int64), cols], a["start"])
    assert np.array_equal(b["finish"][order.astype(np.int64), cols], a["finish"])
    for key in ("start", "finish", "makespan", "busy", "peak_mem", "status"):
        assert np.array_equal(a[key], c[key]), key


# ---- P8: status bits on hand-built candidates ----
def test_status_bits():
    edges = [(0, 1), (1, 2)]
    w = ck.problem(3, edges, [1, 1, 1], 2, comm=1, A=[2, 1, -3], cap=[3, 3])
    ok = run(w, [[0, 0, 0]], [[0, 1, 2]])
    assert ok["status"][0] == 0 and ok["peak_mem"][0, 0] == 3
    w.mem_capacity[0] = 2                                                    # capacity = peak - 1
    assert run(w, [[0, 0, 0]], [[0, 1, 2]])["status"][0] == orc.STATUS_MEM_EXCEEDED
    w.mem_capacity[0] = 3
    assert run(w, [[0, 0, 0]], [[1, 0, 2]])["status"][0] & orc.STATUS_ORDER_INVALID     # dependent pair swapped
    assert run(w, [[0, 0, 0]], [[0, 0, 2]])["status"][0] & orc.STATUS_ORDER_INVALID     # duplicate
    assert run(w, [[0, 0, 0]], [[0, 1, 3]])["status"][0] & orc.STATUS_ORDER_INVALID     # id out of range
    assert run(w, [[0, 2, 0]], [[0, 1, 2]])["status"][0] & orc.STATUS_ASSIGN_RANGE      # machine id = D
    w.link_class = np.array([[0, 0xFF], [0, 0]], np.uint8)
    assert run(w, [[0, 1, 1]], [[0, 1, 2]])["status"][0] == orc.STATUS_NO_CHANNEL       # 0 -> 1 has no channel
    assert run(w, [[1, 0, 0]], [[0, 1, 2]])["status"][0] == 0                           # 1 -> 0 has one


def test_link_class_direction_and_zero_delay_on_one_machine():
    # one edge 0 -> 1; class of (machine of 0 -> machine of 1); two classes with costs 5 and 9
    w = ck.problem(2, [(0, 1)], [2, 3], 2, comm=[[5, 9]], L=2, link_class=[[0, 1], [0, 0]])
    out = run(w, [[0, 1], [1, 0], [0, 0], [1, 1]], [[0, 1]] * 4)
    assert out["start"][1].tolist() == [2 + 9, 2 + 5, 2, 2]


def test_zero_duration_ops_share_an_instant():
    w = ck.problem(3, [(0, 2)], [0, 0, 4], 1)
    out = run(w, [[0, 0, 0]], [[0, 1, 2]])
    assert out["start"][:, 0].tolist() == [0, 0, 0] and out["makespan"][0] == 4


def test_weights_raise_the_initial_level():
    w = ck.problem(3, [], [1, 1, 1], 2, A=[1, -2, 1], W=[10, 20, 5])
    out = run(w, [[0, 1, 0]], [[0, 1, 2]])
    assert out["peak_mem"][:, 0].tolist() == [15 + 2, 20]           # machine 1 only releases: peak is its initial level


# ---- golden fixtures ----
def _ints(s):
    return [int(t) for t in s.split()]


def test_golden_worked_example():
    edges, comm = [(0, 2), (1, 2), (0, 3), (2, 4), (3, 4)], [[2], [1], [5], [3], [1]]
    w = ck.problem(5, edges, [3, 2, 4, 1, 2], 2, comm=comm, A=[2, 1, -1, 3, -2], cap=[4, 3])
    rows = [l for l in open(os.path.join(GOLDEN, "worked_example_two_machines.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for line in rows:
        x, pi, s, e, z, busy, peak, status = [_ints(f) for f in line.split("|")]
        out = run(w, [x], [pi], flags=orc.TIMES_BY_OP)
        assert out["start"][:, 0].tolist() == s and out["finish"][:, 0].tolist() == e
        assert out["makespan"][0] == z[0] and out["busy"][:, 0].tolist() == busy
        assert out["peak_mem"][:, 0].tolist() == peak and out["status"][0] == status[0]


def test_golden_pp2_bidirectional_has_zero_bubble():
    w = ck.problem(8, [(0, 1), (1, 2), (2, 3), (4, 5), (5, 6), (6, 7)], [1, 1, 2, 2, 1, 1, 2, 2], 2)
    row = [l for l in open(os.path.join(GOLDEN, "bidirectional_pp2_zero_bubble.txt")) if l.strip() and l[0] != "#"][0]
    x, pi, z, busy = [_ints(f) for f in row.split("|")]
    out = run(w, [x], [pi])
    assert out["makespan"][0] == z[0] and out["busy"][:, 0].tolist() == busy
    assert (out["makespan"][0] - out["busy"][:, 0] == 0).all()       # bubble (PP/2 - 1) = 0 at PP = 2


# ---- mutation check: the pins are sharp enough to catch a wrong oracle ----
def test_pins_reject_plausible_mistakes():
    """The same checks fail on schedules with a dropped comm term or a transposed link class."""
    w = ck.problem(2, [(0, 1)], [2, 3], 2, comm=[[5, 9]], L=2, link_class=[[0, 1], [0, 0]])
    s, e = np.array([0, 2 + 5]), np.array([2, 2 + 5 + 3])          # used class of (1 -> 0) for an edge going 0 -> 1
    with pytest.raises(AssertionError):
        ck.check_feasible(w, [0, 1], [0, 1], s, e)
    s, e = np.array([0, 12]), np.array([2, 15])                      # one unit late: feasible but not left-shifted
    ck.check_feasible(w, [0, 1], [0, 1], s, e)
    with pytest.raises(AssertionError):
        ck.check_left_shifted(w, [0, 1], [0, 1], s, e)


# ---- selection step: hand cases ----
def test_select_best_hand_cases():
    assert orc.select_best([5, 3, 9, 3], [0, 0, 0, 0]) == (1, 3, 4)                  # tie -> smallest index
    assert orc.select_best([5, 3, 9, 3], [0, 4, 0, 4]) == (0, 5, 2)                  # infeasible ones skipped
    assert orc.select_best([5, 3, 9, 3], [0, 4, 0, 4], reject_mask=3) == (1, 3, 4)   # only the validity bits reject
    assert orc.select_best([5, 3], [2, 1]) == (-1, 2 ** 31 - 1, 0)
    assert orc.select_best([], []) == (-1, 2 ** 31 - 1, 0)
    assert orc.select_best([7], [8], reject_mask=4) == (0, 7, 1)


def test_select_topk_hand_cases_and_library_sort():
    mk = [9, 4, 7, 4, 4, 12, 1]
    st = [0, 0, 2, 0, 4, 0, 1]
    assert orc.select_topk(mk, st, 3) == [0, 1, 3]                    # 4 (c=1), 4 (c=3), then 9; status != 0 never
    assert orc.select_topk(mk, st, 1) == [1]                          # ties go to the smallest index
    assert orc.select_topk(mk, st, 3, reject_mask=3) == [1, 3, 4]     # bit 4 tolerated: three 4s
    assert orc.select_topk(mk, st, 10) == [0, 1, 3, 5]                # fewer qualify than asked for
    assert orc.select_topk(mk, st, 0) == [] and orc.select_topk([], [], 3) == []
    assert orc.select_topk(mk, st, 1) == [orc.select_best(mk, st)[0]]
    rs = np.random.RandomState(11)
    for _ in range(20):                                               # against numpy's stable sort of (makespan, index)
        n = int(rs.randint(1, 60)); k = int(rs.randint(0, n + 3))
        mk = rs.randint(0, 8, n); st = rs.randint(0, 2, n) * rs.randint(1, 16, n)
        ok = np.flatnonzero(st == 0)
        want = sorted(ok[np.argsort(mk[ok], kind="stable")][:k].tolist())
        assert orc.select_topk(mk, st, k) == want
