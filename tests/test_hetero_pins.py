"""Heterogeneous machines (footnote of Section III: the duration of an operation gets a machine index):
the oracle's extension pinned by what the mathematics fixes.  CPU only."""
import copy
import itertools

import numpy as np
import pytest

from oracle import pe_oracle as orc
from paper_2503_09357_b200 import workloads as wl
from tests import checkers as ck


def with_table(w, table):
    w = copy.copy(w)
    w.dur_by_machine = np.asarray(table, np.int32)
    return w


def test_flow_shop_closed_form_with_one_slow_stage():
    """S stages in a row, stage s on machine s, M identical jobs, no communication: the makespan of the
    permutation flow shop with identical jobs is sum_s f_s + (M - 1) max_s f_s, where f_s is what stage s
    costs ON ITS OWN machine; every other entry of the table is a decoy."""
    for S, M, slow in itertools.product((2, 3, 5), (1, 3, 6), (0, 1)):
        f = [3 + s for s in range(S)]
        f[slow] = 11
        ops = [(s, m) for s in range(S) for m in range(M)]
        idx = {sm: n for n, sm in enumerate(ops)}
        edges = [(idx[(s, m)], idx[(s + 1, m)]) for s in range(S - 1) for m in range(M)]
        table = np.full((S * M, S), 1000, np.int32)              # decoys: a wrong lookup blows the makespan up
        for (s, m), n in idx.items():
            table[n, s] = f[s]
        w = with_table(ck.problem(S * M, edges, [999] * (S * M), S, comm=0), table)
        x = [s for s, m in ops]
        pi = [idx[(s, m)] for m in range(M) for s in range(S)]   # job by job: a topological order
        a, o = ck.columns([x], [pi], S * M)
        r = orc.evaluate(w, a, o)
        assert r["makespan"][0] == sum(f) + (M - 1) * max(f)
        assert r["busy"][:, 0].tolist() == [M * f[s] for s in range(S)]
        assert (r["finish"][:, 0] - r["start"][:, 0]).tolist() == [f[s] for m in range(M) for s in range(S)]


@pytest.mark.parametrize("config,kw", [(1, {}), (2, {}), (5, dict(V=256, D=8))])
def test_fixing_the_assignment_reduces_to_the_homogeneous_problem(config, kw):
    """For one candidate at a time, D^o_{i, x_i} is just a duration vector: the homogeneous evaluation with
    dur'[i] = table[i, x_i] (pinned on its own elsewhere) must give the same schedule."""
    w = wl.make_config(config, **kw)
    rs = np.random.RandomState(config)
    table = rs.randint(1, 30, (w.num_ops, w.num_devices)).astype(np.int32)
    K = 24
    assign, order = wl.make_candidates(w, K=K)
    got = orc.evaluate(with_table(w, table), assign, order)
    for c in range(K):
        w1 = copy.copy(w)
        w1.dur = table[np.arange(w.num_ops), assign[:, c]]
        ref = orc.evaluate(w1, assign[:, c:c + 1], order[:, c:c + 1])
        for key in ("start", "finish", "makespan", "busy", "peak_mem", "status"):
            assert np.array_equal(got[key][..., c], ref[key][..., 0]), (key, c)


def test_a_constant_table_changes_nothing_and_one_machine_is_a_prefix_sum():
    w = wl.make_config(1)
    assign, order = wl.make_candidates(w, K=16)
    same = with_table(w, np.repeat(np.asarray(w.dur)[:, None], w.num_devices, axis=1))
    a, b = orc.evaluate(w, assign, order), orc.evaluate(same, assign, order)
    for key in a:
        assert np.array_equal(a[key], b[key])
    rs = np.random.RandomState(3)
    V = 9
    one = with_table(ck.problem(V, [(i, i + 1) for i in range(V - 1)], [50] * V, 1), rs.randint(1, 9, (V, 1)))
    x, pi = [0] * V, list(range(V))
    a1, o1 = ck.columns([x], [pi], V)
    r = orc.evaluate(one, a1, o1)
    assert r["finish"][:, 0].tolist() == np.cumsum(one.dur_by_machine[:, 0]).tolist()


def test_constraints_hold_with_the_table():
    """Eq. 3 with D^o_{i, x_i}, Eqs. 7-8 and 11-13, checked by the independent constraint predicate on the
    explicit bounds, and tightness (no start can move one unit earlier)."""
    rs = np.random.RandomState(5)
    w = ck.problem(6, [(0, 2), (1, 2), (2, 3), (2, 4), (3, 5), (4, 5)], [7] * 6, 3, comm=2)
    w = with_table(w, rs.randint(1, 6, (6, 3)))
    w.assign_mode, w.group = "per_op", None
    assign, order = wl.make_candidates(w, K=40)
    r = orc.evaluate(w, assign, order)
    for c in range(40):
        x, pi, s, e = assign[:, c], order[:, c], r["start"][:, c], r["finish"][:, c]
        by_op_s = np.empty(6, np.int64); by_op_e = np.empty(6, np.int64)
        by_op_s[pi] = s; by_op_e[pi] = e
        assert (by_op_e - by_op_s == w.dur_by_machine[np.arange(6), x]).all()          # Eq. 3
        lbs = ck.lower_bounds(w, x, pi, by_op_s, by_op_e)
        assert all(by_op_s[i] == max(lbs[i]) for i in range(6))                        # feasible and left-shifted
