"""Pins of the oracle's exclusive-channel communication model (flag COMM_EXCLUSIVE; Eqs. 11-15)."""
import numpy as np
import pytest

from oracle import pe_oracle as orc
from paper_2503_09357_b200 import workloads as wl
from tests import checkers as ck


def forward_pipeline(S, M, f, c):
    """S stages on S machines, M microbatches, forward ops only: F(s, m) -> F(s+1, m), transfer time c."""
    op = lambda s, m: s * M + m
    edges = [(op(s, m), op(s + 1, m)) for s in range(S - 1) for m in range(M)]
    w = ck.problem(S * M, edges, [f] * (S * M), S, comm=c)
    x = [s for s in range(S) for _ in range(M)]
    pi = [op(s, m) for m in range(M) for s in range(S)]          # microbatch after microbatch
    return w, x, pi


@pytest.mark.parametrize("S,M,f,c", [(2, 3, 2, 5), (4, 6, 3, 7), (3, 5, 4, 4), (4, 8, 5, 2), (5, 4, 1, 9), (2, 1, 3, 6)])
def test_forward_pipeline_runs_at_the_pace_of_its_slowest_resource(S, M, f, c):
    """A linear pipeline whose channels carry one transfer at a time behaves like a flow shop with the
    channels as extra machines: the last operation ends at S f + (S - 1) c + (M - 1) max(f, c).  With
    transfers as pure delays the channels never limit: S f + (S - 1) c + (M - 1) f."""
    w, x, pi = forward_pipeline(S, M, f, c)
    assign, order = ck.columns([x], [pi], w.num_ops)
    excl = orc.evaluate(w, assign, order, flags=orc.COMM_EXCLUSIVE)
    delay = orc.evaluate(w, assign, order)
    assert int(excl["makespan"][0]) == S * f + (S - 1) * c + (M - 1) * max(f, c)
    assert int(delay["makespan"][0]) == S * f + (S - 1) * c + (M - 1) * f
    assert (excl["start"] >= delay["start"]).all()
    if c <= f:
        assert np.array_equal(excl["start"], delay["start"])


@pytest.mark.parametrize("config,kw", [(1, {}), (2, {}), (4, {}), (5, dict(V=256, D=8))])
def test_library_longest_path_on_the_explicit_constraint_graph_agrees(config, kw):
    w = wl.make_config(config, **kw)
    w.comm = np.maximum(w.comm, 1)                                # the library route needs positive weights
    K = 6
    assign, order = wl.make_candidates(w, K=K)
    out = orc.evaluate(w, assign, order, flags=orc.COMM_EXCLUSIVE)
    differs = False
    for c in range(K):
        ref = ck.exclusive_channel_starts(w, assign[:, c], order[:, c].astype(np.int64))
        by_op = np.empty(w.num_ops, np.int64)
        by_op[order[:, c].astype(np.int64)] = out["start"][:, c]
        assert np.array_equal(by_op, ref)
        differs = differs or not np.array_equal(ref, ck.longest_path_starts(w, assign[:, c], order[:, c].astype(np.int64)))
    if config in (4, 5):
        assert differs                                            # the channels do bind on these workloads


def test_hand_worked_case_two_transfers_share_a_channel():
    """Ops 0 and 1 on machine 0 (durations 2, 1), ops 2 and 3 on machine 1 (durations 1, 1); edges 0 -> 2 and
    1 -> 3, transfer time 4.  pi = 0 1 2 3.  Op 0 ends at 2, op 1 at 3.  Transfer of 0 -> 2 runs 2..6, so op 2
    runs 6..7.  The channel is busy until 6, so the transfer of 1 -> 3 runs 6..10 (as a pure delay it would
    run 3..7) and op 3 runs 10..11 (7..8 as a pure delay, right after op 2)."""
    w = ck.problem(4, [(0, 2), (1, 3)], [2, 1, 1, 1], 2, comm=4)
    assign, order = ck.columns([[0, 0, 1, 1]], [[0, 1, 2, 3]], 4)
    excl = orc.evaluate(w, assign, order, flags=orc.COMM_EXCLUSIVE)
    delay = orc.evaluate(w, assign, order)
    assert excl["start"][:, 0].tolist() == [0, 2, 6, 10] and excl["finish"][:, 0].tolist() == [2, 3, 7, 11]
    assert delay["start"][:, 0].tolist() == [0, 2, 6, 7]
    # opposite directions are different channels: nothing to share
    w2 = ck.problem(4, [(0, 2), (3, 1)], [2, 1, 1, 1], 2, comm=4)
    a2, o2 = ck.columns([[0, 0, 1, 1]], [[0, 3, 2, 1]], 4)
    assert np.array_equal(orc.evaluate(w2, a2, o2, flags=orc.COMM_EXCLUSIVE)["start"], orc.evaluate(w2, a2, o2)["start"])


def test_one_machine_and_missing_channels_move_nothing():
    w = wl.make_config(1)
    K = 8
    assign, order = wl.make_candidates(w, K=K)
    one = np.zeros_like(assign)
    assert np.array_equal(orc.evaluate(w, one, order, flags=orc.COMM_EXCLUSIVE)["finish"], orc.evaluate(w, one, order)["finish"])
    w.link_class = np.full((w.num_devices, w.num_devices), 0xFF, np.uint8)
    a = orc.evaluate(w, assign, order, flags=orc.COMM_EXCLUSIVE); b = orc.evaluate(w, assign, order)
    assert np.array_equal(a["finish"], b["finish"]) and (a["status"] & orc.STATUS_NO_CHANNEL).any()


def test_golden_worked_example_exclusive_channels_and_decoding():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "worked_example_exclusive_channels_and_decoding.txt")
    edges, comm = [(0, 2), (1, 2), (0, 3), (2, 4), (3, 4)], [[2], [1], [5], [3], [1]]
    w = ck.problem(5, edges, [3, 2, 4, 1, 2], 2, comm=comm)
    ints = lambda s: [int(t) for t in s.split()]
    rows = [l for l in open(path) if l.strip() and l[0] != "#"]
    assert [r[0] for r in rows] == ["E", "E", "P", "P", "P"]
    for line in rows:
        f = [x.strip() for x in line.split("|")]
        if f[0] == "E":
            x, pi, s, e, z = [ints(t) for t in f[1:]]
            assign, order = ck.columns([x], [pi], 5)
            out = orc.evaluate(w, assign, order, flags=orc.COMM_EXCLUSIVE | orc.TIMES_BY_OP)
            assert out["start"][:, 0].tolist() == s and out["finish"][:, 0].tolist() == e and int(out["makespan"][0]) == z[0]
        else:
            lst, expect = ints(f[1]), ints(f[2])
            dec, status = orc.decode(w, np.array(lst, np.uint16)[:, None])
            assert status[0] == 0 and dec[:, 0].tolist() == expect
