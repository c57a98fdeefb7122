"""Trace export: one event per operator, on its machine's row, never overlapping on a row."""
import json

import numpy as np

from oracle import pe_oracle as orc
from paper_2503_09357_b200 import workloads as wl
from paper_2503_09357_b200.trace import candidate_trace, write_candidate_trace


def test_trace_of_an_evaluated_candidate(tmp_path):
    w = wl.make_config(1)
    assign, order = wl.make_candidates(w, K=4)
    out = orc.evaluate(w, assign, order, flags=orc.TIMES_BY_OP)
    c = 2
    path = tmp_path / "cand.json"
    write_candidate_trace(path, assign[:, c], out["start"][:, c], out["finish"][:, c])
    tr = json.load(open(path))
    ev = [e for e in tr["traceEvents"] if e["ph"] == "X"]
    assert len(ev) == w.num_ops
    assert max(e["ts"] + e["dur"] for e in ev) == out["makespan"][c]
    for j in range(w.num_devices):
        rows = sorted((e["ts"], e["ts"] + e["dur"]) for e in ev if e["tid"] == j)
        assert all(a[1] <= b[0] for a, b in zip(rows[:-1], rows[1:]))          # one operator at a time (Eq. 7)
        assert sum(b - a for a, b in rows) == out["busy"][j, c]
    assert candidate_trace([0], [0], [3], names=["F0"])["traceEvents"][1]["name"] == "F0"
