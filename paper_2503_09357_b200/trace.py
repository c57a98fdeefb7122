"""Export one evaluated candidate as trace-event JSON (the format chrome://tracing and Perfetto read;
Section V of the paper shows its schedules that way).  Host-side convenience, not part of the hot path:
it only re-arranges outputs of pe_eval_batch."""
import json

import numpy as np


def candidate_trace(assign_col, start_by_op, finish_by_op, names=None, time_unit_us: float = 1.0):
    """Trace events of one candidate: one complete event ("ph": "X") per operator on the row of its
    machine.  `assign_col`, `start_by_op`, `finish_by_op` are length-V arrays indexed by operator."""
    assign_col = np.asarray(assign_col)
    start_by_op = np.asarray(start_by_op)
    finish_by_op = np.asarray(finish_by_op)
    events = []
    for j in sorted(set(int(x) for x in assign_col)):
        events.append({"name": "thread_name", "ph": "M", "pid": 0, "tid": j, "args": {"name": f"machine {j}"}})
    for i in range(len(assign_col)):
        events.append({"name": names[i] if names is not None else f"op {i}", "ph": "X", "pid": 0,
                       "tid": int(assign_col[i]), "ts": float(start_by_op[i]) * time_unit_us,
                       "dur": float(finish_by_op[i] - start_by_op[i]) * time_unit_us, "args": {"op": i}})
    return {"traceEvents": events, "displayTimeUnit": "ns"}


def write_candidate_trace(path, assign_col, start_by_op, finish_by_op, names=None, time_unit_us: float = 1.0):
    with open(path, "w") as f:
        json.dump(candidate_trace(assign_col, start_by_op, finish_by_op, names, time_unit_us), f)
