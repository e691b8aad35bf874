"""The iteration trace as text: one CSV row per iteration (the Gantt chart of one client).

    write_trace_csv(fh, records, offsets, n_lambda, n_clients)

`records` is the host copy of the trace buffer viewed with ITER_REC_DTYPE and `offsets` the host
copy of trace_off (see hos_online_simulate / hos_trace_fill).  Columns: instance, multiplier
index, client, iteration, start_us, duration_us, kind (prefill | decode), n (requests admitted, or
batch size), tokens (prompt tokens admitted, or sum of KV lengths before the step), aux (queue
position of the first admitted request, or requests retired by the step).  Pure host code.
"""
from __future__ import annotations

import numpy as np


def write_trace_csv(fh, records: np.ndarray, offsets: np.ndarray, n_lambda: int, n_clients: int,
                    units=None) -> int:
    """Writes the units in `units` (default: all) and returns the number of rows written."""
    fh.write("instance,multiplier,client,iteration,start_us,duration_us,kind,n,tokens,aux\n")
    n_units = len(offsets) - 1
    rows = 0
    for x in (range(n_units) if units is None else units):
        a, b = int(offsets[x]), int(offsets[x + 1])
        rec = records[a:b]
        dur = rec["dur_us"].astype(np.int64)
        start = np.concatenate([[0], np.cumsum(dur)[:-1]]) if len(rec) else np.zeros(0, np.int64)
        pre = (rec["kind_n"] >> 31) != 0
        n = rec["kind_n"] & 0x7FFFFFFF
        inst, rest = divmod(x, n_lambda * n_clients)
        lam, client = divmod(rest, n_clients)
        for it in range(len(rec)):
            fh.write(f"{inst},{lam},{client},{it},{int(start[it])},{int(dur[it])},"
                     f"{'prefill' if pre[it] else 'decode'},{int(n[it])},{int(rec['tokens'][it])},{int(rec['aux'][it])}\n")
        rows += len(rec)
    return rows
