"""The CSV form of an iteration trace, on the hand-worked example of the simulator's pins."""
import io
import json
import os

import numpy as np

from oracle import hos_oracle as ora
from paper_2502_15763_b200.trace_csv import write_trace_csv

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_csv_rows_of_the_worked_trace():
    g = json.load(open(os.path.join(GOLD, "worked_sim.json")))
    case = g["lambda_1"]
    p = np.array(g["p"], dtype=np.uint32); o = np.array(g["o"], dtype=np.uint32)
    sim = ora.simulate(np.zeros(len(p), np.int32), p, o, 1, g["cost_model"], g["cap"], g["kv_budget"],
                       case.get("lambda_q16", 65536), ora.QUEUE_SORTED, want_trace=True)
    tr = sim.clients[0].trace
    fh = io.StringIO()
    n = write_trace_csv(fh, tr, np.array([0, len(tr)]), 1, 1)
    lines = fh.getvalue().strip().split("\n")
    assert n == len(tr) == len(lines) - 1
    first = lines[1].split(",")
    assert first[:5] == ["0", "0", "0", "0", "0"] and first[6] == "prefill"
    # start times are the running sum of the durations; the last row ends at the makespan
    last = lines[-1].split(",")
    assert int(last[4]) + int(last[5]) == sim.clients[0].makespan_us
    assert sum(int(l.split(",")[5]) for l in lines[1:]) == sim.clients[0].makespan_us


def test_csv_rows_match_the_printed_records():
    g = json.load(open(os.path.join(GOLD, "worked_sim.json")))
    want = g["lambda_1"]["trace"]
    rec = np.zeros(len(want), dtype=ora.REC_DTYPE)
    for i, (d, kn, tok, aux) in enumerate(want):
        rec[i] = (d, kn, tok, aux)
    fh = io.StringIO()
    write_trace_csv(fh, rec, np.array([0, len(rec)]), 1, 1)
    rows = [l.split(",") for l in fh.getvalue().strip().split("\n")[1:]]
    assert [r[6] for r in rows] == ["prefill", "decode", "decode", "prefill", "decode", "decode"]
    assert [int(r[4]) for r in rows] == [0, 23200, 38805, 54410, 75050, 90653]
    assert [[int(r[5]), int(r[7]), int(r[8]), int(r[9])] for r in rows] == \
        [[d, kn & 0x7FFFFFFF, tok, aux] for d, kn, tok, aux in want]
