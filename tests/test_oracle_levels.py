"""Pins for the stepped prefill cost (Eq. 5-7) and the printed form of Eq. 31."""
import json
import os

import numpy as np
import pytest

from oracle import hos_oracle as ora
from tests.trace_check import replay

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rows(trace):
    return [[int(r["dur_us"]), int(r["kind_n"]), int(r["tokens"]), int(r["aux"])] for r in trace]


def test_hand_worked_levels():
    g = json.load(open(os.path.join(GOLD, "worked_levels.json")))
    p, o = np.array(g["p"], dtype=np.uint32), np.array(g["o"], dtype=np.uint32)
    r = ora.simulate_client(np.arange(4), p, o, g["cost_model"], g["cap"], g["kv_budget"], g["lambda_q16"],
                            want_trace=True)
    assert rows(r.trace) == g["trace"] and r.makespan_us == g["makespan_us"]
    lb = ora.lower_bound(p, o, 1, g["cap"], g["cost_model"])
    assert lb["tp_paper_us"] == g["tp_paper_us"] and lb["tp_star_us"] == g["tp_star_us"]
    assert lb["lb_sim_us"] <= r.makespan_us


def test_paper_prefill_example_as_a_level():
    # the paper's printed example: a stage of 5,000 tokens takes 675 ms
    g = json.load(open(os.path.join(GOLD, "paper_cost_examples.json")))
    cm = (0, 0, 29000, 210, 0x7FFFFFFF, 1, 1, [(1000, 155000), (5000, g["prefill_stage"]["expected_us"])])
    p = np.full(200, 25, dtype=np.uint32)
    o = np.ones(200, dtype=np.uint32)
    r = ora.simulate_client(np.arange(200), p, o, cm, 200, 10 ** 9, 65536, want_trace=True)
    assert rows(r.trace)[0][:3] == [675000, (1 << 31) | 200, 5000]
    assert rows(r.trace)[1][0] == g["decode_round"]["expected_us"]
    # one token more would not fit the largest level: the stage stops at 5,000 tokens
    p2 = np.append(p, 1).astype(np.uint32)
    o2 = np.ones(201, dtype=np.uint32)
    r2 = ora.simulate_client(np.arange(201), p2, o2, cm, 250, 10 ** 9, 65536, want_trace=True)
    assert rows(r2.trace)[0][:3] == [675000, (1 << 31) | 200, 5000]


@pytest.mark.parametrize("seed", range(20))
def test_level_traces_obey_the_rules_and_bounds(seed):
    rng = np.random.default_rng(7000 + seed)
    n, M = int(rng.integers(1, 100)), int(rng.integers(1, 4))
    cap = int(rng.choice([1, 2, 8, 32]))
    p = rng.integers(1, 200, size=n).astype(np.uint32)
    o = rng.integers(1, 30, size=n).astype(np.uint32)
    levels = [(200, 9000), (500, 15000), (1500, 30000)][: int(rng.integers(1, 4))]
    cm = (123, 7, 15000, 300, 16, 40, 350, levels)          # a_p, b_p must be ignored
    lam = int(rng.choice([0, 65536, 0xFFFFFFFF]))
    assign = rng.integers(0, M, size=n).astype(np.int32)
    for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
        q_off, q_req = ora.queue_build(assign, p, o, M, mode)
        sim = ora.simulate(assign, p, o, M, cm, cap, 10 ** 6, lam, mode, want_trace=True)
        for j in range(M):
            chk = replay(q_req[q_off[j]:q_off[j + 1]], p, o, cm, cap, 10 ** 6, lam, rows(sim.clients[j].trace))
            assert chk["makespan_us"] == sim.clients[j].makespan_us
        lb = ora.lower_bound(p, o, M, cap, cm)
        assert lb["lb_sim_us"] <= sim.makespan_us
        steal, _ = ora.simulate_steal(assign, p, o, M, cm, cap, 10 ** 6, lam, mode)
        assert lb["lb_sim_us"] <= steal.makespan_us
