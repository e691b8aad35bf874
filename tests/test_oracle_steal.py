"""Pins for the oracle's request stealing (Algorithm 1, second part)."""
import json
import os

import numpy as np
import pytest

from oracle import hos_oracle as ora

GOLD = os.path.join(os.path.dirname(__file__), "golden")
CM = (20000, 40, 15000, 300, 16, 40, 350)
LAMBDAS = (0, 1000, 65536, 1 << 20, 0xFFFFFFFF)


def rows(trace):
    return [[int(r["dur_us"]), int(r["kind_n"]), int(r["tokens"]), int(r["aux"])] for r in trace]


def python_steal_sim(queues, p, o, cm, cap, kv, lam, max_iters=10 ** 9, o_key=None, kv_reserve=0):
    """Independent plain-Python statement of the same rules (lists and dicts, no shared code).

    With a level table in cm[7] (Eq. 5-7) a prefill stage lasts the time of the smallest level that
    holds its prompt tokens, and no stage -- own requests or taken ones -- grows past the largest level."""
    ap, bp, ad, bd, q = cm[:5]
    levels = sorted(cm[7]) if len(cm) > 7 else []
    stage_room = levels[-1][0] if levels else float("inf")

    def stage_time(tokens):
        if not levels:
            return ap + bp * tokens
        return next(t for c, t in levels if tokens <= c)
    M = len(queues)
    o_key = o if o_key is None else o_key                   # what the scheduler believes
    holds = (lambda i: kv_reserve) if kv_reserve else (lambda i: int(p[i]) + int(o[i]))
    waiting = [list(qj) for qj in queues]                  # unclaimed requests per client, in order
    st = [dict(run={}, cand=[], clock=0, waited=0, busy=0, admitted=0, trace=[], done=False) for _ in range(M)]
    served = {}
    while True:
        live = [j for j in range(M) if not st[j]["done"]]
        if not live:
            break
        j = min(live, key=lambda x: (st[x]["clock"], x))
        s = st[j]
        used = lambda: sum(holds(i) for i in list(s["run"]) + s["cand"])
        while waiting[j] and len(s["run"]) + len(s["cand"]) < cap:
            i = waiting[j][0]
            if used() + holds(i) > kv:
                break
            if sum(int(p[x]) for x in s["cand"]) + int(p[i]) > stage_room:
                break
            s["cand"].append(waiting[j].pop(0)); served[i] = j
        if not waiting[j]:
            while len(s["run"]) + len(s["cand"]) < cap:
                left = [sum(int(p[i]) + int(o_key[i]) for i in w) for w in waiting]
                if max(left) <= 0:
                    break
                d = left.index(max(left))                   # first maximum: lowest client on ties
                i = waiting[d][0]
                if used() + holds(i) > kv:
                    break
                if sum(int(p[x]) for x in s["cand"]) + int(p[i]) > stage_room:
                    break
                s["cand"].append(waiting[d].pop(0)); served[i] = j
        if not s["run"] and not s["cand"]:
            s["done"] = True
            continue
        if len(s["trace"]) == max_iters:
            s["done"] = True
            continue
        cp = stage_time(sum(int(p[i]) for i in s["cand"]))
        if s["cand"] and (not s["run"] or lam * s["waited"] > (cp << 16)):
            rec = [cp, (1 << 31) | len(s["cand"]), sum(int(p[i]) for i in s["cand"]), s["admitted"]]
            s["busy"] += cp * len(s["cand"])
            for i in s["cand"]:
                s["run"][i] = [int(p[i]), int(o[i])]
            s["admitted"] += len(s["cand"]); s["cand"] = []; s["waited"] = 0
        else:
            B, S = len(s["run"]), sum(v[0] for v in s["run"].values())
            dur = ad + bd * B + S // q
            gone = []
            for i, v in s["run"].items():
                v[0] += 1; v[1] -= 1
                if v[1] == 0:
                    gone.append(i)
            for i in gone:
                del s["run"][i]
            rec = [dur, B, S, len(gone)]
            s["busy"] += dur * B
            s["waited"] = min(s["waited"] + dur, 2 ** 31 - 1)
        s["clock"] += rec[0]
        s["trace"].append(rec)
    return st, served


def test_hand_worked_steal():
    g = json.load(open(os.path.join(GOLD, "worked_steal.json")))
    p, o = np.array(g["p"], dtype=np.uint32), np.array(g["o"], dtype=np.uint32)
    sim, served = ora.simulate_steal(g["assign"], p, o, g["n_clients"], g["cost_model"], g["cap"],
                                     g["kv_budget"], g["lambda_q16"], ora.QUEUE_SORTED, want_trace=True)
    assert [rows(c.trace) for c in sim.clients] == g["traces"]
    assert served.tolist() == g["served_by"]
    assert [c.makespan_us for c in sim.clients] == g["client_makespan_us"] and sim.makespan_us == g["makespan_us"]
    plain = ora.simulate(g["assign"], p, o, g["n_clients"], g["cost_model"], g["cap"], g["kv_budget"],
                         g["lambda_q16"], ora.QUEUE_SORTED)
    assert plain.makespan_us == g["makespan_without_steal_us"]


def test_single_client_has_nobody_to_steal_from():
    rng = np.random.default_rng(2)
    p = rng.integers(1, 200, size=80).astype(np.uint32)
    o = rng.integers(1, 40, size=80).astype(np.uint32)
    for lam in LAMBDAS:
        a = ora.simulate(np.zeros(80, np.int32), p, o, 1, CM, 8, 10 ** 6, lam, ora.QUEUE_SORTED, want_trace=True)
        b, served = ora.simulate_steal(np.zeros(80, np.int32), p, o, 1, CM, 8, 10 ** 6, lam, ora.QUEUE_SORTED,
                                       want_trace=True)
        assert rows(a.clients[0].trace) == rows(b.clients[0].trace)
        assert a.clients[0].trace_hash == b.clients[0].trace_hash and (served == 0).all()
        assert (a.makespan_us, a.busy_slot_us, a.utilisation) == (b.makespan_us, b.busy_slot_us, b.utilisation)


@pytest.mark.parametrize("seed", range(40))
def test_against_independent_python_statement(seed):
    rng = np.random.default_rng(4000 + seed)
    n, M = int(rng.integers(1, 90)), int(rng.integers(1, 7))
    cap = int(rng.choice([1, 2, 3, 8, 30]))
    p = rng.integers(1, 200, size=n).astype(np.uint32)
    o = rng.integers(1, 30, size=n).astype(np.uint32)
    kv = int(rng.choice([int((p + o).max()), 2 * int((p + o).max()), 10 ** 6]))
    lam = int(rng.choice(LAMBDAS))
    mode = int(rng.integers(0, 2))
    assign = (rng.integers(0, M, size=n) if seed % 3 else np.sort(rng.integers(0, M, size=n))).astype(np.int32)
    if seed % 5 == 0:
        assign[:] = 0                                           # everything queued on one client
    sim, served = ora.simulate_steal(assign, p, o, M, CM, cap, kv, lam, mode, want_trace=True)
    q_off, q_req = ora.queue_build(assign, p, o, M, mode)
    st, served_py = python_steal_sim([q_req[q_off[j]:q_off[j + 1]].tolist() for j in range(M)], p, o, CM, cap, kv, lam)
    for j in range(M):
        assert rows(sim.clients[j].trace) == st[j]["trace"], f"client {j}"
        assert sim.clients[j].makespan_us == st[j]["clock"] and sim.clients[j].busy_slot_us == st[j]["busy"]
        assert sim.clients[j].status == 0
    assert served.tolist() == [served_py[i] for i in range(n)]
    # what the rules fix whatever the schedule: everybody served once, token conservation, lower bound
    assert sorted(served_py) == list(range(n))
    alltr = [r for j in range(M) for r in st[j]["trace"]]
    assert sum(r[2] for r in alltr if r[1] >> 31) == int(p.sum())
    assert sum(r[1] for r in alltr if not r[1] >> 31) == int(o.sum())
    assert sum((r[1] & 0x7FFFFFFF) for r in alltr if r[1] >> 31) == n
    assert ora.lower_bound(p, o, M, cap, CM)["lb_sim_us"] <= sim.makespan_us


def test_stealing_helps_a_lopsided_assignment():
    rng = np.random.default_rng(9)
    n, M, cap = 400, 4, 8
    p = rng.integers(16, 300, size=n).astype(np.uint32)
    o = rng.integers(8, 200, size=n).astype(np.uint32)
    assign = np.zeros(n, dtype=np.int32)                        # all requests queued on client 0
    plain = ora.simulate(assign, p, o, M, CM, cap, 10 ** 6, 65536, ora.QUEUE_SORTED)
    steal, served = ora.simulate_steal(assign, p, o, M, CM, cap, 10 ** 6, 65536, ora.QUEUE_SORTED)
    assert steal.makespan_us < plain.makespan_us / 2
    assert len(set(served.tolist())) == M


def test_iteration_limit_with_stealing():
    p, o = np.full(6, 10, dtype=np.uint32), np.full(6, 5, dtype=np.uint32)
    sim, _ = ora.simulate_steal([0, 0, 0, 1, 1, 1], p, o, 2, CM, 2, 10 ** 6, 65536, ora.QUEUE_SORTED,
                                max_iters=3, want_trace=True)
    assert all(c.status == 1 and len(c.trace) == 3 for c in sim.clients)


def test_hand_worked_steal_refused_by_a_full_stage():
    """Stealing with prefill levels (Algorithm 1 with Eq. 5-7): client 1, with a free slot and its own
    queue used up, may not take client 0's waiting request because its stage of 150 tokens plus the
    70 of that request would pass the largest level (200 tokens)."""
    g = json.load(open(os.path.join(GOLD, "worked_steal_levels.json")))
    p, o = np.array(g["p"], dtype=np.uint32), np.array(g["o"], dtype=np.uint32)
    cm = tuple(g["cost_model"][:7]) + ([tuple(l) for l in g["levels"]],)
    sim, served = ora.simulate_steal(g["assign"], p, o, g["n_clients"], cm, g["cap"], g["kv_budget"],
                                     g["lambda_q16"], ora.QUEUE_SORTED, want_trace=True)
    assert [rows(c.trace) for c in sim.clients] == g["traces"]
    assert served.tolist() == g["served_by"]
    assert [c.makespan_us for c in sim.clients] == g["client_makespan_us"]
    # with a larger top level the same request IS taken (and priced at that level)
    cm2 = tuple(g["cost_model"][:7]) + ([tuple(l) for l in g["levels"]] + [(220, 30000)],)
    sim2, served2 = ora.simulate_steal(g["assign"], p, o, g["n_clients"], cm2, g["cap"], g["kv_budget"],
                                       g["lambda_q16"], ora.QUEUE_SORTED, want_trace=True)
    assert served2.tolist() == g["served_by_with_a_larger_level"]
    assert rows(sim2.clients[1].trace)[0] == [30000, (1 << 31) | 2, 220, 0]


@pytest.mark.parametrize("seed", range(24))
def test_levels_against_independent_python_statement(seed):
    """Stealing combined with the stepped prefill cost: every record, clock and owner against the
    plain-Python model with the level table and the stage capacity."""
    rng = np.random.default_rng(9100 + seed)
    n, M = int(rng.integers(2, 90)), int(rng.integers(2, 7))
    cap = int(rng.choice([2, 3, 8, 30]))
    p = rng.integers(1, 200, size=n).astype(np.uint32)
    o = rng.integers(1, 30, size=n).astype(np.uint32)
    # top levels small enough that stages often stop at the capacity, with free slots left
    levels = [(200, 9000), (320, 15000), (700, 30000)][: int(rng.integers(1, 4))]
    cm = (123, 7, 15000, 300, 16, 40, 350, levels)
    kv = int(rng.choice([2 * int((p + o).max()), 10 ** 6]))
    lam = int(rng.choice(LAMBDAS))
    mode = int(rng.integers(0, 2))
    assign = rng.integers(0, M, size=n).astype(np.int32)
    if seed % 3 == 0:
        assign[:] = rng.integers(0, max(1, M // 2), size=n)     # idle clients: stealing from the start
    sim, served = ora.simulate_steal(assign, p, o, M, cm, cap, kv, lam, mode, want_trace=True)
    q_off, q_req = ora.queue_build(assign, p, o, M, mode)
    st, served_py = python_steal_sim([q_req[q_off[j]:q_off[j + 1]].tolist() for j in range(M)], p, o, cm, cap, kv, lam)
    refused = 0
    for j in range(M):
        assert rows(sim.clients[j].trace) == st[j]["trace"], f"client {j}"
        assert sim.clients[j].makespan_us == st[j]["clock"] and sim.clients[j].busy_slot_us == st[j]["busy"]
        refused += sum(1 for r in st[j]["trace"] if r[1] >> 31 and (r[1] & 0x7FFFFFFF) < cap)
    assert served.tolist() == [served_py[i] for i in range(n)]
    assert all(r[2] <= levels[-1][0] for j in range(M) for r in st[j]["trace"] if r[1] >> 31)
