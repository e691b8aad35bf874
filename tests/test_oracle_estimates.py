"""Pins for scheduling on estimated output lengths with a fixed KV reservation per request."""
import json
import os

import numpy as np
import pytest

from oracle import hos_oracle as ora
from tests import trace_check
from tests.test_oracle_steal import python_steal_sim, rows
from workload import workload
from workload.gen import estimated_outputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")
CM = (20000, 40, 15000, 300, 16, 40, 350)
LAMBDAS = (0, 1000, 65536, 1 << 20, 0xFFFFFFFF)


def random_case(rng, n, M):
    p = rng.integers(1, 300, n).astype(np.uint32)
    o = rng.integers(1, 60, n).astype(np.uint32)
    est = np.clip(np.rint(o * np.exp(0.5 * rng.standard_normal(n))), 1, 100).astype(np.uint32)
    assign = rng.integers(0, M, n).astype(np.int32)
    return p, o, est, assign


def test_hand_worked_estimates():
    g = json.load(open(os.path.join(GOLD, "worked_estimates.json")))
    p, o, est = (np.array(g[k], dtype=np.uint32) for k in ("p", "o", "o_est"))
    q_off, q_req = ora.queue_build(np.zeros(3, np.int32), p, est, 1, ora.QUEUE_SORTED)
    assert list(q_req) == g["queue"]
    r = ora.simulate_client(q_req, p, o, g["cm"], g["cap"], g["kv_budget"], g["lambda_q16"], want_trace=True,
                            kv_reserve=g["kv_reserve"])
    assert rows(r.trace) == g["trace"]
    for f in ("makespan_us", "busy_slot_us", "n_prefill_iters", "n_decode_iters"):
        assert getattr(r, f) == g[f]
    assert r.trace_hash == trace_check.trace_hash(g["trace"])


def test_queue_order_uses_the_estimates():
    rng = np.random.default_rng(5)
    for _ in range(20):
        p, o, est, assign = random_case(rng, 60, 3)
        q_off, q_req = ora.queue_build(assign, p, est, 3, ora.QUEUE_SORTED)
        for j in range(3):
            mem = [i for i in range(60) if assign[i] == j]
            want = sorted(mem, key=lambda i: (-(int(p[i]) + int(est[i])), i))
            assert list(q_req[q_off[j]:q_off[j + 1]]) == want


@pytest.mark.parametrize("lam", LAMBDAS)
def test_fixed_reservation_is_a_smaller_batch_cap(lam):
    """Reserving R tokens per request admits floor(kv / R) requests at most and nothing else:
    the same trace as the plain simulator with that batch cap and no KV limit."""
    rng = np.random.default_rng(lam % 1000 + 7)
    for _ in range(12):
        p, o, est, assign = random_case(rng, 50, 1)
        q_off, q_req = ora.queue_build(assign * 0, p, est, 1, ora.QUEUE_SORTED)
        cap = int(rng.integers(1, 12))
        R = int((p.astype(np.int64) + o).max()) + int(rng.integers(0, 50))
        kv = R * int(rng.integers(1, 12)) + int(rng.integers(0, R))
        a = ora.simulate_client(q_req, p, o, CM, cap, kv, lam, want_trace=True, kv_reserve=R)
        b = ora.simulate_client(q_req, p, o, CM, min(cap, kv // R), 10 ** 12, lam, want_trace=True)
        assert rows(a.trace) == rows(b.trace) and a.makespan_us == b.makespan_us
        assert a.busy_slot_us == b.busy_slot_us and a.trace_hash == b.trace_hash


@pytest.mark.parametrize("mode", [ora.QUEUE_SORTED, ora.QUEUE_FCFS])
def test_replay_checker_with_estimates(mode):
    rng = np.random.default_rng(11 + mode)
    for _ in range(15):
        p, o, est, assign = random_case(rng, 70, 2)
        cap, R = int(rng.integers(1, 9)), 400
        kv = int(rng.integers(R, 6 * R))
        lam = int(rng.choice(LAMBDAS))
        s = ora.simulate(assign, p, o, 2, CM, cap, kv, lam, mode, want_trace=True, o_est=est, kv_reserve=R)
        for j, c in enumerate(s.clients):
            mem = [i for i in range(70) if assign[i] == j]
            queue = sorted(mem, key=lambda i: (-(int(p[i]) + int(est[i])), i)) if mode == ora.QUEUE_SORTED else mem
            rep = trace_check.replay(queue, p, o, CM, cap, kv, lam, rows(c.trace), kv_reserve=R)
            for f, v in rep.items():
                assert getattr(c, f) == v
            assert c.trace_hash == trace_check.trace_hash(rows(c.trace))


def test_exact_estimates_change_nothing():
    w = workload("c0")
    p, o = w.lengths()
    pk = ora.offline_pack(p[0], o[0], w.n_clients, w.cost_model, 5)
    a = ora.simulate(pk["assign"], p[0], o[0], w.n_clients, w.cost_model, w.batch_cap, w.kv_budget, 65536,
                     ora.QUEUE_SORTED)
    b = ora.simulate(pk["assign"], p[0], o[0], w.n_clients, w.cost_model, w.batch_cap, w.kv_budget, 65536,
                     ora.QUEUE_SORTED, o_est=o[0], kv_reserve=0)
    assert [c.trace_hash for c in a.clients] == [c.trace_hash for c in b.clients]
    assert a.makespan_us == b.makespan_us


def test_lower_bound_holds_under_estimates():
    w = workload("c1e").subset(0, 1)
    p, o = w.lengths()
    est = w.estimates()
    lb = ora.lower_bound(p[0], o[0], w.n_clients, w.batch_cap, w.cost_model)
    pk = ora.offline_pack(p[0], est[0], w.n_clients, w.cost_model, 10)      # packed on the estimates
    for lam in LAMBDAS:
        for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
            s = ora.simulate(pk["assign"], p[0], o[0], w.n_clients, w.cost_model, w.batch_cap, w.kv_budget, lam,
                             mode, o_est=est[0], kv_reserve=w.kv_reserve)
            assert lb["lb_sim_us"] <= s.makespan_us
            assert sum(c.n_decode_iters for c in s.clients) >= int(o[0].max())


@pytest.mark.parametrize("seed", range(12))
def test_stealing_under_estimates_against_plain_python(seed):
    rng = np.random.default_rng(100 + seed)
    M = int(rng.integers(2, 5))
    p, o, est, assign = random_case(rng, 40, M)
    cap, R = int(rng.integers(1, 6)), 400
    kv = int(rng.integers(R, 5 * R))
    lam = int(rng.choice(LAMBDAS))
    s, served = ora.simulate_steal(assign, p, o, M, CM, cap, kv, lam, ora.QUEUE_SORTED, want_trace=True,
                                   o_est=est, kv_reserve=R)
    q_off, q_req = ora.queue_build(assign, p, est, M, ora.QUEUE_SORTED)
    st, served_py = python_steal_sim([list(q_req[q_off[j]:q_off[j + 1]]) for j in range(M)], p, o, CM, cap, kv,
                                     lam, o_key=est, kv_reserve=R)
    for j in range(M):
        assert rows(s.clients[j].trace) == st[j]["trace"]
        assert s.clients[j].makespan_us == st[j]["clock"]
    assert {i: int(c) for i, c in enumerate(served)} == served_py


def test_estimate_generator():
    w = workload("c1e")
    _, o = w.lengths()
    est = w.estimates()
    assert est.shape == o.shape and est.dtype == np.uint32
    assert est.min() >= w.dist_o.lo and est.max() <= w.dist_o.hi
    assert np.array_equal(est, w.estimates())                           # seeded
    assert np.array_equal(estimated_outputs(1, o[0], 0.0, w.dist_o.lo, w.dist_o.hi), o[0])
    ratio = np.log(est[0].astype(np.float64) / o[0])
    inner = (est[0] > w.dist_o.lo) & (est[0] < w.dist_o.hi)
    assert abs(ratio[inner].std() - 0.3) < 0.03
    assert workload("c1").estimates() is None
