"""Pins for the oracle's offline part (Eq. 26-30): estimate, order, LPT, local search.

Nothing here compares the oracle with itself: the checks are hand-worked
fixtures, closed forms, classical bounds, brute-force optima and library sorts.
"""
import heapq
import itertools
import json
import os

import numpy as np
import pytest

from oracle import hos_oracle as ora

GOLD = os.path.join(os.path.dirname(__file__), "golden")
CM = (20000, 40, 15000, 300, 16, 40, 350)


def brute_opt(T, M):
    best = None
    for a in itertools.product(range(M), repeat=len(T)):
        loads = [0] * M
        for t, j in zip(T, a):
            loads[j] += t
        m = max(loads)
        best = m if best is None or m < best else best
    return best


def test_estimate_is_the_linear_form():
    p = np.array([1, 16, 512, 4096], dtype=np.uint32)
    o = np.array([1, 8, 512, 2048], dtype=np.uint32)
    assert ora.estimate(p, o, CM).tolist() == [390, 3440, 199680, 880640]
    # coefficients are taken from the cost model, not fixed
    assert ora.estimate(p, o, (0, 0, 1, 0, 1, 3, 5)).tolist() == [8, 88, 4096, 22528]


def test_order_matches_library_sort():
    rng = np.random.default_rng(0)
    for n in (0, 1, 2, 17, 1000):
        T = rng.integers(1, 20, size=n).astype(np.int64)      # many ties
        od = ora.order(T)
        ref = np.lexsort((np.arange(n), -T))                 # T descending, index ascending
        assert od.tolist() == ref.tolist()


def test_worked_two_client_example():
    g = json.load(open(os.path.join(GOLD, "worked_pack.json")))["two_clients"]
    T = np.array(g["T"], dtype=np.int64)
    assign, load = ora.lpt(T, ora.order(T), g["M"])
    assert assign.tolist() == g["lpt_assign"] and load.tolist() == g["lpt_load"]
    assert brute_opt(g["T"], g["M"]) == g["optimum"]
    a2, l2, applied, log = ora.local_search(T, assign, load, 2)
    assert applied == g["rounds_applied"]
    assert a2.tolist() == g["ls_assign"] and l2.tolist() == g["ls_load"]
    assert [[int(m["i"]), int(m["u"]), int(m["k"]), int(m["v"])] for m in log] == g["ls_log"]


def test_worked_move_example():
    g = json.load(open(os.path.join(GOLD, "worked_pack.json")))["move_case"]
    T = np.array(g["T"], dtype=np.int64)
    a2, l2, applied, log = ora.local_search(T, g["assign"], g["load"], 2)
    assert applied == g["rounds_applied"]
    assert a2.tolist() == g["ls_assign"] and l2.tolist() == g["ls_load"]
    assert [[int(m["i"]), int(m["u"]), int(m["k"]), int(m["v"])] for m in log] == g["ls_log"]


def test_lpt_closed_forms():
    # N <= M: every request alone, makespan = T_max, request of rank r on client r
    T = np.array([5, 9, 7], dtype=np.int64)
    assign, load = ora.lpt(T, ora.order(T), 4)
    assert assign.tolist() == [2, 0, 1] and load.tolist() == [9, 7, 5, 0]
    # all equal: round robin, makespan ceil(N/M) * T
    T = np.full(11, 6, dtype=np.int64)
    assign, load = ora.lpt(T, ora.order(T), 4)
    assert assign.tolist() == [i % 4 for i in range(11)] and load.max() == 3 * 6
    # one client
    T = np.array([3, 1, 2], dtype=np.int64)
    assign, load = ora.lpt(T, ora.order(T), 1)
    assert assign.tolist() == [0, 0, 0] and load.tolist() == [6]


def test_lpt_equals_textbook_heap_list_scheduling():
    rng = np.random.default_rng(1)
    for _ in range(30):
        n, M = int(rng.integers(1, 200)), int(rng.integers(1, 12))
        T = rng.integers(1, 50, size=n).astype(np.int64)
        assign, load = ora.lpt(T, ora.order(T), M)
        heap = [(0, j) for j in range(M)]                     # (load, client): ties -> lowest client
        ref = np.empty(n, dtype=np.int64)
        for i in sorted(range(n), key=lambda i: (-T[i], i)):
            l, j = heapq.heappop(heap)
            ref[i] = j
            heapq.heappush(heap, (l + int(T[i]), j))
        assert assign.tolist() == ref.tolist()
        assert load.tolist() == [int(T[ref == j].sum()) for j in range(M)]


@pytest.mark.parametrize("seed", range(40))
def test_tiny_instances_against_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n, M = int(rng.integers(1, 10)), int(rng.integers(1, 4))
    hi = int(rng.choice([3, 10, 1000]))
    T = rng.integers(1, hi + 1, size=n).astype(np.int64)
    opt = brute_opt(T.tolist(), M)
    assign, load = ora.lpt(T, ora.order(T), M)
    # feasibility (Eq. 27-28)
    assert ((assign >= 0) & (assign < M)).all()
    assert load.tolist() == [int(T[assign == j].sum()) for j in range(M)]
    lpt = int(load.max())
    assert opt <= lpt
    assert 3 * M * lpt <= (4 * M - 1) * opt                  # Graham's LPT bound 4/3 - 1/(3M)
    assert M * lpt <= int(T.sum()) + (M - 1) * int(T.max())  # list-scheduling bound
    # local search never leaves the feasible set, never gets worse, never beats the optimum
    a2, l2, applied, log = ora.local_search(T, assign, load, 8)
    assert l2.tolist() == [int(T[a2 == j].sum()) for j in range(M)]
    assert opt <= int(l2.max()) <= lpt
    assert applied == sum(1 for m in log if m["i"] >= 0)


def _all_steps(T, assign, load):
    """Every (v, i, k, u) single step off the critical client, by plain enumeration."""
    M = len(load)
    jmax = int(np.argmax(load))                               # first maximum
    out = []
    for i in np.nonzero(assign == jmax)[0]:
        for k in range(M):
            if k == jmax:
                continue
            out.append((max(load[jmax] - T[i], load[k] + T[i]), int(i), k, -1))
            for u in np.nonzero(assign == k)[0]:
                d = T[i] - T[u]
                if d > 0:
                    out.append((max(load[jmax] - d, load[k] + d), int(i), k, int(u)))
    return jmax, out


@pytest.mark.parametrize("seed", range(25))
def test_local_search_round_by_round(seed):
    rng = np.random.default_rng(500 + seed)
    n, M = int(rng.integers(2, 60)), int(rng.integers(2, 7))
    T = rng.integers(1, int(rng.choice([4, 30, 5000])) + 1, size=n).astype(np.int64)
    assign = rng.integers(0, M, size=n).astype(np.int32)      # arbitrary (bad) start
    load = np.array([int(T[assign == j].sum()) for j in range(M)], dtype=np.int64)
    rounds = 12
    a_end, l_end, applied, log = ora.local_search(T, assign, load, rounds)
    a, l = assign.copy(), load.copy()
    done = False
    for r in range(rounds):
        jmax, steps = _all_steps(T, a, l)
        best = min(steps) if steps else None
        m = log[r]
        if done or best is None or best[0] >= l[jmax]:
            done = True
            assert (int(m["i"]), int(m["u"]), int(m["k"]), int(m["v"])) == (-1, -1, -1, int(l.max()))
            continue
        assert (int(m["v"]), int(m["i"]), int(m["k"]), int(m["u"])) == tuple(int(x) for x in best)
        before = sorted(l.tolist(), reverse=True)
        d = T[best[1]] - (T[best[3]] if best[3] >= 0 else 0)
        a[best[1]] = best[2]
        if best[3] >= 0:
            a[best[3]] = jmax
        l[jmax] -= d
        l[best[2]] += d
        assert sorted(l.tolist(), reverse=True) < before       # strict lexicographic descent
    assert a.tolist() == a_end.tolist() and l.tolist() == l_end.tolist()
    assert applied == sum(1 for m in log if m["i"] >= 0)


def test_local_search_is_a_noop_when_nothing_can_move():
    T = np.array([4, 4, 4], dtype=np.int64)
    a, l, applied, log = ora.local_search(T, [0, 1, 2], [4, 4, 4], 3)
    assert applied == 0 and a.tolist() == [0, 1, 2] and all(m["i"] == -1 for m in log)
    a, l, applied, log = ora.local_search(T, [0, 0, 0], [12], 3)          # single client
    assert applied == 0 and l.tolist() == [12]
