"""Pins for the oracle's stronger packing (MULTIFIT) and its exhaustive optimum, Eq. 26-30.

Independent of the oracle: a hand-worked instance, a plain-Python restatement of the bisection and
of first-fit decreasing, brute force over all assignments, and the published worst-case ratio."""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import hos_oracle as ora

GOLD = os.path.join(os.path.dirname(__file__), "golden")
CM = (20000, 40, 15000, 300, 16, 40, 350)


def python_first_fit(T, order, M, C):
    load, assign = [0] * M, [None] * len(T)
    for i in order:
        fits = [j for j in range(M) if load[j] + T[i] <= C]
        if not fits:
            return None
        assign[i] = fits[0]
        load[fits[0]] += T[i]
    return assign, load


def python_multifit(T, M, max_steps=64):
    order = sorted(range(len(T)), key=lambda i: (-T[i], i))
    total, longest = sum(T), max(T)
    lo = max(-(-total // M), longest)
    hi = max(-(-2 * total // M), longest)
    probes = []
    while lo < hi and len(probes) < max_steps:
        C = (lo + hi) // 2
        ok = python_first_fit(T, order, M, C) is not None
        probes.append([C, ok])
        if ok:
            hi = C
        else:
            lo = C + 1
    return python_first_fit(T, order, M, hi), hi, probes


def brute_opt(T, M):
    best = None
    for a in itertools.product(range(M), repeat=len(T)):
        loads = [0] * M
        for t, j in zip(T, a):
            loads[j] += t
        best = max(loads) if best is None else min(best, max(loads))
    return best


def test_hand_worked_multifit():
    g = json.load(open(os.path.join(GOLD, "worked_multifit.json")))
    T = np.array(g["T"], dtype=np.int64)
    od = ora.order(T)
    _, lpt_load = ora.lpt(T, od, g["M"])
    assert lpt_load.tolist() == g["lpt_load"]
    assign, load, C = ora.multifit(T, od, g["M"])
    assert (assign.tolist(), load.tolist(), C) == (g["assign"], g["load"], g["capacity"])
    assert ora.optimal_makespan(T, g["M"]) == g["optimum"]
    a1, l1, C1 = ora.multifit(T, od, g["M"], max_steps=1)      # one probe: the packing at 13
    assert (a1.tolist(), l1.tolist(), C1) == (g["one_probe"]["assign"], g["one_probe"]["load"], g["one_probe"]["capacity"])
    # the hand-worked probe sequence is what the plain restatement takes too
    _, hi, probes = python_multifit(g["T"], g["M"])
    assert probes == g["probes"] and hi == g["capacity"]


@pytest.mark.parametrize("seed", range(60))
def test_against_plain_python_restatement(seed):
    rng = np.random.default_rng(12000 + seed)
    n, M = int(rng.integers(1, 300)), int(rng.integers(1, 20))
    T = rng.integers(1, int(rng.choice([4, 50, 10 ** 6])), size=n).astype(np.int64)
    steps = int(rng.choice([1, 3, 64]))
    got = ora.multifit(T, ora.order(T), M, steps)
    (assign, load), C, _ = python_multifit(T.tolist(), M, steps)
    assert got is not None and got[2] == C
    assert got[0].tolist() == assign and got[1].tolist() == load
    assert max(load) <= C and sum(load) == int(T.sum())
    assert all(load[j] == int(T[got[0] == j].sum()) for j in range(M))


@pytest.mark.parametrize("seed", range(40))
def test_bounds_against_the_exhaustive_optimum(seed):
    rng = np.random.default_rng(13000 + seed)
    n, M = int(rng.integers(1, 10)), int(rng.integers(1, 4))
    T = rng.integers(1, int(rng.choice([6, 40, 1000])), size=n).astype(np.int64)
    opt = brute_opt(T.tolist(), M)
    assert ora.optimal_makespan(T, M) == opt
    assign, load, C = ora.multifit(T, ora.order(T), M)
    # first-fit decreasing succeeds at every capacity from 13/11 of the optimum on (Yue 1990), and the
    # bisection keeps a feasible upper end, so the capacity found is at most that, rounded up
    assert opt <= int(load.max()) <= C <= -(-13 * opt // 11)
    p = rng.integers(1, 50, size=n).astype(np.uint32)
    o = rng.integers(1, 50, size=n).astype(np.uint32)
    both = ora.offline_pack(p, o, M, CM, 0, multifit_steps=64)
    lpt = ora.offline_pack(p, o, M, CM, 0)
    lb = ora.lower_bound(p, o, M, 4, CM)["lb_pack"]
    topt = brute_opt(ora.estimate(p, o, CM).tolist(), M)
    assert lb <= topt <= both["makespan_est"] <= lpt["makespan_est"]
    assert both["packer"] == (1 if both["makespan_est"] < lpt["makespan_est"] else 0)
    if both["packer"] == 0:
        assert np.array_equal(both["assign"], lpt["assign"])


def test_better_of_two_finished_packings():
    """With local-search rounds both starts are improved and the better final packing is kept: never
    worse than the list schedule with the same rounds, the books stay consistent, and the MULTIFIT
    start does win on some instances."""
    rng = np.random.default_rng(5)
    taken = 0
    for case in range(40):
        n, M = int(rng.integers(20, 200)), int(rng.integers(2, 9))
        rounds = (0, 1, 3, 10)[case % 4]
        p = rng.integers(1, 400, size=n).astype(np.uint32)
        o = rng.integers(1, 400, size=n).astype(np.uint32)
        r = ora.offline_pack(p, o, M, CM, rounds, multifit_steps=64)
        plain = ora.offline_pack(p, o, M, CM, rounds)
        T = ora.estimate(p, o, CM)
        assert all(int(r["load"][j]) == int(T[r["assign"] == j].sum()) for j in range(M))
        assert r["makespan_est"] <= plain["makespan_est"]
        assert (r["packer"] == 1) == (r["makespan_est"] < plain["makespan_est"])
        if r["packer"] == 0:
            assert np.array_equal(r["assign"], plain["assign"]) and r["rounds_applied"] == plain["rounds_applied"]
        else:                       # the kept packing is the search started from the MULTIFIT one
            mf = ora.multifit(T, ora.order(T), M, 64)
            a, l, applied, _ = ora.local_search(T, mf[0], mf[1], rounds)
            assert np.array_equal(r["assign"], a) and r["rounds_applied"] == applied
        taken += r["packer"]
    assert taken > 0
