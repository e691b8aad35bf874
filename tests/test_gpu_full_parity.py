"""Full-coverage parity of the two large workloads: every instance of c4 and every simulation of
c3 against the CPU oracle, element by element, in the launch shape the benchmark times.  The
oracle runs one instance per task in a pool of worker processes (tests/oracle_pool.py)."""
import numpy as np
import pytest

from oracle import hos_oracle as ora
from tests import gpu_harness as H
from tests import oracle_pool as OP
from workload import workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hos():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2502_15763_b200 as m
    m.lib()
    return m


@pytest.fixture(scope="module")
def pool():
    pl = OP.make_pool()
    yield pl
    pl.close()
    pl.join()


def same_offline(g, lbv, e, ls_rounds):
    k = e["k"]
    assert g["status"][k] == 0
    assert np.array_equal(g["assign"][k], e["assign"]), f"assign differs in instance {k}"
    assert np.array_equal(g["load"][k], e["load"]), f"load differs in instance {k}"
    assert int(g["makespan_est"][k]) == e["makespan_est"] and int(g["rounds_applied"][k]) == e["rounds_applied"]
    if ls_rounds > 0:
        for f in ("i", "u", "k", "v"):
            assert np.array_equal(g["ls_log"][k][f], e["ls_log"][f]), f"ls_log.{f} differs in instance {k}"
    for f, v in e["lb"].items():
        assert int(lbv[k][f]) == v, f"lower bound field {f} differs in instance {k}"


def same_simulation(cres, sres, status, rec, k, li, M, trace=None, trace_off=None, nl=1):
    got = np.stack([cres[k, li][f].astype(np.uint64) for f in OP.CLIENT_FIELDS[:5]] +
                   [status[k, li].astype(np.int64).astype(np.uint64)], axis=1)
    assert np.array_equal(got, rec["clients"]), f"client results differ: instance {k}, multiplier {li}"
    s = sres[k, li]
    assert int(s["makespan_us"]) == rec["makespan_us"] and int(s["busy_slot_us"]) == rec["busy_slot_us"]
    assert abs(float(s["utilisation"]) - rec["utilisation"]) <= 1e-9 * abs(rec["utilisation"])
    assert abs(float(s["tokens_per_s"]) - rec["tokens_per_s"]) <= 1e-9 * abs(rec["tokens_per_s"])
    assert np.all(np.abs(cres[k, li]["utilisation"] - rec["client_util"]) <= 1e-9 * np.abs(rec["client_util"]))
    if trace is not None and "trace" in rec:
        x0 = (k * nl + li) * M
        lens = np.diff(trace_off[x0:x0 + M + 1])
        assert np.array_equal(lens, rec["trace_len"]), f"trace lengths differ: instance {k}, multiplier {li}"
        gt = trace[int(trace_off[x0]):int(trace_off[x0 + M])]
        for f in ("dur_us", "kind_n", "tokens", "aux"):
            assert np.array_equal(gt[f], rec["trace"][f]), f"trace.{f} differs: instance {k}, multiplier {li}"


def test_config4_every_instance(hos, pool):
    """All 1,024 instances of c4: assignment, loads, move log, bounds, client results and hashes of
    every instance, the full iteration trace of every 16th."""
    from paper_2502_15763_b200.binding import view_struct
    w = workload("c4")
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    g = H.gpu_offline(hos, p, o, M, cap, kv, cm, w.ls_rounds)
    lbv = view_struct(g["lb"], hos.LB_DTYPE)
    s = H.gpu_simulate(hos, p, o, M, cap, kv, cm, g["assign"], w.lambdas_q16, ora.QUEUE_SORTED)
    tasks = [("c4", k, w.ls_rounds, w.lambdas_q16, ora.QUEUE_SORTED, k % 16 == 0, False) for k in range(w.n_inst)]
    seen = 0
    for e in pool.imap_unordered(OP.whole_path, tasks, chunksize=2):
        same_offline(g, lbv, e, w.ls_rounds)
        same_simulation(s["cres"], s["sres"], s["status"], e["sims"][0], e["k"], 0, M, s["trace"], s["trace_off"])
        seen += 1
    assert seen == w.n_inst == 1024
    # what holds at any size, on the whole batch
    T = 40 * p.astype(np.int64) + 350 * o.astype(np.int64)
    assert np.array_equal(g["load"].sum(1), T.sum(1)) and (g["makespan_est"] == g["load"].max(1)).all()
    assert (lbv["lb_pack"] <= g["makespan_est"]).all()
    assert (lbv["lb_sim_us"] <= s["sres"]["makespan_us"][:, 0]).all()
    assert ((s["sres"]["utilisation"] > 0) & (s["sres"]["utilisation"] <= 1)).all()


def test_config3_every_simulation(hos, pool):
    """All 6,400 simulations of the multiplier sweep (100 instances x 64 values): every client result
    and trace hash; full traces on every tenth instance for every eighth value."""
    w = workload("c3")
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    nl = len(w.lambdas_q16)
    g = H.gpu_offline(hos, p, o, M, cap, kv, cm, 0)
    s = H.gpu_simulate(hos, p, o, M, cap, kv, cm, g["assign"], w.lambdas_q16, ora.QUEUE_SORTED)
    tasks = [("c3", k, 0, w.lambdas_q16, ora.QUEUE_SORTED, False, False) for k in range(w.n_inst)]
    tasks += [("c3", k, 0, w.lambdas_q16[::8], ora.QUEUE_SORTED, True, False) for k in range(0, w.n_inst, 10)]
    n_sims = 0
    for t, e in zip(tasks, pool.imap(OP.whole_path, tasks, chunksize=1)):
        k, traced = e["k"], t[5]
        assert np.array_equal(g["assign"][k], e["assign"])
        for x, rec in enumerate(e["sims"]):
            li = x * 8 if traced else x
            same_simulation(s["cres"], s["sres"], s["status"], rec, k, li, M, s["trace"], s["trace_off"], nl)
            n_sims += 0 if traced else 1
    assert n_sims == 6400


def test_request_stealing_config4_shape_every_instance(hos, pool):
    """Algorithm 1's stealing on 40 instances of c4's shape: results, owners and traces of all of them."""
    w = workload("c4").subset(0, 40)
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    g = H.gpu_offline(hos, p, o, M, cap, kv, cm, 0)
    r = H.gpu_simulate_steal(hos, p, o, M, cap, kv, cm, g["assign"], w.lambdas_q16, ora.QUEUE_SORTED)
    tasks = [("c4", k, 0, w.lambdas_q16, ora.QUEUE_SORTED, True, True) for k in range(w.n_inst)]
    for e in pool.imap_unordered(OP.whole_path, tasks, chunksize=1):
        k = e["k"]
        assert np.array_equal(g["assign"][k], e["assign"])
        rec = e["sims"][0]
        assert np.array_equal(r["served_by"][k, 0], rec["served_by"]), f"served_by differs in instance {k}"
        same_simulation(r["cres"], r["sres"], r["status"], rec, k, 0, M, r["trace"], r["trace_off"])
    plain = H.gpu_simulate(hos, p, o, M, cap, kv, cm, g["assign"], w.lambdas_q16, ora.QUEUE_SORTED, want_trace=False)
    assert (r["status"] == 0).all()
    assert ((r["served_by"] >= 0) & (r["served_by"] < M)).all()
    # with balanced queues stealing only matters at the very end: it cannot be much worse
    assert (r["sres"]["makespan_us"][:, 0] <= 1.02 * plain["sres"]["makespan_us"][:, 0]).all()
