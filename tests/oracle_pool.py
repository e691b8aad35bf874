"""The CPU oracle fanned out over the host cores, one instance per task (test infrastructure).

The oracle itself stays single-threaded; independent instances run in separate processes.  The
pool is started with `spawn`, so that a process that has already used the GPU can create it, and
the workers import only numpy, the workload generators and the oracle.  Every task regenerates
its instance from the workload's seed, so nothing but small argument tuples travels to a worker.
"""
from __future__ import annotations

import multiprocessing as mp
import os

import numpy as np

CLIENT_FIELDS = ("makespan_us", "busy_slot_us", "n_prefill_iters", "n_decode_iters", "trace_hash", "status")


def n_workers() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def make_pool(workers: int = 0):
    return mp.get_context("spawn").Pool(workers or n_workers())


def _client_table(sim):
    """[M][6] unsigned table of the integer client results, plus the utilisations."""
    t = np.array([[getattr(c, f) & 0xFFFFFFFFFFFFFFFF for f in CLIENT_FIELDS] for c in sim.clients], dtype=np.uint64)
    u = np.array([c.utilisation for c in sim.clients], dtype=np.float64)
    return t, u


def _traces(sim):
    """The clients' traces back to back and their lengths."""
    lens = np.array([len(c.trace) for c in sim.clients], dtype=np.int64)
    return np.concatenate([c.trace for c in sim.clients]) if len(sim.clients) else None, lens


def whole_path(task):
    """task = (workload name, instance, ls_rounds, multipliers, queue order, want_trace, steal).
    The whole path of one instance on the oracle: pack, bounds, one simulation per multiplier."""
    from oracle import hos_oracle as ora
    from workload import workload
    name, k, ls_rounds, lambdas, mode, want_trace, steal = task
    w = workload(name).subset(k, 1)
    p, o = w.lengths()
    p, o = p[0], o[0]
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    pk = ora.offline_pack(p, o, M, cm, ls_rounds)
    out = dict(k=k, assign=pk["assign"], load=pk["load"], makespan_est=pk["makespan_est"],
               rounds_applied=pk["rounds_applied"], ls_log=pk["ls_log"], lpt_assign=pk["lpt_assign"],
               lb=ora.lower_bound(p, o, M, cap, cm), sims=[])
    # the simulations run on the packing without local search when the rounds belong to a sweep's copies
    for lam in lambdas:
        if steal:
            s, served = ora.simulate_steal(pk["assign"], p, o, M, cm, cap, kv, int(lam), mode, want_trace=want_trace)
        else:
            s, served = ora.simulate(pk["assign"], p, o, M, cm, cap, kv, int(lam), mode, want_trace=want_trace), None
        t, u = _client_table(s)
        rec = dict(clients=t, client_util=u, makespan_us=s.makespan_us, busy_slot_us=s.busy_slot_us,
                   utilisation=s.utilisation, tokens_per_s=s.tokens_per_s, served_by=served)
        if want_trace:
            rec["trace"], rec["trace_len"] = _traces(s)
        out["sims"].append(rec)
    return out
