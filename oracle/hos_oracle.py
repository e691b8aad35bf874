"""ctypes front end of the CPU oracle (oracle/hos_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It never imports the CUDA package and holds no
arithmetic of the method beyond the final per-simulation ratios, which follow
the definitions stated in `simulate`.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hos_oracle.c")
_HDR = os.path.join(_HERE, "hos_oracle.h")
_LIB = os.path.join(_HERE, "libhos_oracle.so")

QUEUE_SORTED = 0
QUEUE_FCFS = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its sources."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-fPIC", "-shared",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Cost(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in (
        "prefill_fixed_us", "prefill_per_token_us", "decode_fixed_us", "decode_per_seq_us",
        "decode_kv_div", "est_per_prompt_token", "est_per_output_token", "n_levels")] + [
        ("level_cap", C.c_uint32 * 8), ("level_time", C.c_uint32 * 8)]


class _Move(C.Structure):
    _fields_ = [("i", C.c_int32), ("u", C.c_int32), ("k", C.c_int32), ("v", C.c_int64)]


class _Lb(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "lb_pack", "sum_T", "max_T", "pair_T", "lb_sim_us", "tp_star_us", "td_star_us", "chain_us",
        "tp_paper_us")]


class _Client(C.Structure):
    _fields_ = [("makespan_us", C.c_int64), ("busy_slot_us", C.c_int64),
                ("n_prefill_iters", C.c_uint32), ("n_decode_iters", C.c_uint32),
                ("trace_hash", C.c_uint64), ("status", C.c_int32)]


REC_DTYPE = np.dtype([("dur_us", "<u4"), ("kind_n", "<u4"), ("tokens", "<u4"), ("aux", "<u4")])
MOVE_DTYPE = np.dtype([("i", "<i4"), ("u", "<i4"), ("k", "<i4"), ("v", "<i8")], align=True)

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ora_local_search.restype = C.c_int
        _lib.ora_multifit.restype = C.c_int
        _lib.ora_optimal_makespan.restype = C.c_int64
    return _lib


def _cost(cm: Sequence) -> _Cost:
    """cm: the seven coefficients, optionally followed by the prefill levels ((cap_tokens, time_us), ...)."""
    c = _Cost(*[int(x) for x in cm[:7]])
    levels = list(cm[7]) if len(cm) > 7 else []
    c.n_levels = len(levels)
    for l, (cap_tokens, time_us) in enumerate(levels):
        c.level_cap[l] = int(cap_tokens)
        c.level_time[l] = int(time_us)
    return c


def _ptr(a: np.ndarray, ty):
    return a.ctypes.data_as(C.POINTER(ty))


def _u32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.uint32)


def estimate(p, o, cm) -> np.ndarray:
    p, o = _u32(p), _u32(o)
    T = np.empty(p.shape[0], dtype=np.int64)
    lib().ora_estimate(C.c_int(p.shape[0]), _ptr(p, C.c_uint32), _ptr(o, C.c_uint32),
                       C.byref(_cost(cm)), _ptr(T, C.c_int64))
    return T


def order(T) -> np.ndarray:
    T = np.ascontiguousarray(T, dtype=np.int64)
    out = np.empty(T.shape[0], dtype=np.int32)
    lib().ora_order(C.c_int(T.shape[0]), _ptr(T, C.c_int64), _ptr(out, C.c_int32))
    return out


def lpt(T, order_, M: int):
    T = np.ascontiguousarray(T, dtype=np.int64)
    order_ = np.ascontiguousarray(order_, dtype=np.int32)
    assign = np.empty(T.shape[0], dtype=np.int32)
    load = np.zeros(M, dtype=np.int64)
    lib().ora_lpt(C.c_int(T.shape[0]), C.c_int(M), _ptr(T, C.c_int64), _ptr(order_, C.c_int32),
                  _ptr(assign, C.c_int32), _ptr(load, C.c_int64))
    return assign, load


def local_search(T, assign, load, rounds: int):
    """Returns (assign, load, applied, log); the inputs are not modified."""
    T = np.ascontiguousarray(T, dtype=np.int64)
    assign = np.array(assign, dtype=np.int32, copy=True)
    load = np.array(load, dtype=np.int64, copy=True)
    log = np.zeros(max(rounds, 0), dtype=MOVE_DTYPE)
    assert MOVE_DTYPE.itemsize == C.sizeof(_Move)
    applied = lib().ora_local_search(
        C.c_int(T.shape[0]), C.c_int(load.shape[0]), _ptr(T, C.c_int64), _ptr(assign, C.c_int32),
        _ptr(load, C.c_int64), C.c_int(rounds),
        log.ctypes.data_as(C.POINTER(_Move)) if rounds > 0 else None)
    return assign, load, int(applied), log


def multifit(T, order_, M: int, max_steps: int = 64):
    """MULTIFIT packing: (assign, load, capacity found), or None if first-fit decreasing fails at it."""
    T = np.ascontiguousarray(T, dtype=np.int64)
    order_ = np.ascontiguousarray(order_, dtype=np.int32)
    assign = np.empty(T.shape[0], dtype=np.int32)
    load = np.zeros(M, dtype=np.int64)
    cfin = C.c_int64(0)
    ok = lib().ora_multifit(C.c_int(T.shape[0]), C.c_int(M), _ptr(T, C.c_int64), _ptr(order_, C.c_int32),
                            C.c_int(max_steps), _ptr(assign, C.c_int32), _ptr(load, C.c_int64), C.byref(cfin))
    return (assign, load, int(cfin.value)) if ok else None


def optimal_makespan(T, M: int) -> int:
    """Optimum of Eq. 26-30 by exhaustive enumeration (tiny instances only)."""
    T = np.ascontiguousarray(T, dtype=np.int64)
    return int(lib().ora_optimal_makespan(C.c_int(T.shape[0]), C.c_int(M), _ptr(T, C.c_int64)))


def lower_bound(p, o, M: int, cap: int, cm) -> dict:
    p, o = _u32(p), _u32(o)
    out = _Lb()
    lib().ora_lower_bound(C.c_int(p.shape[0]), C.c_int(M), C.c_int(cap), _ptr(p, C.c_uint32),
                          _ptr(o, C.c_uint32), C.byref(_cost(cm)), C.byref(out))
    return {n: int(getattr(out, n)) for n, _ in _Lb._fields_}


def queue_build(assign, p, o, M: int, mode: int):
    """Queues by (p + o descending, index); o is what the scheduler knows (exact or estimated)."""
    p, o = _u32(p), _u32(o)
    assign = np.ascontiguousarray(assign, dtype=np.int32)
    q_off = np.empty(M + 1, dtype=np.int32)
    q_req = np.empty(p.shape[0], dtype=np.int32)
    lib().ora_queue_build(C.c_int(p.shape[0]), C.c_int(M), _ptr(assign, C.c_int32),
                          _ptr(p, C.c_uint32), _ptr(o, C.c_uint32), C.c_int(mode),
                          _ptr(q_off, C.c_int32), _ptr(q_req, C.c_int32))
    return q_off, q_req


@dataclass
class ClientResult:
    makespan_us: int
    busy_slot_us: int
    n_prefill_iters: int
    n_decode_iters: int
    trace_hash: int
    status: int
    trace: Optional[np.ndarray] = None
    utilisation: float = 0.0


def simulate_client(queue, p, o, cm, cap: int, kv_budget: int, lambda_q16: int,
                    max_iters: int = 0xFFFFFFFF, want_trace: bool = False,
                    trace_cap: Optional[int] = None, kv_reserve: int = 0) -> ClientResult:
    """Simulate one client's queue (array of request indices into p, o).  kv_reserve > 0: every
    request reserves that many KV tokens instead of p + o."""
    p, o = _u32(p), _u32(o)
    queue = np.ascontiguousarray(queue, dtype=np.int32)
    res = _Client()
    cost = _cost(cm)

    def run(trace, cap_records):
        lib().ora_simulate_client(
            C.c_int(queue.shape[0]), _ptr(queue, C.c_int32), _ptr(p, C.c_uint32), _ptr(o, C.c_uint32),
            C.byref(cost), C.c_int(cap), C.c_int64(kv_budget), C.c_int64(kv_reserve), C.c_uint32(lambda_q16),
            C.c_uint32(max_iters), C.byref(res),
            trace.ctypes.data_as(C.c_void_p) if trace is not None else None, C.c_int64(cap_records))

    trace = None
    if want_trace:
        if trace_cap is None:                       # count first, then fill
            run(None, 0)
            trace_cap = res.n_prefill_iters + res.n_decode_iters
        trace = np.zeros(trace_cap, dtype=REC_DTYPE)
        run(trace, trace_cap)
        trace = trace[: min(trace_cap, res.n_prefill_iters + res.n_decode_iters)]
    else:
        run(None, 0)
    return ClientResult(int(res.makespan_us), int(res.busy_slot_us), int(res.n_prefill_iters),
                        int(res.n_decode_iters), int(res.trace_hash), int(res.status), trace)


@dataclass
class SimResult:
    makespan_us: int
    busy_slot_us: int
    utilisation: float
    tokens_per_s: float
    clients: List[ClientResult]


def simulate(assign, p, o, M: int, cm, cap: int, kv_budget: int, lambda_q16: int, mode: int,
             max_iters: int = 0xFFFFFFFF, want_trace: bool = False, o_est=None, kv_reserve: int = 0) -> SimResult:
    """One (instance, multiplier) simulation: all M clients, then the per-simulation figures.

    makespan = max over clients; busy = sum over clients;
    utilisation_c = busy_c / (cap * makespan), utilisation = busy / (M * cap * makespan)
    (busy slot-time over offered slot-time), tokens_per_s = sum(o) * 1e6 / makespan
    (the paper's "generation speed").  All zero when the makespan is zero.
    o_est: the output lengths the scheduler knows (queue order); the simulation runs on o.
    """
    p, o = _u32(p), _u32(o)
    q_off, q_req = queue_build(assign, p, o if o_est is None else _u32(o_est), M, mode)
    clients = [simulate_client(q_req[q_off[j]:q_off[j + 1]], p, o, cm, cap, kv_budget, lambda_q16,
                               max_iters, want_trace, kv_reserve=kv_reserve) for j in range(M)]
    makespan = max(c.makespan_us for c in clients)
    busy = sum(c.busy_slot_us for c in clients)
    if makespan > 0:
        for c in clients:
            c.utilisation = float(c.busy_slot_us) / (float(cap) * float(makespan))
        util = float(busy) / (float(M) * float(cap) * float(makespan))
        tps = float(int(o.astype(np.int64).sum())) * 1.0e6 / float(makespan)
    else:
        util, tps = 0.0, 0.0
    return SimResult(makespan, busy, util, tps, clients)


def simulate_steal(assign, p, o, M: int, cm, cap: int, kv_budget: int, lambda_q16: int, mode: int,
                   max_iters: int = 0xFFFFFFFF, want_trace: bool = False, o_est=None, kv_reserve: int = 0):
    """One (instance, multiplier) simulation with Algorithm 1's request stealing: clients advance
    in global time order and an idle client takes the longest waiting request of the client with
    the most queued tokens.  Returns (SimResult, served_by)."""
    p, o = _u32(p), _u32(o)
    n = p.shape[0]
    o_key = o if o_est is None else _u32(o_est)
    q_off, q_req = queue_build(assign, p, o_key, M, mode)
    cost = _cost(cm)
    res = (_Client * M)()
    served = np.full(n, -1, dtype=np.int32)

    def run(traces, caps):
        tp = (C.c_void_p * M)(*[t.ctypes.data if t is not None else None for t in traces]) if traces else None
        cp = (C.c_int64 * M)(*caps) if traces else None
        lib().ora_simulate_steal(
            C.c_int(n), C.c_int(M), _ptr(q_off, C.c_int32), _ptr(q_req, C.c_int32), _ptr(p, C.c_uint32),
            _ptr(o, C.c_uint32), _ptr(o_key, C.c_uint32), C.byref(cost), C.c_int(cap), C.c_int64(kv_budget),
            C.c_int64(kv_reserve), C.c_uint32(lambda_q16),
            C.c_uint32(max_iters), res, tp, cp, _ptr(served, C.c_int32))

    run(None, None)
    traces = [None] * M
    if want_trace:
        caps = [int(r.n_prefill_iters + r.n_decode_iters) for r in res]
        traces = [np.zeros(max(k, 1), dtype=REC_DTYPE) for k in caps]
        run(traces, caps)
        traces = [t[:k] for t, k in zip(traces, caps)]
    clients = [ClientResult(int(r.makespan_us), int(r.busy_slot_us), int(r.n_prefill_iters),
                            int(r.n_decode_iters), int(r.trace_hash), int(r.status), traces[j])
               for j, r in enumerate(res)]
    makespan = max(c.makespan_us for c in clients)
    busy = sum(c.busy_slot_us for c in clients)
    if makespan > 0:
        for c in clients:
            c.utilisation = float(c.busy_slot_us) / (float(cap) * float(makespan))
        util = float(busy) / (float(M) * float(cap) * float(makespan))
        tps = float(int(o.astype(np.int64).sum())) * 1.0e6 / float(makespan)
    else:
        util, tps = 0.0, 0.0
    return SimResult(makespan, busy, util, tps, clients), served


def offline_pack(p, o, M: int, cm, ls_rounds: int = 0, multifit_steps: int = 0):
    """estimate -> order -> LPT (-> MULTIFIT) -> local search.  Returns dict with T, order, assign, load, ...

    multifit_steps > 0: the MULTIFIT packing with at most that many probes is improved by the same
    local search, and the better of the two final packings is kept (the longest-first one unless the
    other's largest load is strictly smaller); `packer` says which (0 LPT, 1 MULTIFIT)."""
    T = estimate(p, o, cm)
    od = order(T)
    assign, load = lpt(T, od, M)
    lpt_assign, lpt_load = assign.copy(), load.copy()
    packer = 0
    if multifit_steps > 0:
        mf = multifit(T, od, M, multifit_steps)
        if mf is not None:
            a1, l1, ap1, lg1 = (local_search(T, assign, load, ls_rounds) if ls_rounds > 0
                                else (assign, load, 0, np.zeros(0, dtype=MOVE_DTYPE)))
            a2, l2, ap2, lg2 = (local_search(T, mf[0], mf[1], ls_rounds) if ls_rounds > 0
                                else (mf[0], mf[1], 0, np.zeros(0, dtype=MOVE_DTYPE)))
            if int(l2.max()) < int(l1.max()):
                a1, l1, ap1, lg1, packer = a2, l2, ap2, lg2, 1
            return dict(T=T, order=od, assign=a1, load=l1, makespan_est=int(l1.max()), rounds_applied=ap1,
                        ls_log=lg1, lpt_assign=lpt_assign, lpt_load=lpt_load, packer=packer)
    applied, log = 0, np.zeros(0, dtype=MOVE_DTYPE)
    if ls_rounds > 0:
        assign, load, applied, log = local_search(T, assign, load, ls_rounds)
    return dict(T=T, order=od, assign=assign, load=load, makespan_est=int(load.max()),
                rounds_applied=applied, ls_log=log, lpt_assign=lpt_assign, lpt_load=lpt_load, packer=packer)
